// Issue-rate probe of the tensor pipe: the denominators of the attention kernel's roofline, measured on the same
// GPU in the same run.  One CTA per SM issues back-to-back tcgen05.mma instructions of the shape the fused kernel
// uses for a full score tile -- M128 N128, K16 for kind::f16 and K32 for kind::i8, both operands in shared memory
// (contents irrelevant: zeros) -- into one accumulator, and returns when they have retired.  The caller times the
// launch with events: ops = CTAs x n_mma x 2*128*128*K.
#include <cuda.h>

#include "common.cuh"
#include "ptx_sm100.cuh"

namespace tilemix {
namespace {

constexpr int kProbeSmem = 64 * 1024 + 1024;

template <bool INT8>
__global__ void __launch_bounds__(128, 1) tensor_probe_kernel(int n_mma, int* status) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sbase = ptx::smem_u32(smem);
    __shared__ uint32_t tmem_base;
    __shared__ __align__(8) uint64_t done;
    const int warp = threadIdx.x >> 5;
    for (int i = threadIdx.x; i < 64 * 1024 / 4; i += blockDim.x) reinterpret_cast<uint32_t*>(smem)[i] = 0u;
    if (threadIdx.x == 0) {
        ptx::mbar_init(ptx::smem_u32(&done), 1);
        ptx::fence_mbar_init();
    }
    if (warp == 0) {
        ptx::tmem_alloc(ptx::smem_u32(&tmem_base), 128);
        ptx::tmem_relinquish();
    }
    ptx::fence_proxy_async_smem();
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    if (warp == 1) {   // the whole warp runs the loop, one elected lane issues
        // A: 128 rows x 128 bytes at sbase, B: 128 rows x 128 bytes at sbase + 32 KB, both K-major with the
        // 128-byte swizzle; one K step advances 32 bytes inside the swizzle atom (+2 in the descriptor)
        constexpr uint32_t hi = ptx::desc_hi(1024, 2);
        const uint32_t a_lo = ptx::desc_lo(sbase, 16), b_lo = ptx::desc_lo(sbase + 32768, 16);
        constexpr uint32_t idesc = INT8 ? ptx::instr_desc(2, 1, 0, 0, 128, 128) : ptx::instr_desc(1, 0, 0, 0, 128, 128);
        for (int i = 0; i < n_mma; ++i) {
            if (INT8) ptx::mma_i8_ss<true>(tmem_base, a_lo + 2 * (i & 3), hi, b_lo + 2 * (i & 3), hi, idesc);
            else ptx::mma_f16_ss<true>(tmem_base, a_lo + 2 * (i & 3), hi, b_lo + 2 * (i & 3), hi, idesc);
        }
        ptx::mma_commit(ptx::smem_u32(&done));
        // bounded wait: n_mma instructions of at most a few hundred clocks each
        bool ok = false;
        for (long long spin = 0; spin < 64ll * n_mma + (1 << 20); ++spin)
            if (ptx::mbar_try_wait(ptx::smem_u32(&done), 0)) { ok = true; break; }
        if (!ok && threadIdx.x == 32) atomicExch(status, TILEMIX_ERR_DEVICE_TIMEOUT);
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, 128);
    }
}

}  // namespace
}  // namespace tilemix

extern "C" int tilemix_tensor_peak_probe(int int8, int n_mma, int* n_ctas, void* workspace, void* stream) {
    using namespace tilemix;
    if (n_mma <= 0 || n_mma > (1 << 22) || workspace == nullptr) return TILEMIX_ERR_SHAPE;
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return static_cast<int>(e);
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return static_cast<int>(e);
    if (n_ctas) *n_ctas = sms;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    e = cudaMemsetAsync(workspace, 0, 16, s);
    if (e != cudaSuccess) return static_cast<int>(e);
    auto kernel = int8 ? tensor_probe_kernel<true> : tensor_probe_kernel<false>;
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kProbeSmem);
    if (e != cudaSuccess) return static_cast<int>(e);
    kernel<<<sms, 128, kProbeSmem, s>>>(n_mma, static_cast<int*>(workspace));
    g_launch_count.fetch_add(1);
    return static_cast<int>(cudaGetLastError());
}
