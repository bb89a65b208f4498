// Blockwise symmetric INT8 quantiser for Q and K (App. C, "Blockwise INT8 Quantization"):
// per block of `blk` rows of one head, delta = absmax/127 and xhat = round(x/delta), in FP32
// with IEEE division and round-half-to-even.  HBM-bound: every FP16 element is read once
// (2 B) and written once as INT8 (1 B); the block is held in registers between the absmax
// reduction and the conversion.
#include <cuda_fp16.h>

#include "common.cuh"
#include "quant8.cuh"

namespace tilemix {

namespace {

constexpr int kThreads = 256;

// One CTA per (batch*head, block).  With a variable-length batch (tok != null) the CTA's block index
// runs over the blocks of all sequences; the sequence is found in the block prefix sums, blocks
// restart at each sequence's first token and scales are stored block-major [blocks, H].  MAXV = 16-byte vectors cached per thread; blocks with more
// than kThreads*MAXV vectors re-read the remainder from global memory (L2) in the second pass.
template <int MAXV>
__global__ void __launch_bounds__(kThreads)
quantize_kernel(const __half* __restrict__ x, int64_t s_batch, int64_t s_head, int64_t s_tok,
                int H, int L, int d, int blk, int n_blk, int8_t* __restrict__ out,
                float* __restrict__ scale, const int32_t* __restrict__ tok,
                const int32_t* __restrict__ blk_off, int n_seqs) {
    const int r = blockIdx.x % n_blk;
    const int bh = blockIdx.x / n_blk;
    const int b = bh / H, h = bh % H;
    int row0 = r * blk;
    int rows = min(blk, L - row0);
    int64_t scale_idx = static_cast<int64_t>(bh) * n_blk + r;
    if (tok != nullptr) {
        const int s = find_seq(blk_off, n_seqs, r);
        const int r_loc = r - blk_off[s];
        row0 = tok[s] + r_loc * blk;
        rows = min(blk, tok[s + 1] - row0);
        scale_idx = static_cast<int64_t>(r) * H + h;
    }
    const int vec_per_row = d >> 3;
    const int nvec = rows * vec_per_row;
    const __half* src = x + b * s_batch + h * s_head + static_cast<int64_t>(row0) * s_tok;
    int8_t* dst = out + (static_cast<int64_t>(bh) * L + row0) * d;

    // (row, 16-byte chunk) of this thread's i-th vector, v = threadIdx.x + i * kThreads, kept
    // incrementally: one division per thread instead of one per vector
    const int step_row = kThreads / vec_per_row, step_c8 = kThreads % vec_per_row;
    const int row_first = threadIdx.x / vec_per_row, c8_first = threadIdx.x - row_first * vec_per_row;
    uint4 cache[MAXV > 0 ? MAXV : 1];
    uint32_t amax2 = 0u;
    int row = row_first, c8 = c8_first;
#pragma unroll
    for (int i = 0; i < MAXV; ++i) {
        const int v = threadIdx.x + i * kThreads;
        cache[i] = make_uint4(0u, 0u, 0u, 0u);
        if (v < nvec) cache[i] = __ldg(reinterpret_cast<const uint4*>(src + row * s_tok + c8 * 8));
        row += step_row;
        c8 += step_c8;
        if (c8 >= vec_per_row) { c8 -= vec_per_row; ++row; }
        amax2 = umax2(amax2, umax2(umax2(habs2_bits(cache[i].x), habs2_bits(cache[i].y)),
                                   umax2(habs2_bits(cache[i].z), habs2_bits(cache[i].w))));
    }
    for (int v = threadIdx.x + MAXV * kThreads; v < nvec; v += kThreads) {
        const int row = v / vec_per_row, c8 = v - row * vec_per_row;
        const uint4 t = __ldg(reinterpret_cast<const uint4*>(src + row * s_tok + c8 * 8));
        amax2 = umax2(amax2, umax2(umax2(habs2_bits(t.x), habs2_bits(t.y)),
                                   umax2(habs2_bits(t.z), habs2_bits(t.w))));
    }
    uint32_t amax = max(amax2 & 0xffffu, amax2 >> 16);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) amax = max(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    __shared__ uint32_t warp_max[kThreads / 32];
    if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = amax;
    __syncthreads();
    amax = 0u;
#pragma unroll
    for (int w = 0; w < kThreads / 32; ++w) amax = max(amax, warp_max[w]);

    const float amax_f = __half2float(__ushort_as_half(static_cast<unsigned short>(amax)));
    const float delta = __fdiv_rn(amax_f, 127.0f);
    const float rdelta = __frcp_rn(delta);
    if (threadIdx.x == 0) scale[scale_idx] = delta;

    if (amax == 0u) {  // zero block: delta = 0, xhat = 0 (no division by zero)
        for (int v = threadIdx.x; v < nvec; v += kThreads)
            *reinterpret_cast<uint2*>(dst + static_cast<int64_t>(v) * 8) = make_uint2(0u, 0u);
        return;
    }
#pragma unroll
    for (int i = 0; i < MAXV; ++i) {
        const int v = threadIdx.x + i * kThreads;
        if (v < nvec) *reinterpret_cast<uint2*>(dst + static_cast<int64_t>(v) * 8) = quant8(cache[i], delta, rdelta);
    }
    for (int v = threadIdx.x + MAXV * kThreads; v < nvec; v += kThreads) {
        const int row = v / vec_per_row, c8 = v - row * vec_per_row;
        const uint4 t = __ldg(reinterpret_cast<const uint4*>(src + row * s_tok + c8 * 8));
        *reinterpret_cast<uint2*>(dst + static_cast<int64_t>(v) * 8) = quant8(t, delta, rdelta);
    }
}

}  // namespace

int launch_quantize(const void* x, const int64_t stride[3], int B, int H, int L, int d, int blk,
                    int8_t* out, float* scale, cudaStream_t stream, const VarlenDev* vl,
                    const int32_t* blk_off, int total_blk) {
    const int n_blk = vl ? total_blk : static_cast<int>(ceil_div(L, blk));
    const int32_t* tok = vl ? vl->tok : nullptr;
    const int n_seqs = vl ? vl->n : 0;
    const int64_t ctas = static_cast<int64_t>(B) * H * n_blk;
    if (ctas <= 0) return cudaSuccess;
    if (ctas > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
    const int64_t nvec = static_cast<int64_t>(blk) * d / 8;
    const __half* xp = static_cast<const __half*>(x);
    const dim3 grid(static_cast<unsigned>(ctas));
    if (nvec <= kThreads * 2) {
        quantize_kernel<2><<<grid, kThreads, 0, stream>>>(xp, stride[0], stride[1], stride[2], H, L,
                                                          d, blk, n_blk, out, scale, tok, blk_off, n_seqs);
    } else {
        quantize_kernel<8><<<grid, kThreads, 0, stream>>>(xp, stride[0], stride[1], stride[2], H, L,
                                                          d, blk, n_blk, out, scale, tok, blk_off, n_seqs);
    }
    g_launch_count.fetch_add(1);
    return static_cast<int>(cudaGetLastError());
}

}  // namespace tilemix
