// Blockwise symmetric INT8 quantiser for Q and K (App. C, "Blockwise INT8 Quantization"):
// per block of `blk` rows of one head, delta = absmax/127 and xhat = round(x/delta), in FP32
// with IEEE division and round-half-to-even.  HBM-bound: every FP16 element is read once
// (2 B) and written once as INT8 (1 B); the block is held in registers between the absmax
// reduction and the conversion.
#include <cuda_fp16.h>

#include "common.cuh"
#include "ptx_sm100.cuh"
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

// ---- streaming form ---------------------------------------------------------------------------------------------
// A quantisation block whose rows are contiguous (token stride = d) is one contiguous piece of memory of at most
// 32 KB: one persistent CTA per SM streams its blocks through a ring of such pieces with untiled bulk copies, so
// that ~190 KB per SM are on the way at any time (the loaded HBM latency is several microseconds: the form above,
// whose loads wait in registers, keeps about half of that in flight and reaches 0.73 of the copy rate).  Same
// arithmetic, same results bit for bit.  Up to two tensors (Q and K) in one launch.
// Three groups of eight consumer warps take the blocks in turn (a block's pass -- wait, load, maximum, barrier, convert,
// store -- is a chain of latencies that one group alone cannot hide).
constexpr int kStreamStages = 6, kStageBytes = 32768, kStreamWarps = 8, kStreamGroups = 3;
constexpr int kStreamThreads = (kStreamGroups * kStreamWarps + 1) * 32;

struct QuantJob {
    const __half* x;
    int8_t* out;
    float* scale;
    int64_t s_batch, s_head;
    int H, L, n_blk, blk;
    int first;                 // index of this tensor's first block in the launch
};
struct QuantJobs {
    QuantJob j[2];
    int n_jobs, total, d;
    unsigned long long wait_limit_ns;
    int test_drop_block;       // testing aid: the producer leaves out the copy of this block of every CTA (-1: none)
};

__global__ void __launch_bounds__(kStreamThreads, 1) quantize_stream_kernel(const QuantJobs jobs) {
    extern __shared__ __align__(128) uint8_t ring[];
    __shared__ __align__(8) uint64_t full[kStreamStages], empty[kStreamStages];
    __shared__ uint32_t warp_max[kStreamGroups][2][kStreamWarps];
    __shared__ int abort_flag;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int s = 0; s < kStreamStages; ++s) {
            ptx::mbar_init(ptx::smem_u32(&full[s]), 1);
            ptx::mbar_init(ptx::smem_u32(&empty[s]), kStreamWarps);
        }
        abort_flag = 0;
        ptx::fence_mbar_init();
    }
    __syncthreads();
    const int n_mine = (jobs.total - static_cast<int>(blockIdx.x) + static_cast<int>(gridDim.x) - 1) / static_cast<int>(gridDim.x);
    const int d = jobs.d, vec_per_row = d >> 3;
    // block t of this CTA: tensor, (batch*head, block), rows
    struct Where { const __half* src; int8_t* dst; float* scale; int rows; };
    auto locate = [&](int t) -> Where {
        const int gidx = static_cast<int>(blockIdx.x) + t * static_cast<int>(gridDim.x);
        const QuantJob& jb = jobs.j[(jobs.n_jobs > 1 && gidx >= jobs.j[1].first) ? 1 : 0];
        const int local = gidx - jb.first, bh = local / jb.n_blk, r = local - bh * jb.n_blk;
        const int b = bh / jb.H, h = bh - b * jb.H, row0 = r * jb.blk;
        Where w;
        w.rows = min(jb.blk, jb.L - row0);
        w.src = jb.x + b * jb.s_batch + h * jb.s_head + static_cast<int64_t>(row0) * d;
        w.dst = jb.out + (static_cast<int64_t>(bh) * jb.L + row0) * d;
        w.scale = jb.scale + static_cast<int64_t>(bh) * jb.n_blk + r;
        return w;
    };
    // Bounded wait on one mbarrier phase; false when the CTA is giving up.
    auto wait = [&](uint64_t* bar, uint32_t parity) -> bool {
        const uint32_t addr = ptx::smem_u32(bar);
        if (ptx::mbar_try_wait(addr, parity)) return true;
        const uint64_t start = ptx::globaltimer_ns();
        uint32_t spins = 0;
        while (!ptx::mbar_try_wait(addr, parity)) {
            if ((++spins & 63u) == 0u) {
                if (*reinterpret_cast<volatile int*>(&abort_flag)) return false;
                if (ptx::globaltimer_ns() - start > jobs.wait_limit_ns) {
                    *reinterpret_cast<volatile int*>(&abort_flag) = 1;
                    return false;
                }
            }
        }
        return true;
    };
    int issued = 0;            // (producer lane) blocks whose copy was started
    int done = 0;              // (consumers) blocks finished
    if (warp == kStreamGroups * kStreamWarps) {
        if (lane == 0) {
            for (int t = 0; t < n_mine; ++t) {
                const int s = t % kStreamStages;
                if (t >= kStreamStages && !wait(&empty[s], ((t / kStreamStages) - 1) & 1)) break;
                if (t == jobs.test_drop_block) continue;   // testing aid: this block never lands, the consumers' wait runs out
                const Where w = locate(t);
                const uint32_t bytes = static_cast<uint32_t>(w.rows) * d * 2u;
                const uint32_t bar = ptx::smem_u32(&full[s]);
                ptx::mbar_arrive_expect_tx(bar, bytes);
                ptx::bulk_load_1d(ptx::smem_u32(ring) + s * kStageBytes, w.src, bytes, bar);
                issued = t + 1;
            }
        }
    } else {
        const int grp = warp / kStreamWarps, gw = warp % kStreamWarps, gtid = tid - grp * kStreamWarps * 32;
        for (int t = grp; t < n_mine; t += kStreamGroups) {
            const int s = t % kStreamStages, par = (t / kStreamGroups) & 1;
            if (!wait(&full[s], (t / kStreamStages) & 1)) break;
            const Where w = locate(t);
            const int nvec = w.rows * vec_per_row;
            const uint4* stage = reinterpret_cast<const uint4*>(ring + s * kStageBytes);
            uint4 cache[8];
            uint32_t amax2 = 0u;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int v = gtid + i * (kStreamWarps * 32);
                cache[i] = make_uint4(0u, 0u, 0u, 0u);
                if (v < nvec) cache[i] = stage[v];
                amax2 = umax2(amax2, umax2(umax2(habs2_bits(cache[i].x), habs2_bits(cache[i].y)),
                                           umax2(habs2_bits(cache[i].z), habs2_bits(cache[i].w))));
            }
            uint32_t amax = max(amax2 & 0xffffu, amax2 >> 16);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) amax = max(amax, __shfl_xor_sync(0xffffffffu, amax, o));
            if (lane == 0) warp_max[grp][par][gw] = amax;
            ptx::bar_sync_named(1 + grp, kStreamWarps * 32);   // every warp of the group has its part of the block in registers
            if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&empty[s]));
            amax = 0u;
#pragma unroll
            for (int x = 0; x < kStreamWarps; ++x) amax = max(amax, warp_max[grp][par][x]);
            const float amax_f = __half2float(__ushort_as_half(static_cast<unsigned short>(amax)));
            const float delta = __fdiv_rn(amax_f, 127.0f);
            const float rdelta = __frcp_rn(delta);
            if (gtid == 0) *w.scale = delta;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int v = gtid + i * (kStreamWarps * 32);
                if (v < nvec)
                    *reinterpret_cast<uint2*>(w.dst + static_cast<int64_t>(v) * 8) =
                        amax == 0u ? make_uint2(0u, 0u) : quant8(cache[i], delta, rdelta);   // zero block: delta = 0, xhat = 0
            }
            done = t + kStreamGroups;      // (this group's next block)
        }
    }
    __syncthreads();
    if (*reinterpret_cast<volatile int*>(&abort_flag)) {
        // A wait ran out (a copy that never landed): the copies still in flight land before the shared memory is
        // given back, and the scales of the blocks that were not finished are marked with NaN.
        if (warp == kStreamGroups * kStreamWarps && lane == 0) {
            for (int t = max(0, issued - kStreamStages); t < issued; ++t) {
                if (t == jobs.test_drop_block) continue;
                for (int spin = 0; spin < (1 << 16); ++spin)
                    if (ptx::mbar_try_wait(ptx::smem_u32(&full[t % kStreamStages]), (t / kStreamStages) & 1)) break;
            }
        }
        if (warp < kStreamGroups * kStreamWarps && (tid % (kStreamWarps * 32)) == 0)
            for (int t = max(done, warp / kStreamWarps); t < n_mine; t += kStreamGroups) *locate(t).scale = __int_as_float(0x7fc00000);
    }
}

bool stream_eligible(const int64_t stride[3], int d, int blk) {
    return stride[2] == d && static_cast<int64_t>(blk) * d * 2 <= kStageBytes && (d % 8) == 0;
}

int launch_stream(QuantJobs& jobs, cudaStream_t stream) {
    if (jobs.total > 0x3fffffff) return cudaErrorInvalidConfiguration;
    jobs.wait_limit_ns = g_wait_limit_ns.load();
    jobs.test_drop_block = g_test_drop.load() == 3 ? 1 : -1;
    // SM count and the kernel's shared-memory attribute: asked for / set once per device
    constexpr int kMaxDev = 64;
    static std::atomic<int> sm_count[kMaxDev];
    constexpr int kSmem = kStreamStages * kStageBytes;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return static_cast<int>(e);
    int sms = (dev >= 0 && dev < kMaxDev) ? sm_count[dev].load(std::memory_order_acquire) : 0;
    if (sms == 0) {
        e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(quantize_stream_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem);
        if (e != cudaSuccess) return static_cast<int>(e);
        if (dev >= 0 && dev < kMaxDev) sm_count[dev].store(sms, std::memory_order_release);
    }
    const int grid = jobs.total < sms ? jobs.total : sms;
    quantize_stream_kernel<<<grid, kStreamThreads, kSmem, stream>>>(jobs);
    g_launch_count.fetch_add(1);
    return static_cast<int>(cudaGetLastError());
}

}  // namespace

// Q and K of a dense batch in one launch when both qualify for the streaming form; otherwise one launch each.
int launch_quantize_pair(const void* q, const int64_t qstride[3], int Hq, int blk_q, int8_t* q8, float* qs,
                         const void* k, const int64_t kstride[3], int Hk, int blk_k, int8_t* k8, float* ks,
                         int B, int L, int d, cudaStream_t stream) {
    if (stream_eligible(qstride, d, blk_q) && stream_eligible(kstride, d, blk_k)) {
        const int nq = static_cast<int>(ceil_div(L, blk_q)), nk = static_cast<int>(ceil_div(L, blk_k));
        const int64_t cq = static_cast<int64_t>(B) * Hq * nq, ck = static_cast<int64_t>(B) * Hk * nk;
        if (cq > 0 && ck > 0 && cq + ck <= 0x3fffffff) {
            QuantJobs jobs{};
            jobs.j[0] = QuantJob{static_cast<const __half*>(q), q8, qs, qstride[0], qstride[1], Hq, L, nq, blk_q, 0};
            jobs.j[1] = QuantJob{static_cast<const __half*>(k), k8, ks, kstride[0], kstride[1], Hk, L, nk, blk_k,
                                 static_cast<int>(cq)};
            jobs.n_jobs = 2; jobs.total = static_cast<int>(cq + ck); jobs.d = d;
            return launch_stream(jobs, stream);
        }
    }
    int rc = launch_quantize(q, qstride, B, Hq, L, d, blk_q, q8, qs, stream);
    if (rc) return rc;
    return launch_quantize(k, kstride, B, Hk, L, d, blk_k, k8, ks, stream);
}

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
    if (vl == nullptr && stream_eligible(stride, d, blk)) {
        QuantJobs jobs{};
        jobs.j[0] = QuantJob{xp, out, scale, stride[0], stride[1], H, L, n_blk, blk, 0};
        jobs.n_jobs = 1; jobs.total = static_cast<int>(ctas); jobs.d = d;
        return launch_stream(jobs, stream);
    }
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
