// Decode step over an INT8 key/value cache (App. C, "Additional Execution Interfaces"): one query
// token per sequence, keys split over CTAs, the H_q/H_k query heads of a KV head served together.
// HBM-bound: a cached token costs d bytes of K8 (or 2d of FP16 K on the FP16 route) plus d bytes of
// V8, each read once.  This file holds the host entry points, the preparation and merge kernels, and the
// warp-level form of the step for head_dim 64 or 64-key tiles: the tiles are streamed into a shared-memory
// ring by untiled bulk copies, a tile ahead of their use, and the H_q/H_k query rows of a KV head are the
// rows of a 16-row warp-level tensor-core operand.  head_dim 128 with 128-key tiles runs the tcgen05 form
// (decode_umma.cu), where the KEYS are the MMA rows.
#include <cuda_fp16.h>
#include <math.h>

#include "common.cuh"
#include "decode.cuh"
#include "ptx_sm100.cuh"

namespace tilemix {

namespace {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;


constexpr int kStages = 2;    // ring of key/value tiles in shared memory when FP16 keys may be read ...
constexpr int kStagesInt8 = 3;   // ... and when there is no FP16 key cache (a stage is a third smaller)
constexpr int kChunk = 128;   // keys per kernel tile when tile_n allows it (64-key tiles with deeper rings were slower)

template <int D, int T>
struct Stage {
    static constexpr int kK = T * D * 2;   // room for the FP16 copy of a key tile
    static constexpr int kV = T * D;
    static constexpr int kBytes = kK + kV;
};

// ---- warp-level tensor-core MMAs (m16n8k32 INT8 / m16n8k16 FP16, FP32 or INT32 accumulators) ----------
// Lane l holds, with g = l / 4 and t = l % 4: A rows g (a0, a2) and g + 8 (a1, a3), B column g, C rows g
// (c0, c1) and g + 8 (c2, c3) at columns 2t, 2t + 1.  Only rows 0..R-1 of A are query rows here, so a1 and
// a3 are always zero and c2, c3 stay zero.
__device__ __forceinline__ void mma_s8(int (&c)[4], uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
                 : "r"(a0), "r"(0u), "r"(a2), "r"(0u), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_f16(float (&c)[4], uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(0u), "r"(a2), "r"(0u), "r"(b0), "r"(b1));
}

// D: head dim; R: query heads per KV head; T: keys per tile (= scale block = routing tile).
// Tiles are contiguous in the cache, so they are streamed into a ring of shared-memory stages with
// untiled bulk copies ("full" / "empty" mbarriers per stage), issued by one lane of the last warp
// before it turns to its own share of a tile.  The eight warps never synchronise with one another
// inside the loop: each one owns 16 keys of every tile (and, for
// 64-key tiles, half of the output columns) and runs its own flash-decoding recurrence on them --
//  (1) scores S[R x 16] = Q K^T on the tensor cores, the R query rows being rows 0..R-1 of a 16-row A
//      operand.  The contraction index may be permuted freely as long as Q and K use the same
//      permutation, so lane t simply takes the 16-byte chunks t, t+4, ... of a row;
//  (2) running maximum and sum of its own keys (two shuffles per row), P = 2^(s - m) times delta_V,
//      rounded to FP16 -- the score fragment is already laid out as the A operand of the next product;
//  (3) O~[R x D] += P V8 on the tensor cores.  V8 is converted to FP16 in registers (exactly); the
//      output columns are permuted (column n of block nb is d = (D/8) n + nb) so that the bytes a
//      lane needs from a cached row are contiguous.
// After the loop the eight (m, z, O~) are merged in shared memory like splits.
constexpr int kConsumerWarps = 8;
constexpr int kDecodeThreads = kConsumerWarps * 32;   // 2 CTAs/SM = 4 warps per scheduler: 128 registers each

template <int D, int R, int T, bool F16K>
__global__ void __launch_bounds__(kDecodeThreads, 2)
decode_kernel(const DecodeParams prm) {
    using St = Stage<D, T>;
    constexpr int W8 = D / 16, W16 = D / 8;       // 32-bit words per lane and row: INT8 / FP16 operand
    constexpr int KS3 = T / 16;                   // 16-key steps of a tile
    constexpr int NSPLIT = kConsumerWarps / KS3;  // warps sharing one step (each takes some column blocks)
    constexpr int NBLK = D / 8 / NSPLIT;          // column blocks per warp
    constexpr int BPG = D / 8;                    // bytes of a cached V row per lane group
    static_assert(KS3 <= kConsumerWarps && kConsumerWarps % KS3 == 0, "tile shape vs warps");
    static_assert(kStagesInt8 * 2 * St::kV >= static_cast<int>(kConsumerWarps * R * (D + 2) * sizeof(float)),
                  "the final merge reuses the ring");
    const int split = blockIdx.x, hk = blockIdx.y, b = blockIdx.z;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = lane >> 2, t = lane & 3;
    // (lengths live on the device and cannot be checked by the host: out-of-range values are clamped)
    const int len = prm.cache_len[b];   // the clamped copy decode_prepare_kernel made
    const int n_tiles = (len + T - 1) / T;
    const int per_split = (n_tiles + prm.n_splits - 1) / prm.n_splits;
    const int t0 = split * per_split, t1 = min(n_tiles, t0 + per_split);

    extern __shared__ __align__(128) uint8_t ring[];   // n_stages x (K tile | V tile)
    // without an FP16 key cache a K slot only ever holds INT8 keys: smaller stages, one more of them
    constexpr int n_stages = F16K ? kStages : kStagesInt8;
    constexpr int k_slot = F16K ? St::kK : St::kV;
    constexpr int stage_bytes = k_slot + St::kV;
    __shared__ __align__(16) uint32_t qh[R][D / 2];   // query rows, FP16 pairs (FP16 route)
    __shared__ __align__(16) uint32_t q8w[R][D / 4];  // quantised query rows, 4 bytes per word (INT8 route)
    __shared__ float dq_s[R];
    __shared__ __align__(8) uint64_t full_bar[kStagesInt8], empty_bar[kStagesInt8];
    __shared__ int abort_flag;
    // route bit (sign) and the two block scales of the first kMetaTiles tiles of this split, staged once
    constexpr int kMetaTiles = 256;
    __shared__ float2 meta[kMetaTiles];   // x = delta_K (negative zero / negated: FP16 route), y = delta_V

    const uint32_t ring_u32 = ptx::smem_u32(ring);
    if (tid == 0) {
        for (int s = 0; s < kStagesInt8; ++s) {
            ptx::mbar_init(ptx::smem_u32(&full_bar[s]), 1);
            ptx::mbar_init(ptx::smem_u32(&empty_bar[s]), kConsumerWarps);
        }
        abort_flag = 0;
        ptx::fence_mbar_init();
    }

    // ---- the query rows of this KV head: FP16 copy and blockwise INT8 (block = the row) ----------
    if (warp < R) {
        const int hq = hk * R + warp;
        const __half* qrow = prm.q + (static_cast<int64_t>(b) * prm.Hq + hq) * D;
        float v[D / 32];
        float amax = 0.f;
#pragma unroll
        for (int x = 0; x < D / 32; ++x) {
            v[x] = __half2float(qrow[lane + 32 * x]);
            amax = fmaxf(amax, fabsf(v[x]));
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
        const float delta = __fdiv_rn(amax, 127.f);
#pragma unroll
        for (int x = 0; x < D / 32; ++x) {
            const int e = lane + 32 * x;
            int q8 = 0;
            if (amax > 0.f) q8 = max(-127, min(127, __float2int_rn(__fdiv_rn(v[x], delta))));
            reinterpret_cast<__half*>(&qh[warp][0])[e] = qrow[e];
            reinterpret_cast<int8_t*>(&q8w[warp][0])[e] = static_cast<int8_t>(q8);
            if (split == 0 && prm.q8_out != nullptr)
                prm.q8_out[(static_cast<int64_t>(b) * prm.Hq + hq) * D + e] = static_cast<int8_t>(q8);
        }
        if (lane == 0) {
            dq_s[warp] = delta;
            if (split == 0 && prm.qs_out != nullptr) prm.qs_out[static_cast<int64_t>(b) * prm.Hq + hq] = delta;
        }
    }

    const int64_t row_base = (static_cast<int64_t>(b) * prm.Hk + hk) * prm.max_len;
    const float* dk = prm.k_scale + (static_cast<int64_t>(b) * prm.Hk + hk) * prm.n_blk;
    const float* dv = prm.v_scale + (static_cast<int64_t>(b) * prm.Hk + hk) * prm.n_blk;
    const uint32_t* wrow = prm.words != nullptr
        ? prm.words + (static_cast<int64_t>(prm.nb == 1 ? 0 : b) * prm.Hk + hk) * prm.W : nullptr;
    // the kernel's tile (T keys) may be a fraction of the scale block / routing tile tile_n
    const int per_blk = prm.tile_n / T;
    auto route_of = [&](int tile) -> bool {
        if (wrow == nullptr) return false;
        const int grp = tile / (per_blk * prm.G);
        return (wrow[grp >> 5] >> (grp & 31)) & 1u;
    };
    // Bounded wait on a ring barrier; false when the CTA is giving up.
    auto wait_ring = [&](uint64_t* bar, uint32_t parity) -> bool {
        const uint32_t addr = ptx::smem_u32(bar);
        if (ptx::mbar_try_wait(addr, parity)) return true;
        const uint64_t start = ptx::globaltimer_ns();
        uint32_t spins = 0;
        while (!ptx::mbar_try_wait(addr, parity)) {
            if ((++spins & 63u) == 0u) {
                if (*reinterpret_cast<volatile int*>(&abort_flag)) return false;
                if (ptx::globaltimer_ns() - start > prm.wait_limit_ns) {
                    *reinterpret_cast<volatile int*>(&abort_flag) = 1;
                    return false;
                }
            }
        }
        return true;
    };
    for (int i = tid; i < kMetaTiles && t0 + i < t1; i += kDecodeThreads) {
        const int tile = t0 + i;
        // delta_K >= 0; the FP16 route is marked by a negative x (its delta_K is not used)
        meta[i] = make_float2(route_of(tile) ? dk[tile / per_blk] : -1.f, dv[tile / per_blk]);
    }
    if constexpr (!F16K) {
        // This instance was chosen because no FP16 key cache was passed: every group inside the cache length has
        // to be INT8-routed.  A 0 bit is found here, before any copy is started; the CTA records it and leaves
        // (no access is made, nothing is in flight).
        int fp16_group = 0;
        for (int tile = t0 + tid; tile < t1; tile += kDecodeThreads) fp16_group |= route_of(tile) ? 0 : 1;
        if (__syncthreads_or(fp16_group)) {
            if (tid == 0 && atomicCAS(&prm.status[0], 0, TILEMIX_ERR_NULL) == 0) {
                prm.status[1] = 16; prm.status[2] = t0; prm.status[3] = 1;
            }
            return;
        }
    } else {
        __syncthreads();   // barriers initialised, query rows and tile metadata staged
    }

    // per-warp flash-decoding state: rows g (< R) of this warp's keys
    float m_run = -INFINITY, z_part = 0.f;          // z_part: this lane's share of the row sum
    float acc[NBLK][2];                             // O~ rows g, columns 2t, 2t+1 of this warp's blocks
#pragma unroll
    for (int nb = 0; nb < NBLK; ++nb) acc[nb][0] = acc[nb][1] = 0.f;

    // Refill of the ring by one lane (of the last warp): tile `tile` into its stage, after every warp
    // has handed that stage back.  Returns false when the CTA is giving up.
    const int8_t* k8 = prm.k8 + row_base * D;
    const int8_t* v8 = prm.v8 + row_base * D;
    const __half* k16 = prm.k16 != nullptr ? prm.k16 + row_base * D : nullptr;
    int last_produced = -1;   // (producer lane) the last tile whose copies were started
    auto produce = [&](int tile) -> bool {
        const int it = tile - t0, stage = it % n_stages;
        if (it == prm.test_drop_tile) return true;   // testing aid: this tile never lands, the consumers' bounded wait runs out
        // the first pass over the ring finds every stage free
        if (it >= n_stages && !wait_ring(&empty_bar[stage], ((it / n_stages) - 1) & 1)) return false;
        const uint32_t rows = static_cast<uint32_t>(min(T, len - tile * T));   // only rows that exist
        const uint32_t bar = ptx::smem_u32(&full_bar[stage]);
        const uint32_t dst = ring_u32 + stage * stage_bytes;
        const bool int8 = route_of(tile);
        const uint32_t kbytes = rows * D * (int8 ? 1u : 2u);
        ptx::mbar_arrive_expect_tx(bar, kbytes + rows * D);
        if (int8) ptx::bulk_load_1d(dst, k8 + static_cast<int64_t>(tile) * T * D, kbytes, bar);
        else ptx::bulk_load_1d(dst, k16 + static_cast<int64_t>(tile) * T * D, kbytes, bar);
        ptx::bulk_load_1d(dst + k_slot, v8 + static_cast<int64_t>(tile) * T * D, rows * D, bar);
        last_produced = tile;
        return true;
    };
    const bool producer = warp == kConsumerWarps - 1 && lane == 0;
    if (producer)
        for (int s = 0; s < n_stages - 1 && t0 + s < t1; ++s) produce(t0 + s);
    {
        // ================================================================ consumers
        const int ks = warp / NSPLIT, nb0 = (warp % NSPLIT) * NBLK;   // this warp's keys and column blocks
        const bool counts_z = (warp % NSPLIT) == 0;                    // one warp per key step sums z
        // A fragments of the INT8 route: lane t's words of query row g, in the order the K words are used
        uint32_t qa8[W8];
#pragma unroll
        for (int wi = 0; wi < W8; ++wi) qa8[wi] = g < R ? q8w[g < R ? g : 0][4 * (t + 4 * (wi / 4)) + (wi % 4)] : 0u;
        const float dq = g < R ? dq_s[g < R ? g : 0] : 0.f;

        for (int tile = t0; tile < t1; ++tile) {
            const int it = tile - t0, stage = it % n_stages;
            if (producer && tile + n_stages - 1 < t1) produce(tile + n_stages - 1);   // keeps the ring full
            // route bit and block scales: from shared memory (global loads for tiles beyond the staged ones)
            bool int8;
            float dkt, dvt;
            if (it < kMetaTiles) {
                const float2 mt = meta[it];
                int8 = mt.x >= 0.f;
                dkt = mt.x;
                dvt = mt.y;
            } else {
                int8 = route_of(tile);
                dkt = int8 ? dk[tile / per_blk] : 0.f;
                dvt = dv[tile / per_blk];
            }
            if (!wait_ring(&full_bar[stage], (it / n_stages) & 1)) break;
            const uint8_t* kst = ring + stage * stage_bytes;
            const uint8_t* vst = kst + k_slot;
            // ---- (1) scores of this warp's 16 keys, rows g: s[nb][0..1] = keys 8 nb + 2t, 2t + 1 ----------
            float sc[2][2];
            if (int8) {
                const float a = prm.scale_log2 * dq * dkt;
#pragma unroll
                for (int nb = 0; nb < 2; ++nb) {
                    const uint8_t* krow = kst + (16 * ks + 8 * nb + g) * D;       // B column g = that key
                    uint32_t kw[W8];
#pragma unroll
                    for (int ch = 0; ch < W8 / 4; ++ch) {
                        const uint4 q = *reinterpret_cast<const uint4*>(krow + 16 * (t + 4 * ch));
                        kw[4 * ch] = q.x; kw[4 * ch + 1] = q.y; kw[4 * ch + 2] = q.z; kw[4 * ch + 3] = q.w;
                    }
                    int c[4] = {0, 0, 0, 0};
#pragma unroll
                    for (int k = 0; k < W8 / 2; ++k) mma_s8(c, qa8[2 * k], qa8[2 * k + 1], kw[2 * k], kw[2 * k + 1]);
                    sc[nb][0] = static_cast<float>(c[0]) * a;
                    sc[nb][1] = static_cast<float>(c[1]) * a;
                }
            } else {
                uint32_t qa16[W16];
#pragma unroll
                for (int ch = 0; ch < W16 / 4; ++ch) {
                    uint4 q = make_uint4(0u, 0u, 0u, 0u);
                    if (g < R) q = *reinterpret_cast<const uint4*>(&qh[g < R ? g : 0][4 * (t + 4 * ch)]);
                    qa16[4 * ch] = q.x; qa16[4 * ch + 1] = q.y; qa16[4 * ch + 2] = q.z; qa16[4 * ch + 3] = q.w;
                }
#pragma unroll
                for (int nb = 0; nb < 2; ++nb) {
                    const uint8_t* krow = kst + (16 * ks + 8 * nb + g) * D * 2;
                    float c[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                    for (int ch = 0; ch < W16 / 4; ++ch) {
                        const uint4 q = *reinterpret_cast<const uint4*>(krow + 16 * (t + 4 * ch));
                        mma_f16(c, qa16[4 * ch], qa16[4 * ch + 1], q.x, q.y);
                        mma_f16(c, qa16[4 * ch + 2], qa16[4 * ch + 3], q.z, q.w);
                    }
                    sc[nb][0] = c[0] * prm.scale_log2;
                    sc[nb][1] = c[1] * prm.scale_log2;
                }
            }
            // keys beyond the cached length (stale shared memory) do not exist
            const int j0 = tile * T + 16 * ks + 2 * t;
#pragma unroll
            for (int nb = 0; nb < 2; ++nb) {
                if (j0 + 8 * nb >= len) sc[nb][0] = -INFINITY;
                if (j0 + 8 * nb + 1 >= len) sc[nb][1] = -INFINITY;
            }
            // ---- (2) this warp's online softmax over its own keys ------------------------------------------
            float tmax = fmaxf(fmaxf(sc[0][0], sc[0][1]), fmaxf(sc[1][0], sc[1][1]));
            tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 1));
            tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 2));
            const float m_new = fmaxf(m_run, tmax);
            // a warp whose 16 keys of this tile all lie beyond the cache keeps its state (m_new may be -inf)
            const float m_use = m_new == -INFINITY ? 0.f : m_new;
            const float alpha = exp2f(m_run - m_use);        // 0 on the first keys, 1 if the maximum stands
            float p[2][2];
#pragma unroll
            for (int nb = 0; nb < 2; ++nb) {
                p[nb][0] = exp2f(sc[nb][0] - m_use);
                p[nb][1] = exp2f(sc[nb][1] - m_use);
            }
            z_part = z_part * alpha + ((p[0][0] + p[0][1]) + (p[1][0] + p[1][1]));
            m_run = m_new;
            if (__any_sync(0xffffffffu, alpha != 1.f)) {
#pragma unroll
                for (int nb = 0; nb < NBLK; ++nb) { acc[nb][0] *= alpha; acc[nb][1] *= alpha; }
            }
            // P x delta_V, FP16: the score fragment (row g, keys 2t, 2t+1 of each 8-key block) is the A
            // fragment of the PV product over these 16 keys
            const __half2 h0 = __floats2half2_rn(p[0][0] * dvt, p[0][1] * dvt);
            const __half2 h2 = __floats2half2_rn(p[1][0] * dvt, p[1][1] * dvt);
            const uint32_t pa0 = g < R ? *reinterpret_cast<const uint32_t*>(&h0) : 0u;
            const uint32_t pa2 = g < R ? *reinterpret_cast<const uint32_t*>(&h2) : 0u;
            // ---- (3) O~ += P V8 ------------------------------------------------------------------------------
            // the four cached rows whose pairs this lane feeds: keys 2t, 2t+1 and 2t+8, 2t+9 of the step,
            // at this lane group's columns of this warp's blocks
            const uint8_t* vbase = vst + (16 * ks + 2 * t) * D + BPG * g + nb0;
            const __half2 off = __floats2half2_rn(1152.f, 1152.f);
#pragma unroll
            for (int w = 0; w < NBLK / 4; ++w) {
                // four column blocks at a time: one 32-bit word of each of the four rows
                uint32_t u[4];
#pragma unroll
                for (int r4 = 0; r4 < 4; ++r4)
                    u[r4] = *reinterpret_cast<const uint32_t*>(vbase + ((r4 & 1) + (r4 >> 1) * 8) * D + 4 * w) ^ 0x80808080u;
                if (w == NBLK / 4 - 1) {
                    // last read of this stage by this warp: hand the stage back
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&empty_bar[stage]));
                }
                // bytes of rows (k0, k1) and (k2, k3) interleaved: {k0[e], k1[e]} pairs for e = 0..3
                const uint32_t lo01 = __byte_perm(u[0], u[1], 0x5140), hi01 = __byte_perm(u[0], u[1], 0x7362);
                const uint32_t lo23 = __byte_perm(u[2], u[3], 0x5140), hi23 = __byte_perm(u[2], u[3], 0x7362);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const uint32_t s01 = e < 2 ? lo01 : hi01, s23 = e < 2 ? lo23 : hi23;
                    const uint32_t sel = (e & 1) ? 0x4342u : 0x4140u;
                    // half2(1024 + (x + 128)) - 1152 = half2(x), exactly
                    uint32_t b0 = __byte_perm(s01, 0x64646464u, sel), b1 = __byte_perm(s23, 0x64646464u, sel);
                    const __half2 v0 = __hsub2(*reinterpret_cast<const __half2*>(&b0), off);
                    const __half2 v1 = __hsub2(*reinterpret_cast<const __half2*>(&b1), off);
                    // rows g + 8 of the product do not exist: their accumulators start at 0 and are dropped, so
                    // that the MMAs of different column blocks do not depend on one another
                    float c[4] = {acc[4 * w + e][0], acc[4 * w + e][1], 0.f, 0.f};
                    mma_f16(c, pa0, pa2, *reinterpret_cast<const uint32_t*>(&v0), *reinterpret_cast<const uint32_t*>(&v1));
                    acc[4 * w + e][0] = c[0]; acc[4 * w + e][1] = c[1];
                }
            }
            if (!counts_z) z_part = 0.f;   // the row sum of a key step is counted by one of its warps
        }
    }

    // ---- merge of the eight warps, then (m, z, O~) of this split to the workspace --------------------
    __syncthreads();   // every warp is out of the ring (all copies it waited for have landed)
    if (*reinterpret_cast<volatile int*>(&abort_flag)) {
        if (tid == 0 && atomicCAS(&prm.status[0], 0, TILEMIX_ERR_DEVICE_TIMEOUT) == 0) {
            prm.status[1] = 16; prm.status[2] = t0; prm.status[3] = 0;
        }
        // the copies still in flight land before this CTA's shared memory is given back (each stage's latest one)
        if (producer) {
            for (int tile = max(t0, last_produced - n_stages + 1); tile <= last_produced; ++tile) {
                const int it = tile - t0;
                if (it == prm.test_drop_tile) continue;
                for (int spin = 0; spin < (1 << 16); ++spin)
                    if (ptx::mbar_try_wait(ptx::smem_u32(&full_bar[it % n_stages]), (it / n_stages) & 1)) break;
            }
        }
        return;
    }
    float (*red)[R][D + 2] = reinterpret_cast<float (*)[R][D + 2]>(ring);   // per warp and row: O~[D], m, z
    {
        const int nb0 = (warp % NSPLIT) * NBLK;
        if constexpr (NSPLIT > 1) {
            // warps of one key step hold disjoint column blocks: zero the rest of this warp's plane first
            for (int idx = lane; idx < R * D; idx += 32) red[warp][idx / D][idx % D] = 0.f;
            __syncwarp();
        }
        float z = z_part;
        z += __shfl_xor_sync(0xffffffffu, z, 1);
        z += __shfl_xor_sync(0xffffffffu, z, 2);
        if (g < R) {
#pragma unroll
            for (int nb = 0; nb < NBLK; ++nb) {
                // column n of block nb is d = (D/8) n + nb; this lane holds n = 2t, 2t+1
                red[warp][g][BPG * (2 * t) + nb0 + nb] = acc[nb][0];
                red[warp][g][BPG * (2 * t + 1) + nb0 + nb] = acc[nb][1];
            }
            if (t == 0) { red[warp][g][D] = m_run; red[warp][g][D + 1] = z; }
        }
    }
    __syncthreads();
    for (int idx = tid; idx < R * D; idx += kDecodeThreads) {
        const int r = idx / D, e = idx - r * D;
        float m = -INFINITY;
#pragma unroll
        for (int w = 0; w < kConsumerWarps; ++w) m = fmaxf(m, red[w][r][D]);
        float o = 0.f, z = 0.f;
        if (m > -INFINITY) {
#pragma unroll
            for (int w = 0; w < kConsumerWarps; ++w) {
                const float mw = red[w][r][D];
                if (mw == -INFINITY) continue;
                const float wgt = exp2f(mw - m);
                o += red[w][r][e] * wgt;
                z += red[w][r][D + 1] * wgt;
            }
        }
        const int64_t row = (static_cast<int64_t>(b) * prm.Hq + hk * R + r) * prm.n_splits + split;
        prm.o_part[row * D + e] = o;
        if (e == 0) { prm.m_part[row] = m; prm.z_part[row] = z; }
    }
}

// Merge of the splits: m = max m_s, z = sum z_s 2^(m_s - m), O = sum O~_s 2^(m_s - m) / z.  One block per query head,
// one thread per output element.  The parts are taken 32 at a time: lane s of every warp loads (m_s, z_s) and the
// weights are shared by shuffles, so that the loads of O~_s depend on one round trip only and are in flight
// together (a part that nobody wrote has m_s = -inf, weight 0, and is not loaded).
template <int D>
__global__ void __launch_bounds__(D)
decode_merge_kernel(const float* __restrict__ o_part, const float* __restrict__ m_part,
                    const float* __restrict__ z_part, int n_splits, __half* __restrict__ out,
                    float* __restrict__ lse) {
    ptx::griddep_wait();   // (when launched as a programmatic dependent of the step kernel)
    const int64_t row = blockIdx.x;
    const int e = threadIdx.x, lane = e & 31;
    float m = -INFINITY, z = 0.f, o = 0.f;
    for (int s0 = 0; s0 < n_splits; s0 += 32) {
        const int s = s0 + lane;
        const float ms = s < n_splits ? m_part[row * n_splits + s] : -INFINITY;
        const float zs = s < n_splits ? z_part[row * n_splits + s] : 0.f;
        float mc = ms;
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) mc = fmaxf(mc, __shfl_xor_sync(0xffffffffu, mc, d));
        const float m_new = fmaxf(m, mc);
        if (m_new == -INFINITY) continue;                    // (the same in every lane)
        const float back = m == -INFINITY ? 0.f : exp2f(m - m_new);
        const float w = ms == -INFINITY ? 0.f : exp2f(ms - m_new);
        const float zw = ms == -INFINITY ? 0.f : zs * w;
        z *= back; o *= back; m = m_new;
        const int cnt = min(32, n_splits - s0);
        const float* src = o_part + (row * n_splits + s0) * D + e;
#pragma unroll 8
        for (int i = 0; i < cnt; ++i) {
            const float wi = __shfl_sync(0xffffffffu, w, i);
            z += __shfl_sync(0xffffffffu, zw, i);
            if (wi != 0.f) o += src[static_cast<int64_t>(i) * D] * wi;
        }
    }
    out[row * D + e] = __float2half_rn(z > 0.f ? o / z : 0.f);
    if (e == 0 && lse != nullptr) lse[row] = z > 0.f ? (m + log2f(z)) * kLn2 : -INFINITY;
}

template <int D, int R, int T>
int launch_cfg(const DecodeParams& prm, __half* out, float* lse, cudaStream_t stream) {
    const dim3 grid(prm.n_splits, prm.Hk, prm.B);
    constexpr int kRing = kStages * Stage<D, T>::kBytes;   // = kStagesInt8 stages of INT8 keys and values
    static_assert(kRing == kStagesInt8 * 2 * Stage<D, T>::kV, "both ring shapes fill the same bytes");
    // no FP16 key cache: the instance whose ring holds three INT8-only stages
    auto kernel = prm.k16 != nullptr ? decode_kernel<D, R, T, true> : decode_kernel<D, R, T, false>;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kRing);
    if (e != cudaSuccess) return static_cast<int>(e);
    kernel<<<grid, kDecodeThreads, kRing, stream>>>(prm);
    g_launch_count.fetch_add(1);
    e = cudaGetLastError();
    if (e != cudaSuccess) return static_cast<int>(e);
    decode_merge_kernel<D><<<prm.B * prm.Hq, D, 0, stream>>>(prm.o_part, prm.m_part, prm.z_part, prm.n_splits, out, lse);
    g_launch_count.fetch_add(1);
    return static_cast<int>(cudaGetLastError());
}

template <int D, int T>
int launch_r(int R, const DecodeParams& prm, __half* out, float* lse, cudaStream_t stream) {
    switch (R) {
        case 1: return launch_cfg<D, 1, T>(prm, out, lse, stream);
        case 2: return launch_cfg<D, 2, T>(prm, out, lse, stream);
        case 4: return launch_cfg<D, 4, T>(prm, out, lse, stream);
        case 8: return launch_cfg<D, 8, T>(prm, out, lse, stream);
        default: return TILEMIX_ERR_UNSUPPORTED;
    }
}

constexpr size_t kDecodeStatusBytes = 256;   // status record of the bounded waits
constexpr int kDecodeWave = 148;             // CTAs of one wave of the tcgen05 form (one per SM)
constexpr int kDecodeBalanceRows = 160;      // rows of a batch whose splits that kernel can balance

// Before the step: clears the status record and copies the cache lengths, clamped to [0, max_len], into the
// workspace (they live on the device, so the host cannot check them; the step itself reads the copy).
__global__ void decode_prepare_kernel(const int32_t* __restrict__ cache_len, int B, int max_len, int* status,
                                      int32_t* __restrict__ len_out) {
    ptx::griddep_launch_dependents();   // the step kernel may set itself up meanwhile; it waits before it reads these
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < 4) status[i] = 0;
    if (i < B) len_out[i] = min(max(cache_len[i], 0), max_len);
}

size_t decode_len_bytes(int B) { return (static_cast<size_t>(B) * sizeof(int32_t) + 255) / 256 * 256; }

struct DecodeGeometry {
    int n_blk, T_mask, W, n_splits;
    int n_parts;            // partial results per query head in the workspace (the tcgen05 form writes two per split)
    int balanced, n_ctas, split_cap;   // tcgen05 form with an automatic split count: see DecodeParams
    size_t o_bytes, mz_bytes;
};

int resolve_decode(const tilemix_decode_t* p, DecodeGeometry* g) {
    if (p == nullptr) return TILEMIX_ERR_NULL;
    if (p->batch <= 0 || p->heads_q <= 0 || p->heads_kv <= 0 || p->head_dim <= 0 || p->max_len <= 0 ||
        p->tile_n <= 0 || p->group <= 0 || p->n_splits < -1)
        return TILEMIX_ERR_SHAPE;
    if (p->heads_q % p->heads_kv != 0) return TILEMIX_ERR_SHAPE;
    if (p->mask_batch != 1 && p->mask_batch != p->batch) return TILEMIX_ERR_SHAPE;
    const int R = p->heads_q / p->heads_kv;
    if ((p->head_dim != 64 && p->head_dim != 128) || (p->tile_n != 64 && p->tile_n != 128) ||
        (R != 1 && R != 2 && R != 4 && R != 8))
        return TILEMIX_ERR_UNSUPPORTED;
    g->n_blk = static_cast<int>(ceil_div(p->max_len, p->tile_n));
    g->T_mask = static_cast<int>(ceil_div(p->max_len, static_cast<int64_t>(p->group) * p->tile_n));
    g->W = static_cast<int>(ceil_div(g->T_mask, 32));
    // n_splits: > 0 as given, 0 chosen here (the same for every row), -1 chosen here and, where the kernel can do
    // it, shared out over the rows by the kernel
    const bool balance = p->n_splits == -1;
    int splits = balance ? 0 : p->n_splits;
    const bool umma = p->head_dim == 128 && p->tile_n == 128;   // the tcgen05 form of the step (decode_umma.cu)
    g->balanced = 0; g->n_ctas = 0; g->split_cap = 0;
    if (splits == 0) {
        if (umma) {
            // one CTA per SM, HBM-bound once every SM streams: a single wave, as many splits as fit into it
            // (measured at 8 x 8 KV heads and 32K keys: 2 splits = 128 CTAs 104 us, 9 splits = 3.9 waves 123 us),
            // at least four key tiles per split
            const int64_t n_rows = static_cast<int64_t>(p->batch) * p->heads_kv;
            const int64_t want = kDecodeWave / n_rows;
            splits = static_cast<int>(want < 1 ? 1 : want);
            const int cap = g->n_blk / 4 > 0 ? g->n_blk / 4 : 1;
            if (splits > cap) splits = cap;
            // On request, for a batch whose rows fit one wave: the kernel shares the wave's CTAs out by the rows'
            // cost (cache length, FP16-routed groups), up to split_cap to a row; the workspace has room for that
            // many.  Not the default: with rows of one length it gains ~3 % (the FP16-routed groups differ) and
            // loses ~5 us -- a full wave leaves no SM on which the merge kernel can wait ahead of time.
            if (balance && n_rows <= kDecodeWave && n_rows <= kDecodeBalanceRows) {
                int row_cap = 8 * splits < 16 ? 16 : 8 * splits;
                if (row_cap > cap) row_cap = cap;
                const int64_t ctas = n_rows * row_cap < kDecodeWave ? n_rows * row_cap : kDecodeWave;
                g->balanced = 1; g->n_ctas = static_cast<int>(ctas); g->split_cap = row_cap;
            }
        } else {
            // at most two full waves of two CTAs per SM over the whole batch (measured: more splits cost
            // more in per-CTA set-up and merge than they gain, and a third, partial wave idles a quarter
            // of the GPU), at least two key tiles per split
            const int64_t want = (148 * 2 * 2) / (static_cast<int64_t>(p->batch) * p->heads_kv);
            splits = static_cast<int>(want < 1 ? 1 : want);
            const int cap = g->n_blk / 2 > 0 ? g->n_blk / 2 : 1;
            if (splits > cap) splits = cap;
        }
    }
    if (splits > g->n_blk) splits = g->n_blk;
    if (splits > 65535) return TILEMIX_ERR_UNSUPPORTED;
    g->n_splits = splits;
    g->n_parts = umma ? 2 * (g->balanced ? g->split_cap : splits) : splits;
    const size_t rows = static_cast<size_t>(p->batch) * p->heads_q * g->n_parts;
    g->o_bytes = (rows * p->head_dim * sizeof(float) + 255) / 256 * 256;
    g->mz_bytes = (rows * sizeof(float) + 255) / 256 * 256;
    return TILEMIX_OK;
}

}  // namespace
}  // namespace tilemix

using namespace tilemix;

extern "C" {

size_t tilemix_decode_workspace_size(const tilemix_decode_t* p) {
    DecodeGeometry g;
    if (resolve_decode(p, &g)) return 0;
    return kDecodeStatusBytes + decode_len_bytes(p->batch) + g.o_bytes + 2 * g.mz_bytes;
}

int tilemix_decode_int8kv(const tilemix_decode_t* p, const void* q_f16, const void* k_f16, const int8_t* k_i8,
                          const float* k_scale, const int8_t* v_i8, const float* v_scale,
                          const uint32_t* mask_words, const int32_t* cache_len, void* out_f16, float* lse,
                          int8_t* q_i8_out, float* q_scale_out, void* workspace, size_t workspace_bytes,
                          void* stream) {
    DecodeGeometry g;
    int rc = resolve_decode(p, &g);
    if (rc) return rc;
    if (!q_f16 || !k_i8 || !k_scale || !v_i8 || !v_scale || !cache_len || !out_f16 || !workspace) return TILEMIX_ERR_NULL;
    if (mask_words == nullptr && k_f16 == nullptr) return TILEMIX_ERR_NULL;   // all FP16 needs the FP16 cache
    if (!aligned16(q_f16) || !aligned16(k_i8) || !aligned16(v_i8) || !aligned16(out_f16) || !aligned16(workspace) ||
        (k_f16 && !aligned16(k_f16)))
        return TILEMIX_ERR_ALIGN;
    if (workspace_bytes < kDecodeStatusBytes + decode_len_bytes(p->batch) + g.o_bytes + 2 * g.mz_bytes) return TILEMIX_ERR_WORKSPACE;
    DecodeParams prm{};
    prm.B = p->batch; prm.Hq = p->heads_q; prm.Hk = p->heads_kv; prm.max_len = p->max_len; prm.G = p->group;
    prm.nb = p->mask_batch; prm.W = g.W; prm.n_splits = g.n_splits; prm.n_blk = g.n_blk;
    prm.tile_n = p->tile_n;
    prm.n_parts = g.n_parts; prm.balanced = g.balanced; prm.n_rows = p->batch * p->heads_kv;
    prm.n_ctas = g.n_ctas; prm.split_cap = g.split_cap;
    const float scale = p->softmax_scale > 0.f ? p->softmax_scale : 1.0f / sqrtf(static_cast<float>(p->head_dim));
    prm.scale_log2 = scale * kLog2e;
    prm.q = static_cast<const __half*>(q_f16);
    prm.k16 = static_cast<const __half*>(k_f16);
    prm.k8 = k_i8; prm.k_scale = k_scale; prm.v8 = v_i8; prm.v_scale = v_scale;
    prm.words = mask_words;
    prm.status = static_cast<int*>(workspace);
    prm.wait_limit_ns = g_wait_limit_ns.load();
    prm.test_drop_tile = g_test_drop.load() == 2 ? 1 : -1;
    int32_t* len_ws = reinterpret_cast<int32_t*>(static_cast<uint8_t*>(workspace) + kDecodeStatusBytes);
    prm.cache_len = len_ws;
    prm.cache_len_raw = cache_len;
    uint8_t* ws = static_cast<uint8_t*>(workspace) + kDecodeStatusBytes + decode_len_bytes(p->batch);
    prm.o_part = reinterpret_cast<float*>(ws);
    prm.m_part = reinterpret_cast<float*>(ws + g.o_bytes);
    prm.z_part = reinterpret_cast<float*>(ws + g.o_bytes + g.mz_bytes);
    prm.q8_out = q_i8_out; prm.qs_out = q_scale_out;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int R = p->heads_q / p->heads_kv;
    __half* out = static_cast<__half*>(out_f16);
    const int prep_threads = p->batch > 4 ? p->batch : 4;
    decode_prepare_kernel<<<(prep_threads + 255) / 256, 256, 0, s>>>(cache_len, p->batch, p->max_len, prm.status, len_ws);
    g_launch_count.fetch_add(1);
    cudaError_t pe = cudaGetLastError();
    if (pe != cudaSuccess) return static_cast<int>(pe);
    // keys are streamed and processed one routing tile at a time (64-key chunks with a deeper ring
    // were slower: the per-chunk barriers cost more than the extra bytes in flight gain)
    if (p->head_dim == 128 && p->tile_n == 128) {
        // the tcgen05 form of the step (decode_umma.cu), then the same merge
        rc = launch_decode_umma(R, prm, s);
        if (rc) return rc;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(prm.B * prm.Hq); cfg.blockDim = dim3(128); cfg.stream = s;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr; cfg.numAttrs = 1;
        const cudaError_t me = cudaLaunchKernelEx(&cfg, decode_merge_kernel<128>, static_cast<const float*>(prm.o_part),
                                                  static_cast<const float*>(prm.m_part), static_cast<const float*>(prm.z_part),
                                                  g.n_parts, out, lse);
        g_launch_count.fetch_add(1);
        return static_cast<int>(me);
    }
    if (p->head_dim == 128 && p->tile_n == 64) return launch_r<128, 64>(R, prm, out, lse, s);
    if (p->head_dim == 64 && p->tile_n == 128) return launch_r<64, kChunk>(R, prm, out, lse, s);
    if (p->head_dim == 64 && p->tile_n == 64) return launch_r<64, 64>(R, prm, out, lse, s);
    return TILEMIX_ERR_UNSUPPORTED;
}

}  // extern "C"
