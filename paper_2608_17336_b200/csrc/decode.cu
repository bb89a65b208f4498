// Decode step over an INT8 key/value cache (App. C, "Additional Execution Interfaces"): one query
// token per sequence, keys split over CTAs, the H_q/H_k query heads of a KV head served together.
// HBM-bound: a cached token costs d bytes of K8 (or 2d of FP16 K on the FP16 route) plus d bytes of
// V8, each read once: the tiles are contiguous in the cache and are streamed into a shared-memory ring
// by untiled bulk copies, a tile ahead of their use.  All arithmetic is on the CUDA cores (dp4a for the
// INT8 route), because with at most 8 query rows per KV head there is no tile for the tensor cores to
// work on.
#include <cuda_fp16.h>
#include <math.h>

#include "common.cuh"
#include "ptx_sm100.cuh"

namespace tilemix {

namespace {

constexpr int kThreads = 256;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

struct DecodeParams {
    int B, Hq, Hk, max_len, G, nb, W, n_splits, n_blk;
    float scale_log2;
    const __half* q;
    const __half* k16;
    const int8_t* k8;
    const float* k_scale;
    const int8_t* v8;
    const float* v_scale;
    const uint32_t* words;
    const int32_t* cache_len;
    float* o_part;   // [B, Hq, n_splits, D]
    float* m_part;   // [B, Hq, n_splits]
    float* z_part;
    int8_t* q8_out;
    float* qs_out;
    int* status;     // 4 ints at the start of the workspace (same record as the attention kernel's)
};

__device__ __forceinline__ float round_to_half(float x) { return __half2float(__float2half_rn(x)); }

// 4 signed bytes of `w` -> 4 floats, without the conversion unit: byte b of (w ^ 0x80808080) placed in
// the low mantissa byte of 2^23 gives the float 2^23 + (x + 128); subtracting 2^23 + 128 is exact.
__device__ __forceinline__ void bytes_to_floats(uint32_t w, float2 (&f)[2]) {
    const uint32_t u = w ^ 0x80808080u;
    const float2 bias = make_float2(-8388736.f, -8388736.f);
    f[0] = __fadd2_rn(make_float2(__uint_as_float(__byte_perm(u, 0x4B000000u, 0x7650)),
                                  __uint_as_float(__byte_perm(u, 0x4B000000u, 0x7651))), bias);
    f[1] = __fadd2_rn(make_float2(__uint_as_float(__byte_perm(u, 0x4B000000u, 0x7652)),
                                  __uint_as_float(__byte_perm(u, 0x4B000000u, 0x7653))), bias);
}

constexpr int kStages = 2;                 // ring of key/value tiles in shared memory
constexpr uint64_t kTimeoutNs = 2000000000ull;

template <int D, int T>
struct Stage {
    static constexpr int kK = T * D * 2;   // room for the FP16 copy of a key tile
    static constexpr int kV = T * D;
    static constexpr int kBytes = kK + kV;
};

// Bounded wait on a "tile landed" barrier; false when the time limit ran out.
__device__ __forceinline__ bool wait_tile(uint32_t bar, uint32_t parity) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = ptx::globaltimer_ns();
    uint32_t it = 0;
    while (!ptx::mbar_try_wait(bar, parity)) {
        if ((++it & 63u) == 0u && ptx::globaltimer_ns() - t0 > kTimeoutNs) return false;
    }
    return true;
}

// D: head dim; R: query heads per KV head; T: key tile (= scale block).
// Key/value tiles are contiguous in the cache, so one thread streams them into a ring of shared-
// memory stages with untiled bulk copies a tile ahead of their use; with two CTAs per SM this keeps
// ~64 KB per SM in flight.  Per tile: (1) scores of all 256 threads from the K stage, (2) the online
// softmax of each query row by one warp, (3) the PV sums from the V stage.
template <int D, int R, int T>
__global__ void __launch_bounds__(kThreads, (R <= 4 ? 2 : 1))
decode_kernel(const DecodeParams prm) {
    constexpr int CH = D / 16;           // 16-byte chunks (lanes) per cached row
    constexpr int KPP = kThreads / CH;   // keys per pass of the CTA
    constexpr int KPT = T / KPP;         // keys per thread per tile
    using St = Stage<D, T>;
    static_assert(KPT >= 1 && T % KPP == 0, "tile too small for the thread mapping");
    static_assert(kStages * St::kBytes >= static_cast<int>(kThreads / 32 * R * D * sizeof(float)),
                  "the final reduction reuses the ring");
    const int split = blockIdx.x, hk = blockIdx.y, b = blockIdx.z;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int slot = tid / CH, c = tid % CH;   // key slot of a pass, chunk of the row
    const int len = prm.cache_len[b];
    const int n_tiles = (len + T - 1) / T;
    const int per_split = (n_tiles + prm.n_splits - 1) / prm.n_splits;
    const int t0 = split * per_split, t1 = min(n_tiles, t0 + per_split);

    extern __shared__ __align__(128) uint8_t ring[];   // kStages x (K tile | V tile)
    __shared__ __align__(16) uint32_t qh[R][D / 2];   // query rows, FP16 pairs (FP16 route)
    __shared__ __align__(16) uint32_t q8w[R][D / 4];  // quantised query rows, 4 bytes per word (INT8 route)
    __shared__ float dq_s[R];
    __shared__ float S[2][R][T];               // scores, then probabilities with delta_V folded in
    __shared__ float alpha_s[2][R];
    __shared__ __align__(8) uint64_t full_bar[kStages];

    const uint32_t ring_u32 = ptx::smem_u32(ring);
    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) ptx::mbar_init(ptx::smem_u32(&full_bar[s]), 1);
        ptx::fence_mbar_init();
    }

    // ---- the query rows of this KV head: FP32 copy and blockwise INT8 (block = the row) ----------
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
    const int8_t* k8 = prm.k8 + row_base * D;
    const int8_t* v8 = prm.v8 + row_base * D;
    const __half* k16 = prm.k16 != nullptr ? prm.k16 + row_base * D : nullptr;
    const float* dk = prm.k_scale + (static_cast<int64_t>(b) * prm.Hk + hk) * prm.n_blk;
    const float* dv = prm.v_scale + (static_cast<int64_t>(b) * prm.Hk + hk) * prm.n_blk;
    const uint32_t* wrow = prm.words != nullptr
        ? prm.words + (static_cast<int64_t>(prm.nb == 1 ? 0 : b) * prm.Hk + hk) * prm.W : nullptr;
    auto route_of = [&](int tile) -> bool {
        if (wrow == nullptr) return false;
        const int g = tile / prm.G;
        return (wrow[g >> 5] >> (g & 31)) & 1u;
    };
    // One thread streams a tile (the K copy its group is routed to, and V8; only the rows that exist).
    auto issue = [&](int tile, int stage) {
        const uint32_t rows = static_cast<uint32_t>(min(T, len - tile * T));
        const uint32_t bar = ptx::smem_u32(&full_bar[stage]);
        const uint32_t dst = ring_u32 + stage * St::kBytes;
        const bool int8 = route_of(tile);
        const uint32_t kbytes = rows * D * (int8 ? 1u : 2u);
        ptx::mbar_arrive_expect_tx(bar, kbytes + rows * D);
        if (int8) ptx::bulk_load_1d(dst, k8 + static_cast<int64_t>(tile) * T * D, kbytes, bar);
        else ptx::bulk_load_1d(dst, k16 + static_cast<int64_t>(tile) * T * D, kbytes, bar);
        ptx::bulk_load_1d(dst + St::kK, v8 + static_cast<int64_t>(tile) * T * D, rows * D, bar);
    };
    __syncthreads();   // barriers initialised, query rows staged
    if (tid == 0)
        for (int s = 0; s < kStages - 1 && t0 + s < t1; ++s) issue(t0 + s, s);

    float2 acc[R][8];
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[r][e] = make_float2(0.f, 0.f);
    float m_run = -INFINITY, z_run = 0.f;     // state of query row `warp` (warps < R), same in all lanes
    // this thread's 16 columns of every quantised query row, kept in registers for the whole CTA
    uint4 q8r[R];
#pragma unroll
    for (int r = 0; r < R; ++r) q8r[r] = *reinterpret_cast<const uint4*>(&q8w[r][4 * c]);

    for (int tile = t0; tile < t1; ++tile) {
        const int it = tile - t0;
        const int buf = it & 1, stage = it % kStages;
        const bool int8 = route_of(tile);
        const bool landed = wait_tile(ptx::smem_u32(&full_bar[stage]), (it / kStages) & 1);
        // Everyone is past the previous tile here, so its stage can be refilled.
        if (__syncthreads_or(!landed)) {
            if (tid == 0 && atomicCAS(&prm.status[0], 0, TILEMIX_ERR_DEVICE_TIMEOUT) == 0) {
                prm.status[1] = 16; prm.status[2] = tile; prm.status[3] = 0;
            }
            return;   // no copy of this CTA is known to be in flight into a stage it would still read
        }
        if (tid == 0 && tile + kStages - 1 < t1) issue(tile + kStages - 1, (it + kStages - 1) % kStages);
        const uint8_t* kst = ring + stage * St::kBytes;
        const uint8_t* vst = kst + St::kK;
        // ---- phase 1: scores of the tile (log2 domain) --------------------------------------
        const float dkt = int8 ? dk[tile] : 0.f;
#pragma unroll
        for (int kt = 0; kt < KPT; ++kt) {
            const int key = kt * KPP + slot;
            const int j = tile * T + key;
            float s[R];
            if (int8) {
                uint4 kq = make_uint4(0u, 0u, 0u, 0u);
                if (j < len) kq = *reinterpret_cast<const uint4*>(kst + key * D + 16 * c);
                int dot[R];
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    dot[r] = __dp4a(static_cast<int>(kq.x), static_cast<int>(q8r[r].x), 0);
                    dot[r] = __dp4a(static_cast<int>(kq.y), static_cast<int>(q8r[r].y), dot[r]);
                    dot[r] = __dp4a(static_cast<int>(kq.z), static_cast<int>(q8r[r].z), dot[r]);
                    dot[r] = __dp4a(static_cast<int>(kq.w), static_cast<int>(q8r[r].w), dot[r]);
                }
#pragma unroll
                for (int r = 0; r < R; ++r) {
#pragma unroll
                    for (int o = CH / 2; o > 0; o >>= 1) dot[r] += __shfl_xor_sync(0xffffffffu, dot[r], o);
                    s[r] = static_cast<float>(dot[r]) * (prm.scale_log2 * dq_s[r] * dkt);
                }
            } else {
                uint4 k0 = make_uint4(0u, 0u, 0u, 0u), k1 = k0;
                if (j < len) {
                    const uint4* src = reinterpret_cast<const uint4*>(kst + (key * D + 16 * c) * 2);
                    k0 = src[0];
                    k1 = src[1];
                }
                const uint32_t kw[8] = {k0.x, k0.y, k0.z, k0.w, k1.x, k1.y, k1.z, k1.w};
                float2 kf[8];
#pragma unroll
                for (int w = 0; w < 8; ++w) kf[w] = __half22float2(*reinterpret_cast<const __half2*>(&kw[w]));
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    // this thread's 16 columns of query row r (two 16-byte reads, the same for every key)
                    const uint4 qa = *reinterpret_cast<const uint4*>(&qh[r][8 * c]);
                    const uint4 qb = *reinterpret_cast<const uint4*>(&qh[r][8 * c + 4]);
                    const uint32_t qw[8] = {qa.x, qa.y, qa.z, qa.w, qb.x, qb.y, qb.z, qb.w};
                    float dot = 0.f;
#pragma unroll
                    for (int w = 0; w < 8; ++w) {
                        const float2 qv = __half22float2(*reinterpret_cast<const __half2*>(&qw[w]));
                        dot = fmaf(kf[w].x, qv.x, dot);
                        dot = fmaf(kf[w].y, qv.y, dot);
                    }
#pragma unroll
                    for (int o = CH / 2; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
                    s[r] = dot * prm.scale_log2;
                }
            }
            if (c == 0) {
#pragma unroll
                for (int r = 0; r < R; ++r) S[buf][r][key] = j < len ? s[r] : -INFINITY;
            }
        }
        __syncthreads();
        // ---- phase 2: online softmax of query row `warp`; P gets delta_V and is rounded to FP16 ----
        if (warp < R) {
            float sv[T / 32];
            float tmax = -INFINITY;
#pragma unroll
            for (int x = 0; x < T / 32; ++x) {
                sv[x] = S[buf][warp][lane + 32 * x];
                tmax = fmaxf(tmax, sv[x]);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, o));
            const float m_new = fmaxf(m_run, tmax);       // finite: the tile holds at least one key
            const float alpha = exp2f(m_run - m_new);     // 0 on the first tile
            const float dvt = dv[tile];
            float sum = 0.f;
#pragma unroll
            for (int x = 0; x < T / 32; ++x) {
                const float p = exp2f(sv[x] - m_new);
                sum += p;
                S[buf][warp][lane + 32 * x] = round_to_half(p * dvt);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
            z_run = z_run * alpha + sum;
            m_run = m_new;
            if (lane == 0) alpha_s[buf][warp] = alpha;
        }
        __syncthreads();
        // ---- phase 3: O~ = alpha * O~ + P V8 over this thread's keys and 16 columns ----------------
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const float a = alpha_s[buf][r];     // the same for the whole CTA; 1 unless the maximum moved
            if (a != 1.f) {
                const float2 a2 = make_float2(a, a);
#pragma unroll
                for (int e = 0; e < 8; ++e) acc[r][e] = __fmul2_rn(acc[r][e], a2);
            }
        }
#pragma unroll
        for (int kt = 0; kt < KPT; ++kt) {
            const int key = kt * KPP + slot;
            if (tile * T + key >= len) continue;       // rows that were not copied
            const uint4 vq = *reinterpret_cast<const uint4*>(vst + key * D + 16 * c);
            const uint32_t vw[4] = {vq.x, vq.y, vq.z, vq.w};
            float2 vf[8];
#pragma unroll
            for (int w = 0; w < 4; ++w) bytes_to_floats(vw[w], *reinterpret_cast<float2(*)[2]>(&vf[2 * w]));
#pragma unroll
            for (int r = 0; r < R; ++r) {
                const float p = S[buf][r][key];
                const float2 pp = make_float2(p, p);
#pragma unroll
                for (int e = 0; e < 8; ++e) acc[r][e] = __ffma2_rn(vf[e], pp, acc[r][e]);
            }
        }
        // the next tile writes the other score buffer; the sync at its top orders the reuse of the stage
    }

    // ---- partial result of this split: sum over the key slots, then (m, z, O~) to the workspace -----
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
        for (int e = 0; e < 8; ++e) {
#pragma unroll
            for (int o = CH; o < 32; o <<= 1) {
                acc[r][e].x += __shfl_xor_sync(0xffffffffu, acc[r][e].x, o);
                acc[r][e].y += __shfl_xor_sync(0xffffffffu, acc[r][e].y, o);
            }
        }
    __syncthreads();   // every thread is done with the ring: reuse it for the reduction over the warps
    float (*red)[R][D] = reinterpret_cast<float (*)[R][D]>(ring);
    if (lane < CH) {
#pragma unroll
        for (int r = 0; r < R; ++r)
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                red[warp][r][16 * lane + 2 * e] = acc[r][e].x;
                red[warp][r][16 * lane + 2 * e + 1] = acc[r][e].y;
            }
    }
    __syncthreads();
    for (int idx = tid; idx < R * D; idx += kThreads) {
        const int r = idx / D, e = idx - r * D;
        float o = 0.f;
#pragma unroll
        for (int w = 0; w < kThreads / 32; ++w) o += red[w][r][e];
        const int64_t row = (static_cast<int64_t>(b) * prm.Hq + hk * R + r) * prm.n_splits + split;
        prm.o_part[row * D + e] = o;
    }
    if (warp < R && lane == 0) {
        const int64_t row = (static_cast<int64_t>(b) * prm.Hq + hk * R + warp) * prm.n_splits + split;
        prm.m_part[row] = m_run;
        prm.z_part[row] = z_run;
    }
}

// Merge of the splits: m = max m_s, z = sum z_s 2^(m_s - m), O = sum O~_s 2^(m_s - m) / z.
template <int D>
__global__ void __launch_bounds__(D)
decode_merge_kernel(const float* __restrict__ o_part, const float* __restrict__ m_part,
                    const float* __restrict__ z_part, int n_splits, __half* __restrict__ out,
                    float* __restrict__ lse) {
    const int64_t row = blockIdx.x;
    const int e = threadIdx.x;
    float m = -INFINITY;
    for (int s = 0; s < n_splits; ++s) m = fmaxf(m, m_part[row * n_splits + s]);
    float z = 0.f, o = 0.f;
    if (m > -INFINITY) {
        for (int s = 0; s < n_splits; ++s) {
            const float ms = m_part[row * n_splits + s];
            if (ms == -INFINITY) continue;
            const float w = exp2f(ms - m);
            z += z_part[row * n_splits + s] * w;
            o += o_part[(row * n_splits + s) * D + e] * w;
        }
    }
    out[row * D + e] = __float2half_rn(z > 0.f ? o / z : 0.f);
    if (e == 0 && lse != nullptr) lse[row] = z > 0.f ? (m + log2f(z)) * kLn2 : -INFINITY;
}

template <int D, int R, int T>
int launch_cfg(const DecodeParams& prm, __half* out, float* lse, cudaStream_t stream) {
    const dim3 grid(prm.n_splits, prm.Hk, prm.B);
    constexpr int kRing = kStages * Stage<D, T>::kBytes;
    cudaError_t e = cudaFuncSetAttribute(decode_kernel<D, R, T>, cudaFuncAttributeMaxDynamicSharedMemorySize, kRing);
    if (e != cudaSuccess) return static_cast<int>(e);
    e = cudaMemsetAsync(prm.status, 0, 16, stream);
    if (e != cudaSuccess) return static_cast<int>(e);
    decode_kernel<D, R, T><<<grid, kThreads, kRing, stream>>>(prm);
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

struct DecodeGeometry {
    int n_blk, T_mask, W, n_splits;
    size_t o_bytes, mz_bytes;
};

int resolve_decode(const tilemix_decode_t* p, DecodeGeometry* g) {
    if (p == nullptr) return TILEMIX_ERR_NULL;
    if (p->batch <= 0 || p->heads_q <= 0 || p->heads_kv <= 0 || p->head_dim <= 0 || p->max_len <= 0 ||
        p->tile_n <= 0 || p->group <= 0 || p->n_splits < 0)
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
    int splits = p->n_splits;
    if (splits == 0) {
        // at most two full waves of two CTAs per SM over the whole batch (measured: more splits cost
        // more in per-CTA set-up and merge than they gain, and a third, partial wave idles a quarter
        // of the GPU), at least two key tiles per split
        const int64_t want = (148 * 2 * 2) / (static_cast<int64_t>(p->batch) * p->heads_kv);
        splits = static_cast<int>(want < 1 ? 1 : want);
        const int cap = g->n_blk / 2 > 0 ? g->n_blk / 2 : 1;
        if (splits > cap) splits = cap;
    }
    if (splits > g->n_blk) splits = g->n_blk;
    if (splits > 65535) return TILEMIX_ERR_UNSUPPORTED;
    g->n_splits = splits;
    const size_t rows = static_cast<size_t>(p->batch) * p->heads_q * splits;
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
    return kDecodeStatusBytes + g.o_bytes + 2 * g.mz_bytes;
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
    if (workspace_bytes < kDecodeStatusBytes + g.o_bytes + 2 * g.mz_bytes) return TILEMIX_ERR_WORKSPACE;
    DecodeParams prm{};
    prm.B = p->batch; prm.Hq = p->heads_q; prm.Hk = p->heads_kv; prm.max_len = p->max_len; prm.G = p->group;
    prm.nb = p->mask_batch; prm.W = g.W; prm.n_splits = g.n_splits; prm.n_blk = g.n_blk;
    const float scale = p->softmax_scale > 0.f ? p->softmax_scale : 1.0f / sqrtf(static_cast<float>(p->head_dim));
    prm.scale_log2 = scale * kLog2e;
    prm.q = static_cast<const __half*>(q_f16);
    prm.k16 = static_cast<const __half*>(k_f16);
    prm.k8 = k_i8; prm.k_scale = k_scale; prm.v8 = v_i8; prm.v_scale = v_scale;
    prm.words = mask_words; prm.cache_len = cache_len;
    prm.status = static_cast<int*>(workspace);
    uint8_t* ws = static_cast<uint8_t*>(workspace) + kDecodeStatusBytes;
    prm.o_part = reinterpret_cast<float*>(ws);
    prm.m_part = reinterpret_cast<float*>(ws + g.o_bytes);
    prm.z_part = reinterpret_cast<float*>(ws + g.o_bytes + g.mz_bytes);
    prm.q8_out = q_i8_out; prm.qs_out = q_scale_out;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int R = p->heads_q / p->heads_kv;
    __half* out = static_cast<__half*>(out_f16);
    if (p->head_dim == 128 && p->tile_n == 128) return launch_r<128, 128>(R, prm, out, lse, s);
    if (p->head_dim == 128 && p->tile_n == 64) return launch_r<128, 64>(R, prm, out, lse, s);
    if (p->head_dim == 64 && p->tile_n == 128) return launch_r<64, 128>(R, prm, out, lse, s);
    if (p->head_dim == 64 && p->tile_n == 64) return launch_r<64, 64>(R, prm, out, lse, s);
    return TILEMIX_ERR_UNSUPPORTED;
}

}  // extern "C"
