// Fused TileMix attention forward for sm_100a (Sec. 4.1 loops, Sec. 4.3 "Tile-group dispatch",
// Sec. 3.1 online softmax, App. C score formulas).
//
// One CTA owns two adjacent query tiles (A = 2p, B = 2p+1) of one (batch, query head) and
// streams the key/value tiles 0..B once for both.  Warp roles:
//   warps 0-3   softmax group A  (one thread per query row of tile A)
//   warps 4-7   softmax group B
//   warp  8     TMA producer     (one thread): Q16/Q8 once, then per key tile the K operand(s)
//                                the routing bits ask for (FP16 and/or INT8) and V, into a
//                                ring of equally sized shared-memory chunks
//   warp  9     MMA issuer       (one thread): tcgen05.mma kind::f16 or kind::i8 for S = Q K^T
//                                per the routing bit, then kind::f16 for O += P V with P read
//                                from tensor memory; also owns the TMEM allocation
// Tensor memory: S_A | S_B | O_A | O_B (FP32 / INT32 accumulators); the FP16 probabilities P
// overwrite the first half of their S columns.  The two groups alternate: while group A turns
// S_A into P_A on the ALUs, the tensor pipe runs PV_B and the next QK_B, and vice versa.
//
// Every wait is bounded: when one runs out the CTA records a status, raises an abort flag all
// roles poll, drains what is in flight and returns.
#include <cuda.h>
#include <cuda_fp16.h>

#include "common.cuh"
#include "ptx_sm100.cuh"

namespace tilemix {

namespace {

constexpr int kWarpsPerGroup = 4;
constexpr int kProducerWarp = 8;
constexpr int kMmaWarp = 9;
constexpr int kThreads = 320;
constexpr int kRing = 8;
constexpr int kMaxWords = 64;             // packed words per row kept in shared memory
constexpr uint64_t kTimeoutNs = 2000000000ull;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
// Lazy rescale: the running maximum only moves when a tile exceeds it by more than this many
// powers of two, so P stays <= 2^kTau (representable in FP16) and O is rarely rescaled.
constexpr float kTau = 8.0f;

enum Role : int { kRoleSoftmaxA = 0, kRoleSoftmaxB = 1, kRoleProducer = 2, kRoleMma = 3 };
enum Bar : int { kBarQ = 0, kBarRingFull = 1, kBarRingEmpty = 2, kBarS = 3, kBarP = 4, kBarO = 5, kBarDrain = 6 };

template <int D, int T>
struct Cfg {
    static constexpr int kM = 128;                    // rows of one MMA / TMEM tile
    static constexpr int kChunk = T * 128;            // ring chunk: T rows of 128 bytes
    static constexpr int kHalves = D / 64;            // 64-element column slabs of an FP16 tile
    static constexpr int kQ16Slab = kM * 128;
    static constexpr int kQ16Tile = kQ16Slab * kHalves;
    static constexpr int kQ8Tile = kM * D;
    static constexpr int kK8Bytes = T * D;
    static constexpr int kI8RowBytes = D;             // 128 -> 128B swizzle, 64 -> 64B swizzle
    static constexpr uint32_t kI8Layout = (D == 128) ? 2u : 4u;
    static constexpr uint32_t kI8Sbo = 8u * D;
    static constexpr int kSCols = T;
    static constexpr int kOCols = D;
    static constexpr int kTmemCols = 2 * (kSCols + kOCols);
    static constexpr int kOffQ16 = 0;
    static constexpr int kOffQ8 = 2 * kQ16Tile;
    static constexpr int kOffRing = kOffQ8 + 2 * kQ8Tile;
    static constexpr int kOffBars = kOffRing + kRing * kChunk;
    static constexpr int kNumBars = 2 + 2 * kRing + 2 + 2 + 2 + 1;
    static constexpr int kOffMisc = kOffBars + kNumBars * 8;       // tmem base, abort flag
    static constexpr int kOffWords = kOffMisc + 16;
    static constexpr int kSmemBytes = kOffWords + 2 * kMaxWords * 4;
    static constexpr int kSmemAlloc = kSmemBytes + 1024;           // slack to align the base
    static_assert(kK8Bytes <= kChunk, "INT8 key tile must fit one ring chunk");
    static_assert(kTmemCols == 256 || kTmemCols == 512, "TMEM allocation must be a power of two");
    static_assert(kSmemAlloc <= 232448, "exceeds the 227 KB shared memory of a CTA");
    static_assert(T % 32 == 0 && D % 64 == 0, "tile shape");
};

struct Params {
    int B, Hq, Hk, L, G, T_m, W, nb;
    int has_int8;                 // INT8 operands present
    float scale_log2;             // softmax scale * log2(e)
    const float* q_scale;         // [B,Hq,T_m]
    const float* k_scale;         // [B,Hk,T_n]
    const uint32_t* words;        // [nb,Hk,T_m,W] or null (all FP16)
    __half* out;
    int64_t os[3];
    float* lse;                   // nullable
    int* status;                  // 4 ints
    const int32_t* dbg_tiles;     // nullable
    int dbg_n;
    int32_t* dbg_raw;
    uint8_t* dbg_kind;
};

struct Ctx {
    volatile int* abort_flag;
    int* status;
};

__device__ __forceinline__ void record_timeout(const Ctx& cx, int role, int tile, int which) {
    *cx.abort_flag = 1;
    if (atomicCAS(&cx.status[0], 0, TILEMIX_ERR_DEVICE_TIMEOUT) == 0) {
        cx.status[1] = role;
        cx.status[2] = tile;
        cx.status[3] = which;
    }
}

// Bounded wait on one mbarrier phase.  Returns false when the CTA is aborting.
__device__ __forceinline__ bool wait_bar(const Ctx& cx, uint32_t bar, uint32_t parity, int role,
                                         int tile, int which) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = ptx::globaltimer_ns();
    uint32_t it = 0;
    while (!ptx::mbar_try_wait(bar, parity)) {
        if ((++it & 127u) == 0u) {
            if (*cx.abort_flag) return false;
            if (ptx::globaltimer_ns() - t0 > kTimeoutNs) {
                record_timeout(cx, role, tile, which);
                return false;
            }
        }
    }
    return true;
}

// Bookkeeping of the chunk ring; producer and MMA issuer run the same sequence of take() calls.
struct Ring {
    uint32_t slot = 0;
    uint32_t phases = 0;  // per-slot phase bit of the next use
    // n consecutive chunks that do not wrap around the end of the ring
    __device__ __forceinline__ uint32_t take(int n) {
        if (slot + n > kRing) slot = 0;
        const uint32_t s = slot;
        slot = (slot + n) % kRing;
        return s;
    }
    __device__ __forceinline__ uint32_t phase(uint32_t s) const { return (phases >> s) & 1u; }
    __device__ __forceinline__ void flip(uint32_t s) { phases ^= 1u << s; }
};

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ uint32_t route_bit(const uint32_t* row_words, int n, int G) {
    const int g = n / G;
    return (row_words[g >> 5] >> (g & 31)) & 1u;
}

template <int D, int T>
__global__ void __launch_bounds__(kThreads, 1)
attention_kernel(const Params prm, const __grid_constant__ CUtensorMap tm_q16,
                 const __grid_constant__ CUtensorMap tm_k16, const __grid_constant__ CUtensorMap tm_v16,
                 const __grid_constant__ CUtensorMap tm_q8, const __grid_constant__ CUtensorMap tm_k8) {
    using C = Cfg<D, T>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sbase = ptx::smem_u32(smem);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    // An earlier CTA of this launch already failed: do nothing (decided once per CTA).
    __shared__ int s_skip;
    if (threadIdx.x == 0) s_skip = *reinterpret_cast<volatile int*>(prm.status);
    __syncthreads();
    if (s_skip != 0) return;

    // ---- work item -------------------------------------------------------------------
    const int n_pairs = (prm.T_m + 1) >> 1;
    const int bh = blockIdx.x / n_pairs;
    const int pr = n_pairs - 1 - (blockIdx.x - bh * n_pairs);   // longest rows first
    const int b = bh / prm.Hq, hq = bh - b * prm.Hq;
    const int hk = hq / (prm.Hq / prm.Hk);
    const int mA = 2 * pr, mB = 2 * pr + 1;
    const bool hasB = mB < prm.T_m;
    const int nkv = (hasB ? mB : mA) + 1;

    // ---- shared memory ------------------------------------------------------------------
    const uint32_t bar0 = sbase + C::kOffBars;
    auto bar_q = [&](int t) { return bar0 + 8u * t; };
    auto bar_full = [&](int s) { return bar0 + 8u * (2 + s); };
    auto bar_empty = [&](int s) { return bar0 + 8u * (2 + kRing + s); };
    auto bar_s = [&](int t) { return bar0 + 8u * (2 + 2 * kRing + t); };
    auto bar_p = [&](int t) { return bar0 + 8u * (4 + 2 * kRing + t); };
    auto bar_o = [&](int t) { return bar0 + 8u * (6 + 2 * kRing + t); };
    const uint32_t bar_drain = bar0 + 8u * (8 + 2 * kRing);
    uint32_t* misc = reinterpret_cast<uint32_t*>(smem + C::kOffMisc);   // [0] tmem base, [1] abort
    uint32_t* words_s = reinterpret_cast<uint32_t*>(smem + C::kOffWords);
    Ctx cx{reinterpret_cast<volatile int*>(&misc[1]), prm.status};

    if (threadIdx.x == 0) {
        ptx::mbar_init(bar_q(0), 1);
        ptx::mbar_init(bar_q(1), 1);
        for (int s = 0; s < kRing; ++s) {
            ptx::mbar_init(bar_full(s), 1);
            ptx::mbar_init(bar_empty(s), 1);
        }
        for (int t = 0; t < 2; ++t) {
            ptx::mbar_init(bar_s(t), 1);
            ptx::mbar_init(bar_p(t), kWarpsPerGroup * 32);
            ptx::mbar_init(bar_o(t), 1);
        }
        ptx::mbar_init(bar_drain, 1);
        misc[1] = 0;
        ptx::fence_mbar_init();
    }
    // routing words of rows A and B (zeros = FP16 everywhere)
    for (int i = threadIdx.x; i < 2 * kMaxWords; i += kThreads) {
        const int t = i / kMaxWords, w = i - t * kMaxWords;
        const int m = t ? mB : mA;
        uint32_t v = 0u;
        if (prm.words != nullptr && w < prm.W && m < prm.T_m) {
            const int nbi = (prm.nb == 1) ? 0 : b;
            v = prm.words[((static_cast<int64_t>(nbi) * prm.Hk + hk) * prm.T_m + m) * prm.W + w];
        }
        words_s[i] = v;
    }
    if (warp == kMmaWarp) {
        ptx::tmem_alloc(ptx::smem_u32(&misc[0]), C::kTmemCols);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = misc[0];
    const uint32_t* wordsA = words_s;
    const uint32_t* wordsB = words_s + kMaxWords;

    // which K operands key tile j must bring: bit0 = FP16 copy, bit1 = INT8 copy
    auto k_needs = [&](int j) -> uint32_t {
        uint32_t need = 0u;
        if (j <= mA) need |= route_bit(wordsA, j, prm.G) ? 2u : 1u;
        if (hasB) need |= route_bit(wordsB, j, prm.G) ? 2u : 1u;
        return need;
    };

    if (warp == kProducerWarp) {
        // ================================================================ TMA producer
        if (lane == 0) {
            ptx::tma_prefetch_desc(&tm_q16);
            ptx::tma_prefetch_desc(&tm_k16);
            ptx::tma_prefetch_desc(&tm_v16);
            if (prm.has_int8) {
                ptx::tma_prefetch_desc(&tm_q8);
                ptx::tma_prefetch_desc(&tm_k8);
            }
            for (int t = 0; t < (hasB ? 2 : 1); ++t) {
                const int m = t ? mB : mA;
                const uint32_t bytes = C::kQ16Tile + (prm.has_int8 ? C::kQ8Tile : 0);
                ptx::mbar_arrive_expect_tx(bar_q(t), bytes);
                for (int c = 0; c < C::kHalves; ++c)
                    ptx::tma_load_4d(sbase + C::kOffQ16 + t * C::kQ16Tile + c * C::kQ16Slab, &tm_q16,
                                     bar_q(t), c * 64, m * T, hq, b);
                if (prm.has_int8)
                    ptx::tma_load_4d(sbase + C::kOffQ8 + t * C::kQ8Tile, &tm_q8, bar_q(t), 0, m * T, hq, b);
            }
            Ring ring;
            ring.phases = 0xffu;   // first wait on every "empty" barrier passes immediately
            uint32_t issued = 0u, full_phase = 0u, last_parity = 0u;   // per-slot bits
            bool ok = true;
            auto fill = [&](uint32_t s, const CUtensorMap* tm, uint32_t bytes, int c0, int row) {
                if (!ok) return;
                if (!wait_bar(cx, bar_empty(s), ring.phase(s), kRoleProducer, row / T, kBarRingEmpty)) {
                    ok = false;
                    return;
                }
                ring.flip(s);
                ptx::mbar_arrive_expect_tx(bar_full(s), bytes);
                ptx::tma_load_4d(sbase + C::kOffRing + s * C::kChunk, tm, bar_full(s), c0, row, hk, b);
                last_parity = (last_parity & ~(1u << s)) | (full_phase & (1u << s));
                full_phase ^= 1u << s;
                issued |= 1u << s;
            };
            for (int j = 0; j < nkv && ok; ++j) {
                const uint32_t need = k_needs(j);
                if (need & 1u) {
                    const uint32_t s = ring.take(C::kHalves);
                    for (int c = 0; c < C::kHalves; ++c) fill(s + c, &tm_k16, C::kChunk, c * 64, j * T);
                }
                if (need & 2u) fill(ring.take(1), &tm_k8, C::kK8Bytes, 0, j * T);
                const uint32_t s = ring.take(C::kHalves);
                for (int c = 0; c < C::kHalves; ++c) fill(s + c, &tm_v16, C::kChunk, c * 64, j * T);
            }
            if (!ok || *cx.abort_flag) {
                // let copies that are still in flight land before the CTA's memory is released
                for (uint32_t s = 0; s < kRing; ++s) {
                    if (!(issued >> s & 1u)) continue;
                    for (int it = 0; it < (1 << 20); ++it)
                        if (ptx::mbar_try_wait(bar_full(s), (last_parity >> s) & 1u)) break;
                }
            }
        }
    } else if (warp == kMmaWarp) {
        // ================================================================ MMA issuer
        if (lane == 0) {
            constexpr uint32_t kIdescQK16 = ptx::instr_desc(1, 0, 0, 0, C::kM, T);
            constexpr uint32_t kIdescQK8 = ptx::instr_desc(2, 1, 0, 0, C::kM, T);
            constexpr uint32_t kIdescPV = ptx::instr_desc(1, 0, 0, 1, C::kM, D);
            Ring ring;
            bool ok = true;
            auto acquire = [&](uint32_t s, int j) {   // wait until chunk s holds its data
                if (!ok) return;
                if (!wait_bar(cx, bar_full(s), ring.phase(s), kRoleMma, j, kBarRingFull)) ok = false;
                ring.flip(s);
            };
            // S_t = Q_t K_j^T on the route of tile t
            auto issue_qk = [&](int t, uint32_t int8_route, uint32_t s16, uint32_t s8) {
                const uint32_t d_tmem = tmem_base + t * C::kSCols;
                if (int8_route) {
                    const uint32_t a0 = sbase + C::kOffQ8 + t * C::kQ8Tile;
                    const uint32_t b0 = sbase + C::kOffRing + s8 * C::kChunk;
#pragma unroll
                    for (int k = 0; k < D / 32; ++k)
                        ptx::mma_i8_ss(d_tmem, ptx::smem_desc(a0 + k * 32, 16, C::kI8Sbo, C::kI8Layout),
                                       ptx::smem_desc(b0 + k * 32, 16, C::kI8Sbo, C::kI8Layout), kIdescQK8,
                                       k > 0);
                } else {
#pragma unroll
                    for (int c = 0; c < C::kHalves; ++c) {
                        const uint32_t a0 = sbase + C::kOffQ16 + t * C::kQ16Tile + c * C::kQ16Slab;
                        const uint32_t b0 = sbase + C::kOffRing + (s16 + c) * C::kChunk;
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            ptx::mma_f16_ss(d_tmem, ptx::smem_desc(a0 + k * 32, 16, 1024, 2),
                                            ptx::smem_desc(b0 + k * 32, 16, 1024, 2), kIdescQK16,
                                            (c | k) > 0);
                    }
                }
            };
            // O_t (+)= P_t V_j with P in tensor memory (two FP16 per 32-bit column)
            auto issue_pv = [&](int t, uint32_t sv, uint32_t accumulate) {
                const uint32_t d_tmem = tmem_base + 2 * C::kSCols + t * C::kOCols;
                const uint32_t a_tmem = tmem_base + t * C::kSCols;
                const uint32_t b0 = sbase + C::kOffRing + sv * C::kChunk;
#pragma unroll
                for (int k = 0; k < T / 16; ++k)
                    ptx::mma_f16_ts(d_tmem, a_tmem + k * 8, ptx::smem_desc(b0 + k * 2048, C::kChunk, 1024, 2),
                                    kIdescPV, accumulate | (k > 0));
            };

            for (int t = 0; t < (hasB ? 2 : 1) && ok; ++t)
                if (!wait_bar(cx, bar_q(t), 0, kRoleMma, t, kBarQ)) ok = false;

            // slots of the K operands of the tile whose QK^T is issued next
            uint32_t need = k_needs(0), k16 = 0, k8 = 0;
            if (need & 1u) { k16 = ring.take(C::kHalves); for (int c = 0; c < C::kHalves; ++c) acquire(k16 + c, 0); }
            if (need & 2u) { k8 = ring.take(1); acquire(k8, 0); }
            if (ok) {
                ptx::tc_fence_after_sync();
                issue_qk(0, route_bit(wordsA, 0, prm.G), k16, k8);
                ptx::mma_commit(bar_s(0));
                if (hasB) {
                    issue_qk(1, route_bit(wordsB, 0, prm.G), k16, k8);
                    ptx::mma_commit(bar_s(1));
                }
                if (need & 1u) for (int c = 0; c < C::kHalves; ++c) ptx::mma_commit(bar_empty(k16 + c));
                if (need & 2u) ptx::mma_commit(bar_empty(k8));
            }
            for (int j = 0; j < nkv && ok; ++j) {
                const uint32_t sv = ring.take(C::kHalves);
                const bool more = j + 1 < nkv;
                need = more ? k_needs(j + 1) : 0u;
                if (need & 1u) k16 = ring.take(C::kHalves);
                if (need & 2u) k8 = ring.take(1);
                bool v_ready = false, k_ready = false;
                for (int t = 0; t < 2 && ok; ++t) {
                    const int m_t = t ? mB : mA;
                    if ((t == 1 && !hasB) || j > m_t) continue;
                    if (!wait_bar(cx, bar_p(t), j & 1, kRoleMma, j, kBarP)) { ok = false; break; }
                    if (!v_ready) { for (int c = 0; c < C::kHalves; ++c) acquire(sv + c, j); v_ready = true; }
                    if (!ok) break;
                    ptx::tc_fence_after_sync();
                    issue_pv(t, sv, j > 0);
                    if (j == m_t) ptx::mma_commit(bar_o(t));
                    if (j + 1 <= m_t) {
                        if (!k_ready) {
                            if (need & 1u) for (int c = 0; c < C::kHalves; ++c) acquire(k16 + c, j + 1);
                            if (need & 2u) acquire(k8, j + 1);
                            k_ready = true;
                            if (!ok) break;
                            ptx::tc_fence_after_sync();
                        }
                        issue_qk(t, route_bit(t ? wordsB : wordsA, j + 1, prm.G), k16, k8);
                        ptx::mma_commit(bar_s(t));
                    }
                }
                if (!ok) break;
                for (int c = 0; c < C::kHalves; ++c) ptx::mma_commit(bar_empty(sv + c));
                if (need & 1u) for (int c = 0; c < C::kHalves; ++c) ptx::mma_commit(bar_empty(k16 + c));
                if (need & 2u) ptx::mma_commit(bar_empty(k8));
            }
            // every MMA issued by this thread has retired before TMEM / shared memory go away
            ptx::mma_commit(bar_drain);
            wait_bar(cx, bar_drain, 0, kRoleMma, nkv, kBarDrain);
        }
    } else {
        // ================================================================ softmax groups
        const int t = warp / kWarpsPerGroup;
        const int m_t = t ? mB : mA;
        if (t == 0 || hasB) {
            const int quarter = warp & 3;
            const int row = quarter * 32 + lane;
            const uint32_t lane_base = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
            const uint32_t t_s = lane_base + t * C::kSCols;
            const uint32_t t_o = lane_base + 2 * C::kSCols + t * C::kOCols;
            const uint32_t* words_t = t ? wordsB : wordsA;
            const int64_t i_glob = static_cast<int64_t>(m_t) * T + row;
            const bool row_valid = row < T && i_glob < prm.L;
            const float dq = prm.has_int8 ? prm.q_scale[(static_cast<int64_t>(b) * prm.Hq + hq) * prm.T_m + m_t] : 0.f;
            const float* dk_row = prm.has_int8 ? prm.k_scale + (static_cast<int64_t>(b) * prm.Hk + hk) * prm.T_m : nullptr;
            float m_run = -INFINITY, z = 0.f;
            bool ok = true;
            const int role = t ? kRoleSoftmaxB : kRoleSoftmaxA;

            for (int j = 0; j <= m_t; ++j) {
                const uint32_t int8_route = route_bit(words_t, j, prm.G);
                float a = prm.scale_log2;
                if (int8_route) {
                    a *= dq * dk_row[j];
                    if (a == 0.f) a = 1.f;   // a zero block: every accumulator is 0 already
                }
                ok = wait_bar(cx, bar_s(t), j & 1, role, j, kBarS);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                ptx::tc_fence_after_sync();

                uint32_t s[T];
#pragma unroll
                for (int c = 0; c < T / 32; ++c)
                    ptx::tmem_ld32(t_s + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&s[c * 32]));
                ptx::tmem_wait_ld();

                if (prm.dbg_n > 0) {   // debug mode: raw accumulators of the requested tiles
                    int idx = -1;
                    if (lane == 0) {
                        for (int e = 0; e < prm.dbg_n; ++e) {
                            const int32_t* q = prm.dbg_tiles + 4 * e;
                            if (q[0] == b && q[1] == hq && q[2] == m_t && q[3] == j) { idx = e; break; }
                        }
                    }
                    idx = __shfl_sync(0xffffffffu, idx, 0);
                    if (idx >= 0 && row < T) {
                        int32_t* dst = prm.dbg_raw + (static_cast<int64_t>(idx) * T + row) * T;
#pragma unroll
                        for (int c = 0; c < T; c += 4)
                            *reinterpret_cast<uint4*>(dst + c) = make_uint4(s[c], s[c + 1], s[c + 2], s[c + 3]);
                        if (row == 0) prm.dbg_kind[idx] = static_cast<uint8_t>(int8_route);
                    }
                }

                // common score domain: FP32 raw accumulators (App. C), then causal legality
                float mx = -INFINITY;
                const bool diag = (j == m_t);
#pragma unroll
                for (int c = 0; c < T; ++c) {
                    float v = int8_route ? __int2float_rn(static_cast<int>(s[c])) : __uint_as_float(s[c]);
                    if (diag && c > row) v = -INFINITY;
                    s[c] = __float_as_uint(v);
                    mx = fmaxf(mx, v);
                }
                // shared online-softmax state (Sec. 3.1) in the log2 domain
                const float m_tile = mx * a;
                const bool grow = m_tile > m_run + kTau;
                float alpha = 1.f;
                if (grow) {
                    alpha = fast_exp2(m_run - m_tile);
                    m_run = m_tile;
                }
                float sum = 0.f;
                // P = 2^(a*raw - m), rounded to FP16 and packed two per word into s[0 .. T/2)
#pragma unroll
                for (int c = 0; c < T; c += 2) {
                    const float p0 = fast_exp2(fmaf(__uint_as_float(s[c]), a, -m_run));
                    const float p1 = fast_exp2(fmaf(__uint_as_float(s[c + 1]), a, -m_run));
                    sum += p0 + p1;
                    const __half2 h = __floats2half2_rn(p0, p1);
                    s[c >> 1] = *reinterpret_cast<const uint32_t*>(&h);
                }
                z = z * alpha + sum;

                if (j > 0 && __any_sync(0xffffffffu, grow)) {
                    // O~ *= alpha.  PV of tile j-1 has retired: it was issued before the QK^T
                    // whose completion this group has just observed.
#pragma unroll
                    for (int c = 0; c < D / 32; ++c) {
                        uint32_t o[32];
                        ptx::tmem_ld32(t_o + c * 32, o);
                        ptx::tmem_wait_ld();
#pragma unroll
                        for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
                        ptx::tmem_st32(t_o + c * 32, o);
                    }
                }
#pragma unroll
                for (int c = 0; c < T / 64; ++c)
                    ptx::tmem_st32(t_s + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&s[c * 32]));
                ptx::tmem_wait_st();
                ptx::tc_fence_before_sync();
                ptx::mbar_arrive(bar_p(t));
            }

            if (ok) {
                ok = wait_bar(cx, bar_o(t), 0, role, m_t + 1, kBarO);
                ok = __all_sync(0xffffffffu, ok);
            }
            if (ok) {
                ptx::tc_fence_after_sync();
                const float inv = 1.f / z;
                __half* dst = prm.out + b * prm.os[0] + hq * prm.os[1] + i_glob * prm.os[2];
#pragma unroll
                for (int c = 0; c < D / 32; ++c) {
                    uint32_t o[32];
                    ptx::tmem_ld32(t_o + c * 32, o);
                    ptx::tmem_wait_ld();
                    if (row_valid) {
#pragma unroll
                        for (int e = 0; e < 32; e += 8) {
                            uint32_t h[4];
#pragma unroll
                            for (int u = 0; u < 4; ++u) {
                                const __half2 hv = __floats2half2_rn(__uint_as_float(o[e + 2 * u]) * inv,
                                                                     __uint_as_float(o[e + 2 * u + 1]) * inv);
                                h[u] = *reinterpret_cast<const uint32_t*>(&hv);
                            }
                            *reinterpret_cast<uint4*>(dst + c * 32 + e) = make_uint4(h[0], h[1], h[2], h[3]);
                        }
                    }
                }
                if (row_valid && prm.lse != nullptr)
                    prm.lse[(static_cast<int64_t>(b) * prm.Hq + hq) * prm.L + i_glob] = (m_run + log2f(z)) * kLn2;
            }
        }
    }

    // ---- teardown -----------------------------------------------------------------------
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == kMmaWarp) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, C::kTmemCols);
    }
}

// ---------------------------------------------------------------------------------- host
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

int get_encoder(EncodeTiledFn* fn) {
    void* sym = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres);
    if (e != cudaSuccess) return static_cast<int>(e);
    if (qres != cudaDriverEntryPointSuccess || sym == nullptr) return static_cast<int>(cudaErrorNotSupported);
    *fn = reinterpret_cast<EncodeTiledFn>(sym);
    return 0;
}

// 4-D map over [B, H, L, d] (innermost first: d, L, H, B); box = box_d x box_rows x 1 x 1.
int encode_map(EncodeTiledFn enc, CUtensorMap* tm, const void* base, int elem_bytes, int d, int L, int H,
               int B, const int64_t stride_elems[3], int box_d, int box_rows, CUtensorMapSwizzle swz) {
    const cuuint64_t dims[4] = {static_cast<cuuint64_t>(d), static_cast<cuuint64_t>(L),
                                static_cast<cuuint64_t>(H), static_cast<cuuint64_t>(B)};
    const cuuint64_t strides[3] = {static_cast<cuuint64_t>(stride_elems[2]) * elem_bytes,
                                   static_cast<cuuint64_t>(stride_elems[1]) * elem_bytes,
                                   static_cast<cuuint64_t>(stride_elems[0]) * elem_bytes};
    const cuuint32_t box[4] = {static_cast<cuuint32_t>(box_d), static_cast<cuuint32_t>(box_rows), 1u, 1u};
    const cuuint32_t estr[4] = {1u, 1u, 1u, 1u};
    const CUresult r = enc(tm, elem_bytes == 2 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_UINT8,
                           4, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                           swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return static_cast<int>(r);
}

template <int D, int T>
int launch_impl(const Geometry& g, const void* q, const void* k, const void* v, const int8_t* q8,
                const int8_t* k8, const float* qs, const float* ks, const uint32_t* words, void* out,
                float* lse, void* workspace, const tilemix_debug_t* dbg, cudaStream_t stream) {
    using C = Cfg<D, T>;
    EncodeTiledFn enc = nullptr;
    int rc = get_encoder(&enc);
    if (rc) return rc;
    const bool has8 = !(g.flags & TILEMIX_FORCE_FP16) && q8 != nullptr;
    CUtensorMap tq, tk, tv, tq8, tk8;
    if ((rc = encode_map(enc, &tq, q, 2, g.d, g.L, g.Hq, g.B, g.qs, 64, C::kM, CU_TENSOR_MAP_SWIZZLE_128B))) return rc;
    if ((rc = encode_map(enc, &tk, k, 2, g.d, g.L, g.Hk, g.B, g.ks, 64, T, CU_TENSOR_MAP_SWIZZLE_128B))) return rc;
    if ((rc = encode_map(enc, &tv, v, 2, g.d, g.L, g.Hk, g.B, g.vs, 64, T, CU_TENSOR_MAP_SWIZZLE_128B))) return rc;
    if (has8) {
        const CUtensorMapSwizzle sw8 = (D == 128) ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B;
        const int64_t dq[3] = {static_cast<int64_t>(g.Hq) * g.L * g.d, static_cast<int64_t>(g.L) * g.d, g.d};
        const int64_t dk[3] = {static_cast<int64_t>(g.Hk) * g.L * g.d, static_cast<int64_t>(g.L) * g.d, g.d};
        if ((rc = encode_map(enc, &tq8, q8, 1, g.d, g.L, g.Hq, g.B, dq, D, C::kM, sw8))) return rc;
        if ((rc = encode_map(enc, &tk8, k8, 1, g.d, g.L, g.Hk, g.B, dk, D, T, sw8))) return rc;
    } else {
        tq8 = tq;
        tk8 = tk;
    }
    Params prm{};
    prm.B = g.B; prm.Hq = g.Hq; prm.Hk = g.Hk; prm.L = g.L; prm.G = g.G; prm.T_m = g.T_m; prm.W = g.W;
    prm.nb = g.nb;
    prm.has_int8 = has8 ? 1 : 0;
    prm.scale_log2 = g.scale * kLog2e;
    prm.q_scale = qs; prm.k_scale = ks;
    prm.words = has8 ? words : nullptr;
    prm.out = static_cast<__half*>(out);
    prm.os[0] = g.os[0]; prm.os[1] = g.os[1]; prm.os[2] = g.os[2];
    prm.lse = lse;
    prm.status = static_cast<int*>(workspace);
    if (dbg != nullptr && dbg->n_tiles > 0) {
        prm.dbg_tiles = dbg->tiles; prm.dbg_n = dbg->n_tiles; prm.dbg_raw = dbg->raw; prm.dbg_kind = dbg->kind;
    }
    cudaError_t e = cudaMemsetAsync(workspace, 0, 16, stream);
    if (e != cudaSuccess) return static_cast<int>(e);
    e = cudaFuncSetAttribute(attention_kernel<D, T>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemAlloc);
    if (e != cudaSuccess) return static_cast<int>(e);
    const int64_t ctas = static_cast<int64_t>(g.B) * g.Hq * ((g.T_m + 1) / 2);
    if (ctas > 0x7fffffffLL) return static_cast<int>(cudaErrorInvalidConfiguration);
    attention_kernel<D, T><<<static_cast<unsigned>(ctas), kThreads, C::kSmemAlloc, stream>>>(prm, tq, tk, tv, tq8, tk8);
    g_launch_count.fetch_add(1);
    return static_cast<int>(cudaGetLastError());
}

}  // namespace

int launch_attention(const Geometry& g, const void* q, const void* k, const void* v, const int8_t* q8,
                     const int8_t* k8, const float* qs, const float* ks, const uint32_t* words, void* out,
                     float* lse, void* workspace, const tilemix_debug_t* dbg, cudaStream_t stream) {
    if (g.d == 128 && g.tile_m == 128)
        return launch_impl<128, 128>(g, q, k, v, q8, k8, qs, ks, words, out, lse, workspace, dbg, stream);
    if (g.d == 64 && g.tile_m == 64)
        return launch_impl<64, 64>(g, q, k, v, q8, k8, qs, ks, words, out, lse, workspace, dbg, stream);
    return TILEMIX_ERR_UNSUPPORTED;
}

}  // namespace tilemix
