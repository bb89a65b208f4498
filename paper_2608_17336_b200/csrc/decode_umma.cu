// Decode step over an INT8 key/value cache (App. C, "Additional Execution Interfaces"), tcgen05 form for head
// dimension 128 and 128-key tiles.  HBM-bound by design: a cached token costs d bytes of K8 (2d of FP16 K on the
// FP16 route) plus d bytes of V8, each read once.  The warp-level form (decode.cu) spends ~3300 warp instructions
// per key tile, most of them on feeding mma.sync fragments; here the two products are single-thread tcgen05
// instructions and the only per-element work left is what the method asks for -- V8 -> FP16 on chip:
//
//   S^T[128 keys x 16] = K_tile Q^T     A = the key tile as it lands in shared memory (K-major, 128-byte swizzle:
//                                       INT8 rows of 128 bytes, or two 64-column slabs of FP16 rows), B = the R
//                                       query rows of this KV head (INT8 copy quantised here, or FP16).  Keys are the
//                                       M rows, so every softmax thread owns one key (one TMEM lane) and R scores;
//                                       kind::i8 or kind::f16 by the tile's routing bit.
//   P[R x 128 keys]                     2^(s - m) * delta_V rounded to FP16, written by the key's thread into a
//                                       K-major operand tile; the row maximum m is shared by a stream's four warps
//                                       and lazy: it moves only when a step's maximum exceeds it by 2^8.
//   V16[64 keys x 128] = FP16(V8)       two groups of eight warps convert the INT8 rows exactly (1024 + (x + 128) as
//                                       FP16 bits, minus 1152), half a tile each, into the MN-major swizzled layout.
//   O[64 x 128] (+)= P V16              kind::f16, accumulator in tensor memory; rows 0..R-1 are the output.
//
// Warps: 0-7 softmax (two independent streams of four warps, see below), 8-23 conversion, 24 copy producer, 25 QK^T
// issuer, 26 PV issuer.  K8 / FP16 K slabs / V8 travel through a ring of eleven 16 KB units (an INT8-routed tile
// takes two, an FP16-routed tile three); what bounds the step is the data in flight -- the loaded HBM latency is
// several microseconds, so a CTA per SM keeps ~170 KB on the way -- and the fixed cost of each role's waits, which is
// why every role is either duplicated (softmax streams, conversion groups) or split in two (the issuers).
// Every wait is bounded; a CTA that gives up records a status, drains what is in flight and returns.
#include <cuda.h>
#include <cuda_fp16.h>
#include <math.h>

#include "common.cuh"
#include "decode.cuh"
#include "ptx_sm100.cuh"

namespace tilemix {
namespace {

constexpr int D = 128, T = 128;
constexpr int kUnit = T * D;              // bytes of a ring unit
constexpr int kUnits = 11;
constexpr int kSlots = 8;                 // barrier slots of tiles in the ring (at most kUnits / 2 tiles fit)
constexpr int kVHalf = (T / 2) * D * 2;   // FP16 copy of half a V tile (64 keys): two 64-column slabs of 8 KB
constexpr int kPRows = 64;                // M of the PV product
constexpr int kPTile = 2048;              // P of a key tile: rows 0..7 of two 64-key slabs (1 KB each)
constexpr int kMetaTiles = 256;
// Operand tiles of which only the first eight rows mean anything (P: M = 64 rows, Q: N = 16 rows) are stored as
// their first 8-row group only.  The tensor pipe reads the other row groups from whatever follows in shared memory
// (they produce rows of O / columns of S^T that nobody reads), so these tiles sit BELOW the ring: everything the
// descriptors can reach (8 KB + 1 KB past a P tile) is inside this CTA's shared memory.
constexpr int kOffP = 0;                         // 2 pair buffers x 2 tiles
constexpr int kOffQ8 = kOffP + 4 * kPTile;       // 8 rows x 128 bytes
constexpr int kOffQ16 = kOffQ8 + 1024;           // two slabs of 8 rows x 128 bytes
constexpr int kOffRing = kOffQ16 + 2048 + 1024;
constexpr int kOffV16 = kOffRing + kUnits * kUnit;
constexpr int kOffMeta = kOffV16 + 2 * kVHalf;
constexpr int kOffSmall = kOffMeta + kMetaTiles * 8;
static_assert(kOffRing % 1024 == 0 && kOffV16 % 1024 == 0, "swizzled tiles start on 1 KB boundaries");

// Two independent softmax streams of four warps each: stream g takes the steps (pairs of key tiles) j = g, g + 2, ...
// with its own running maximum, row sums and O accumulator, and ends as its own partial result -- to the merge
// kernel a CTA is two splits.  A stream's step is a chain of waits and short dependent instruction runs
// (~2600 clk); two of them in flight hide that latency.
constexpr int kStreams = 2, kStreamWarps = 4, kSoftmaxWarps = kStreams * kStreamWarps, kConvWarps = 16;
constexpr int kConvWarp0 = kSoftmaxWarps, kProducerWarp = kConvWarp0 + kConvWarps;
constexpr int kQkWarp = kProducerWarp + 1, kPvWarp = kQkWarp + 1;
constexpr int kThreads = (kPvWarp + 1) * 32;
constexpr int kConvThreads = kConvWarps * 32;
constexpr int kTmemCols = 512;            // S^T: four buffers of 16 columns from column 0; O of stream g: 128 + 128 g
constexpr uint32_t kColO = 128;
constexpr float kMoveAbove = 8.f;         // m moves when a step's maximum exceeds it by more than 2^8
constexpr int kRowsPerLane = 5, kMaxRows = 32 * kRowsPerLane;   // rows of a batch whose splits one warp can balance

struct Small {
    uint64_t full[kSlots], freeb[kSlots];
    uint64_t s_ready[2], s_free[2], p_ready[2], xchg[2];      // per pair buffer
    uint64_t v_ready[2], pv_done[2];                          // per V16 buffer (half of a tile)
    uint64_t pv_pair[2];                                      // per pair buffer: the PVs of a step have retired
    uint64_t zbar[kStreams], drain_qk, drain_pv;
    uint32_t slot_info[kSlots];           // ring units of the tile in a slot: K (byte 0), second K slab (1), V (2)
    float warp_max[kStreams][kStreamWarps][8];
    float zsum[kStreams][kStreamWarps][8];
    float dq[8];
    uint32_t tmem_base;
    int abort_flag;
    int row_cost[kMaxRows];               // balanced splits: cost of every (sequence, KV head) row of the batch
    int asg[4];                           // ... and this CTA's row, split and the row's number of splits
};
constexpr int kSmemBytes = kOffSmall + static_cast<int>(sizeof(Small)) + 1024;   // + slack to align the base to 1 KB
static_assert(kSmemBytes <= 227 * 1024, "shared memory of one CTA");

enum Which : int { kWFull = 1, kWFree = 2, kWS = 3, kWSFree = 4, kWP = 5, kWV = 6, kWPV = 7, kWXchg = 8, kWDrain = 9 };

template <int R, bool F16K>
__global__ void __launch_bounds__(kThreads, 1)
decode_umma_kernel(const __grid_constant__ CUtensorMap tm_k8, const __grid_constant__ CUtensorMap tm_k16,
                   const DecodeParams prm) {
    constexpr int RC = R <= 4 ? 4 : 8;    // score columns a softmax thread loads per key
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_u32 = ptx::smem_u32(smem_raw);
    const uint32_t sbase = (raw_u32 + 1023u) & ~1023u;
    uint8_t* sm = smem_raw + (sbase - raw_u32);
    Small& sh = *reinterpret_cast<Small*>(sm + kOffSmall);
    float2* meta = reinterpret_cast<float2*>(sm + kOffMeta);   // x = delta_K (negative: FP16 route), y = delta_V

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // Cost of the first nb groups of one 32-group mask word: a routing group costs 2 units per tile on the INT8
    // route (K8 + V8) and 3 on the FP16 route.  `row_words`: the mask words of a (sequence, KV head) row, or null.
    auto row_words = [&](int bb, int hh) -> const uint32_t* {
        return prm.words != nullptr ? prm.words + (static_cast<int64_t>(prm.nb == 1 ? 0 : bb) * prm.Hk + hh) * prm.W : nullptr;
    };
    auto row_groups = [&](int bb) -> int {
        const int l = min(max(prm.cache_len_raw[bb], 0), prm.max_len);
        return ((l + T - 1) / T + prm.G - 1) / prm.G;
    };
    auto word_cost = [&](const uint32_t* wr, int w, int nb) -> int {
        const uint32_t bits = wr != nullptr ? wr[w] & (nb >= 32 ? 0xffffffffu : ((1u << nb) - 1u)) : 0u;
        return 3 * nb - __popc(bits);
    };
    // Balanced splits (one wave of CTAs over a batch of at most kMaxRows rows): thread i adds up the cost of row i.
    if (prm.balanced && tid < prm.n_rows) {
        const int bb = tid / prm.Hk;
        const uint32_t* wr = row_words(bb, tid - bb * prm.Hk);
        const int ng = row_groups(bb);
        int c = 0;
        for (int w = 0; 32 * w < ng; ++w) c += word_cost(wr, w, min(32, ng - 32 * w));
        sh.row_cost[tid] = c;
    }
    // ---- set-up that needs nothing from the kernel before this one: barriers, tensor memory -----------------
    if (tid == 0) {
        for (int s = 0; s < kSlots; ++s) {
            ptx::mbar_init(ptx::smem_u32(&sh.full[s]), 1);
            ptx::mbar_init(ptx::smem_u32(&sh.freeb[s]), 1 + kConvWarps);
        }
        for (int i = 0; i < 2; ++i) {
            ptx::mbar_init(ptx::smem_u32(&sh.s_ready[i]), 1);
            ptx::mbar_init(ptx::smem_u32(&sh.s_free[i]), kStreamWarps * 32);
            ptx::mbar_init(ptx::smem_u32(&sh.p_ready[i]), kStreamWarps * 32);
            ptx::mbar_init(ptx::smem_u32(&sh.xchg[i]), kStreamWarps);
            ptx::mbar_init(ptx::smem_u32(&sh.zbar[i]), kStreamWarps);
            ptx::mbar_init(ptx::smem_u32(&sh.v_ready[i]), kConvWarps / 2);
            ptx::mbar_init(ptx::smem_u32(&sh.pv_done[i]), 1);
            ptx::mbar_init(ptx::smem_u32(&sh.pv_pair[i]), 1);
        }
        ptx::mbar_init(ptx::smem_u32(&sh.drain_qk), 1);
        ptx::mbar_init(ptx::smem_u32(&sh.drain_pv), 1);
        sh.abort_flag = 0;
        ptx::fence_mbar_init();
    }
    if (warp == kProducerWarp) {
        ptx::tmem_alloc(ptx::smem_u32(&sh.tmem_base), kTmemCols);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();                      // barriers initialised, tensor memory allocated, row costs written
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(&sh.tmem_base);
    auto leave = [&]() {                  // early exits: tensor memory goes back first
        __syncthreads();
        if (warp == kProducerWarp) ptx::tmem_dealloc(tmem_base, kTmemCols);
    };
    // ---- which part of which row -------------------------------------------------------------------------------
    // Uniform form: the grid is (splits, KV heads, sequences).  Balanced form: gridDim.x CTAs, one per SM, are
    // shared out over the rows so that the largest cost of a CTA is as small as it can be -- with one wave the
    // CTA with the most bytes ends last, and rows differ (cache lengths, FP16-routed groups).  Row i gets
    // s_i = clamp(ceil(c_i / tau), 1, cap) CTAs for the smallest tau whose total fits the grid; CTAs left over
    // leave.  Every CTA finds the same tau (one warp, a binary search over at most 15 steps).
    int split = blockIdx.x, hk = blockIdx.y, b = blockIdx.z, row_splits = prm.n_splits;
    if (prm.balanced) {
        if (warp == 0) {
            int c[kRowsPerLane], cmax = 0;
#pragma unroll
            for (int k = 0; k < kRowsPerLane; ++k) {
                const int i = kRowsPerLane * lane + k;
                c[k] = i < prm.n_rows ? sh.row_cost[i] : -1;    // -1: no such row
                cmax = max(cmax, c[k]);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) cmax = max(cmax, __shfl_xor_sync(0xffffffffu, cmax, o));
            auto share = [&](int cost, int tau) -> int {        // clamp(ceil(cost / tau), 1, cap), exact
                const int num = cost + tau - 1;
                int q = static_cast<int>(__fdividef(static_cast<float>(num), static_cast<float>(tau)));
                if (q * tau > num) --q;
                else if ((q + 1) * tau <= num) ++q;
                return min(max(q, 1), prm.split_cap);
            };
            auto count = [&](int tau) -> int {
                int n = 0;
#pragma unroll
                for (int k = 0; k < kRowsPerLane; ++k) n += c[k] >= 0 ? share(c[k], tau) : 0;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) n += __shfl_xor_sync(0xffffffffu, n, o);
                return n;
            };
            int lo = 1, hi = max(cmax, 1);                      // count(hi) = number of rows <= gridDim.x
            while (lo < hi) {
                const int mid = (lo + hi) >> 1;
                if (count(mid) <= static_cast<int>(gridDim.x)) hi = mid; else lo = mid + 1;
            }
            int s_k[kRowsPerLane], mine = 0;
#pragma unroll
            for (int k = 0; k < kRowsPerLane; ++k) { s_k[k] = c[k] >= 0 ? share(c[k], hi) : 0; mine += s_k[k]; }
            int start = mine;                                   // inclusive scan over the lanes
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int v = __shfl_up_sync(0xffffffffu, start, o);
                if (lane >= o) start += v;
            }
            start -= mine;                                      // first CTA of this lane's rows
            if (lane == 0) sh.asg[0] = -1;
            __syncwarp();
#pragma unroll
            for (int k = 0; k < kRowsPerLane; ++k) {
                const int cta = static_cast<int>(blockIdx.x) - start;
                if (cta >= 0 && cta < s_k[k]) { sh.asg[0] = kRowsPerLane * lane + k; sh.asg[1] = cta; sh.asg[2] = s_k[k]; }
                start += s_k[k];
            }
        }
        __syncthreads();
        const int row = sh.asg[0];
        if (row < 0) { leave(); return; }                       // a CTA left over
        split = sh.asg[1]; row_splits = sh.asg[2];
        b = row / prm.Hk; hk = row - b * prm.Hk;
    }
    // This grid may run beside the prepare kernel (programmatic dependent launch): it takes the length from the
    // caller's array with the same clamp, and waits for the prepare kernel (which clears the status record) only
    // where it is about to write that record.
    const int len = min(max(prm.cache_len_raw[b], 0), prm.max_len);
    const int n_tiles = (len + T - 1) / T;
    const uint32_t* wrow = row_words(b, hk);
    // The splits of a row share its BYTES, not its tiles.  Split k of n takes the groups [bound(k C / n),
    // bound((k + 1) C / n)), C the cost of the row and bound(x) the first group at which the running cost reaches
    // x; every thread computes the two bounds it needs (a scan over at most W mask words).
    const int n_groups = (n_tiles + prm.G - 1) / prm.G;
    auto word_bits = [&](int w) -> int { return min(32, n_groups - 32 * w); };                  // groups of word w that exist
    int total = 0;
    for (int w = 0; 32 * w < n_groups; ++w) total += word_cost(wrow, w, word_bits(w));
    auto bound = [&](long long x) -> int {
        if (x <= 0) return 0;
        int acc = 0, w = 0;
        for (; 32 * w < n_groups; ++w) {
            const int c = word_cost(wrow, w, word_bits(w));
            if (acc + c >= x) break;
            acc += c;
        }
        if (32 * w >= n_groups) return n_groups;
        const int nb = word_bits(w);
        int i = 1;
        while (i < nb && acc + word_cost(wrow, w, i) < x) ++i;    // smallest i with the cost of i groups of this word >= x - acc
        return 32 * w + i;
    };
    const int g0 = bound(static_cast<long long>(split) * total / row_splits);
    const int g1 = split + 1 == row_splits ? n_groups : bound(static_cast<long long>(split + 1) * total / row_splits);
    const int t0 = min(n_tiles, g0 * prm.G), t1 = min(n_tiles, g1 * prm.G);
    const int n_it = t1 - t0;
    const int n_pairs = (n_it + 1) / 2;   // the softmax warps take two key tiles per step
    const int n_parts = prm.n_parts;      // partial results per query head in the workspace (two per split, at least)
    const int64_t out_row0 = (static_cast<int64_t>(b) * prm.Hq + hk * R) * n_parts + kStreams * split;   // + r * n_parts + stream

    // Query row r of this KV head: FP16 copy and blockwise INT8 (block = the row), both as K-major operand rows in
    // shared memory (to_smem), and -- from the one split of the row that starts at its first group -- the quantised
    // row and its scale to the caller's buffers.
    const bool q_writer = g0 == 0 && (g1 > 0 || split + 1 == row_splits);
    // parts of the row that no split writes (balanced form: the row has fewer splits than the workspace has room
    // for): marked empty for the merge by the row's first split
    if (split == 0)
        for (int idx = tid; idx < R * (n_parts - kStreams * row_splits); idx += kThreads) {
            const int r = idx / (n_parts - kStreams * row_splits), part = kStreams * row_splits + idx % (n_parts - kStreams * row_splits);
            prm.m_part[(static_cast<int64_t>(b) * prm.Hq + hk * R + r) * n_parts + part] = -INFINITY;
        }
    auto prep_query_row = [&](int r, bool to_smem) {
        const int hq = hk * R + r;
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
            if (to_smem) {
                *reinterpret_cast<__half*>(sm + kOffQ16 + (e >> 6) * 1024 + r * 128 + ((((e & 63) >> 3) ^ r) << 4) + (e & 7) * 2) = qrow[e];
                *reinterpret_cast<int8_t*>(sm + kOffQ8 + r * 128 + (((e >> 4) ^ r) << 4) + (e & 15)) = static_cast<int8_t>(q8);
            }
            if (q_writer && prm.q8_out != nullptr)
                prm.q8_out[(static_cast<int64_t>(b) * prm.Hq + hq) * D + e] = static_cast<int8_t>(q8);
        }
        if (lane == 0) {
            if (to_smem) sh.dq[r] = delta;
            if (q_writer && prm.qs_out != nullptr) prm.qs_out[static_cast<int64_t>(b) * prm.Hq + hq] = delta;
        }
    };

    if (n_it <= 0) {                      // a split without keys: the merge skips it
        for (int idx = tid; idx < kStreams * R * D; idx += kThreads) {
            const int g = idx / (R * D), rd = idx % (R * D);
            prm.o_part[(out_row0 + static_cast<int64_t>(rd / D) * n_parts + g) * D + (rd % D)] = 0.f;
        }
        if (tid < kStreams * R) {
            prm.m_part[out_row0 + static_cast<int64_t>(tid % R) * n_parts + tid / R] = -INFINITY;
            prm.z_part[out_row0 + static_cast<int64_t>(tid % R) * n_parts + tid / R] = 0.f;
        }
        if (q_writer && warp < R) prep_query_row(warp, false);   // (a row without keys still reports its quantised query)
        leave();
        return;
    }

    const float* dk = prm.k_scale + (static_cast<int64_t>(b) * prm.Hk + hk) * prm.n_blk;
    const float* dv = prm.v_scale + (static_cast<int64_t>(b) * prm.Hk + hk) * prm.n_blk;
    auto route_of = [&](int tile) -> bool {
        if (wrow == nullptr) return false;
        const int grp = tile / prm.G;
        return (wrow[grp >> 5] >> (grp & 31)) & 1u;
    };
    if constexpr (!F16K) {
        // No FP16 key cache was passed: every group inside the cache length has to be INT8-routed.  A 0 bit is
        // found here, before anything is allocated or copied; the CTA records it and leaves.
        int fp16_group = 0;
        for (int tile = t0 + tid; tile < t1; tile += kThreads) fp16_group |= route_of(tile) ? 0 : 1;
        if (__syncthreads_or(fp16_group)) {
            ptx::griddep_wait();
            if (tid == 0 && atomicCAS(&prm.status[0], 0, TILEMIX_ERR_NULL) == 0) {
                prm.status[1] = 16; prm.status[2] = t0; prm.status[3] = 1;
            }
            leave();
            return;
        }
    }

    ptx::griddep_launch_dependents();     // the merge kernel may be brought in; it waits for this grid to finish
    volatile int* abort_flag = &sh.abort_flag;

    // Bounded wait on one mbarrier phase; false when the CTA is giving up.
    auto wait = [&](uint64_t* bar, uint32_t parity, int which) -> bool {
        const uint32_t addr = ptx::smem_u32(bar);
        if (ptx::mbar_try_wait(addr, parity)) return true;
        const uint64_t start = ptx::globaltimer_ns();
        uint32_t spins = 0;
        while (!ptx::mbar_try_wait(addr, parity)) {
            if ((++spins & 63u) == 0u) {
                if (*abort_flag) return false;
                if (ptx::globaltimer_ns() - start > prm.wait_limit_ns) {
                    *abort_flag = 1;
                    ptx::griddep_wait();
                    if (atomicCAS(&prm.status[0], 0, TILEMIX_ERR_DEVICE_TIMEOUT) == 0) {
                        prm.status[1] = 16; prm.status[2] = t0; prm.status[3] = which;
                    }
                    return false;
                }
            }
        }
        return true;
    };
    auto tile_int8 = [&](int it) -> bool { return it < kMetaTiles ? meta[it].x >= 0.f : route_of(t0 + it); };
    constexpr uint32_t kHi = ptx::desc_hi(1024, 2);   // 8-row groups of 1024 bytes, 128-byte swizzle

    int last_issued = -1;                 // (producer lane) the last tile whose copies were started
    if (warp == kProducerWarp) {
        // ============================================================ copy producer (one lane)
        if (lane == 0) {
            const int8_t* v8g = prm.v8 + (static_cast<int64_t>(b) * prm.Hk + hk) * prm.max_len * D;
            int head = 0, used = 0, freed = 0;
            // Route bits straight from the mask words (the staged tile metadata is not there yet when this loop
            // starts), without a division per tile: group index and position inside the group advance with the
            // tile, one mask word is kept in a register, and the routes of the tiles in the ring are remembered
            // as bits (tile it -> bit it % 32) for the moment their units come back.
            uint32_t grp = static_cast<uint32_t>(t0 / prm.G), in_grp = static_cast<uint32_t>(t0 % prm.G);
            uint32_t cw = wrow != nullptr ? wrow[grp >> 5] : 0u, routes = 0u;
            for (int it = 0; it < n_it; ++it) {
                const bool i8 = (cw >> (grp & 31u)) & 1u;
                routes = (routes & ~(1u << (it & 31))) | (static_cast<uint32_t>(i8) << (it & 31));
                if (++in_grp == static_cast<uint32_t>(prm.G)) {
                    in_grp = 0;
                    ++grp;
                    if ((grp & 31u) == 0u && wrow != nullptr && it + 1 < n_it) cw = wrow[grp >> 5];
                }
                const int need = i8 ? 2 : 3;
                bool ok = true;
                while (used + need > kUnits || it - freed >= kSlots) {
                    if (!wait(&sh.freeb[freed % kSlots], (freed / kSlots) & 1, kWFree)) { ok = false; break; }
                    used -= ((routes >> (freed & 31)) & 1u) ? 2 : 3;
                    ++freed;
                }
                if (!ok) break;
                const int s = it % kSlots;
                const uint32_t u0 = head, u1 = (head + 1) % kUnits, u2 = (head + 2) % kUnits;
                const uint32_t uv = i8 ? u1 : u2;
                head = (head + need) % kUnits;
                used += need;
                *reinterpret_cast<volatile uint32_t*>(&sh.slot_info[s]) = u0 | (u1 << 8) | (uv << 16);
                if (it == prm.test_drop_tile) continue;   // testing aid: this tile never lands, the consumers' waits run out
                const int tile = t0 + it;
                const uint32_t rows = static_cast<uint32_t>(min(T, len - tile * T));
                const uint32_t bar = ptx::smem_u32(&sh.full[s]);
                // the tiled copies always bring a whole box (rows past the cache are stale or zero-filled and are
                // masked as keys); the plain copy of V8 brings the rows that exist
                ptx::mbar_arrive_expect_tx(bar, (i8 ? kUnit : 2 * kUnit) + rows * D);
                if (i8) {
                    ptx::tma_load_4d(sbase + kOffRing + u0 * kUnit, &tm_k8, bar, 0, tile * T, hk, b);
                } else {
                    ptx::tma_load_4d(sbase + kOffRing + u0 * kUnit, &tm_k16, bar, 0, tile * T, hk, b);
                    ptx::tma_load_4d(sbase + kOffRing + u1 * kUnit, &tm_k16, bar, 64, tile * T, hk, b);
                }
                ptx::bulk_load_1d(sbase + kOffRing + uv * kUnit, v8g + static_cast<int64_t>(tile) * T * D, rows * D, bar);
                last_issued = it;
            }
        }
    } else {
        // ---- everyone but the producer: the operand tiles of Q are made while the first copies fly -----------------
        const int nid = tid < kProducerWarp * 32 ? tid : tid - 32;
        {
            // rows R..7 of the P and Q tiles are never written: zero them once (finite values in the unused rows)
            uint4* z = reinterpret_cast<uint4*>(sm + kOffP);
            for (int i = nid; i < (kOffRing - kOffP) / 16; i += kThreads - 32) z[i] = make_uint4(0u, 0u, 0u, 0u);
        }
        for (int i = nid; i < kMetaTiles && i < n_it; i += kThreads - 32) {
            const int tile = t0 + i;
            meta[i] = make_float2(route_of(tile) ? dk[tile] : -1.f, dv[tile]);
        }
        ptx::bar_sync_named(1, kThreads - 32);
        if (warp >= kConvWarp0 && warp < kConvWarp0 + R) prep_query_row(warp - kConvWarp0, true);
        ptx::fence_proxy_async_smem();        // operand tiles written with ordinary stores, read by the tensor pipe
        ptx::bar_sync_named(1, kThreads - 32);

        if (warp == kQkWarp) {
        // ============================================================ QK^T issuer (whole warp, elected-lane issue)
        constexpr uint32_t kIdescQK8 = ptx::instr_desc(2, 1, 0, 0, T, 16);
        constexpr uint32_t kIdescQK16 = ptx::instr_desc(1, 0, 0, 0, T, 16);
        const uint32_t q8_lo = ptx::desc_lo(sbase + kOffQ8, 16);
        bool ok = true;
        for (int j = 0; j < n_pairs && ok; ++j) {
            const int pb = j & 1;
            if (j >= 2 && !wait(&sh.s_free[pb], ((j >> 1) - 1) & 1, kWSFree)) break;   // the softmax warps have read pair j - 2
            for (int h = 0; h < 2; ++h) {
                const int it = 2 * j + h;
                if (it >= n_it) break;
                const int s = it % kSlots;
                if (!wait(&sh.full[s], (it / kSlots) & 1, kWFull)) { ok = false; break; }
                ptx::tc_fence_after_sync();
                const uint32_t info = *reinterpret_cast<volatile uint32_t*>(&sh.slot_info[s]);
                const uint32_t d_tmem = tmem_base + (2 * pb + h) * 16;
                if (tile_int8(it)) {
                    const uint32_t a_lo = ptx::desc_lo(sbase + kOffRing + (info & 0xffu) * kUnit, 16);
                    ptx::mma_i8_ss<false>(d_tmem, a_lo, kHi, q8_lo, kHi, kIdescQK8);
#pragma unroll
                    for (int k = 1; k < D / 32; ++k)
                        ptx::mma_i8_ss<true>(d_tmem, a_lo + 2 * k, kHi, q8_lo + 2 * k, kHi, kIdescQK8);
                } else {
#pragma unroll
                    for (int c = 0; c < 2; ++c) {
                        const uint32_t a_lo = ptx::desc_lo(sbase + kOffRing + ((info >> (8 * c)) & 0xffu) * kUnit, 16);
                        const uint32_t b_lo = ptx::desc_lo(sbase + kOffQ16 + c * 1024, 16);
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            if (c == 0 && k == 0) ptx::mma_f16_ss<false>(d_tmem, a_lo, kHi, b_lo, kHi, kIdescQK16);
                            else ptx::mma_f16_ss<true>(d_tmem, a_lo + 2 * k, kHi, b_lo + 2 * k, kHi, kIdescQK16);
                        }
                    }
                }
                ptx::mma_commit(ptx::smem_u32(&sh.freeb[s]));     // the key tile has been read
            }
            if (ok) ptx::mma_commit(ptx::smem_u32(&sh.s_ready[pb]));
        }
        // every MMA issued by this warp has retired before tensor / shared memory go away
        ptx::mma_commit(ptx::smem_u32(&sh.drain_qk));
        wait(&sh.drain_qk, 0, kWDrain);
        } else if (warp == kPvWarp) {
        // ============================================================ PV issuer (whole warp, elected-lane issue)
        constexpr uint32_t kIdescPV = ptx::instr_desc(1, 0, 0, 1, kPRows, D);
        bool ok = true;
        for (int j = 0; j < n_pairs && ok; ++j) {
            const int pb = j & 1;
            if (!wait(&sh.p_ready[pb], (j >> 1) & 1, kWP)) break;
            for (int h = 0; h < 2; ++h) {
                const int it = 2 * j + h;
                if (it >= n_it) break;
                const uint32_t a_base = ptx::desc_lo(sbase + kOffP + (2 * pb + h) * kPTile, 16);
                // the FP16 copy of V arrives in two halves of 64 keys, each in its own buffer
#pragma unroll
                for (int hf = 0; hf < 2; ++hf) {
                    if (!wait(&sh.v_ready[hf], it & 1, kWV)) { ok = false; break; }
                    ptx::tc_fence_after_sync();
                    const uint32_t b_base = ptx::desc_lo(sbase + kOffV16 + hf * kVHalf, kVHalf / 2);
#pragma unroll
                    for (int k = 0; k < 4; ++k)   // 16 keys per step: 32 bytes of a P row, 16 rows (2048 bytes) of V16
                        ptx::mma_f16_ss_rt(tmem_base + kColO + pb * 128, a_base + hf * (1024 >> 4) + 2 * k, kHi,
                                           b_base + k * 128, kHi, kIdescPV, (j >= kStreams || h > 0 || hf > 0 || k > 0) ? 1u : 0u);
                    ptx::mma_commit(ptx::smem_u32(&sh.pv_done[hf]));
                }
                if (!ok) break;
            }
            if (ok) ptx::mma_commit(ptx::smem_u32(&sh.pv_pair[pb]));
        }
        ptx::mma_commit(ptx::smem_u32(&sh.drain_pv));
        wait(&sh.drain_pv, 0, kWDrain);
        } else if (warp >= kConvWarp0) {
        // ============================================================ V8 -> FP16 (two groups of eight warps)
        // Group hf converts keys 64 hf .. 64 hf + 63 of every tile into its own FP16 buffer (a role's step is mostly
        // the fixed cost of its waits and its proxy fence: two groups in parallel halve it per tile).  A thread takes
        // its two 16-byte pieces of a landed V8 tile into registers (the ring unit goes back to the producer at
        // once) and converts them when the PV that read the buffer last has retired.
        // Piece idx of a half = columns 16q .. 16q+15 of one of its 64 keys.  Eight consecutive pieces are four
        // pieces of one 64-column half of a key and four of the other half of the next key: read as INT8 they are
        // the two halves of a 128-byte line, and as FP16 they are the even 16-byte chunks of one key's 128-byte row
        // and the odd ones of the other's (the swizzle flips the parity with the row), so a quarter warp's
        // 128-bit loads and stores each fall into eight different bank groups.
        const int hf = (warp - kConvWarp0) >> 3;
        const int cid = ((warp - kConvWarp0) & 7) * 32 + lane;
        constexpr int kGroupThreads = kConvThreads / 2, kPer = (T / 2) * D / 16 / kGroupThreads;
        const __half2 off = __floats2half2_rn(1152.f, 1152.f);
        uint8_t* vbuf = sm + kOffV16 + hf * kVHalf;
        for (int it = 0; it < n_it; ++it) {
            const int s = it % kSlots;
            if (!wait(&sh.full[s], (it / kSlots) & 1, kWFull)) break;
            const uint32_t info = *reinterpret_cast<volatile uint32_t*>(&sh.slot_info[s]);
            const uint8_t* src = sm + kOffRing + ((info >> 16) & 0xffu) * kUnit + hf * (T / 2) * D;
            uint4 in[kPer];
#pragma unroll
            for (int j = 0; j < kPer; ++j) {
                const int idx = cid + kGroupThreads * j;
                const int row = ((idx >> 4) << 1) | ((idx >> 2) & 1), q = ((((idx >> 3) ^ (idx >> 2)) & 1) << 2) | (idx & 3);
                in[j] = *reinterpret_cast<const uint4*>(src + row * D + q * 16);
            }
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&sh.freeb[s]));    // the V8 tile has been read
            if (it >= 1 && !wait(&sh.pv_done[hf], (it - 1) & 1, kWPV)) break;   // the PV that read this buffer
#pragma unroll
            for (int j = 0; j < kPer; ++j) {
                const int idx = cid + kGroupThreads * j;
                const int row = ((idx >> 4) << 1) | ((idx >> 2) & 1), q = ((((idx >> 3) ^ (idx >> 2)) & 1) << 2) | (idx & 3);
                const uint32_t w[4] = {in[j].x, in[j].y, in[j].z, in[j].w};
                uint32_t h[8];
#pragma unroll
                for (int y = 0; y < 4; ++y) {
                    // half2(1024 + (x + 128)) - 1152 = half2(x), exactly
                    const uint32_t u = w[y] ^ 0x80808080u;
                    uint32_t lo = __byte_perm(u, 0x64646464u, 0x4140), hi = __byte_perm(u, 0x64646464u, 0x4342);
                    const __half2 v0 = __hsub2(*reinterpret_cast<const __half2*>(&lo), off);
                    const __half2 v1 = __hsub2(*reinterpret_cast<const __half2*>(&hi), off);
                    h[2 * y] = *reinterpret_cast<const uint32_t*>(&v0);
                    h[2 * y + 1] = *reinterpret_cast<const uint32_t*>(&v1);
                }
                // slab q / 4, 16-byte chunks 2(q % 4) and + 1 of the key's 128-byte row, swizzled by the row
                uint8_t* rowp = vbuf + (q >> 2) * (kVHalf / 2) + row * 128;
                const int c0 = 2 * (q & 3), sw = row & 7;
                *reinterpret_cast<uint4*>(rowp + ((c0 ^ sw) << 4)) = make_uint4(h[0], h[1], h[2], h[3]);
                *reinterpret_cast<uint4*>(rowp + (((c0 + 1) ^ sw) << 4)) = make_uint4(h[4], h[5], h[6], h[7]);
            }
            ptx::fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&sh.v_ready[hf]));
        }
        } else {
        // ============================================================ softmax (thread = one key of each tile of a step)
        const int g = warp >> 2, wq = warp & 3;       // stream, TMEM lane quarter
        const int key = wq * 32 + lane;
        float m_run[R], z_part[R], a_q[R];
        uint32_t p_off[R];
#pragma unroll
        for (int r = 0; r < R; ++r) {
            m_run[r] = -INFINITY;
            z_part[r] = 0.f;
            a_q[r] = prm.scale_log2 * sh.dq[r];
            p_off[r] = (key >> 6) * 1024 + r * 128 + ((((key & 63) >> 3) ^ r) << 4) + (key & 7) * 2;
        }
        const uint32_t t_lane = tmem_base + (static_cast<uint32_t>(wq * 32) << 16);
        const uint32_t col_o = kColO + g * 128;
        const int64_t orow = out_row0 + static_cast<int64_t>(lane < R ? lane : 0) * n_parts + g;   // (lanes < R of quarter 0)
        if (g >= n_pairs) {
            // a stream without a step: an empty partial result, which the merge skips
            for (int idx = key; idx < R * D; idx += kStreamWarps * 32)
                prm.o_part[(out_row0 + static_cast<int64_t>(idx / D) * n_parts + g) * D + (idx % D)] = 0.f;
            if (wq == 0 && lane < R) { prm.m_part[orow] = -INFINITY; prm.z_part[orow] = 0.f; }
        }
        for (int j = g; j < n_pairs; j += kStreams) {
            const uint32_t par = (j >> 1) & 1;        // phase parity of this stream's barriers at this step
            const bool two = 2 * j + 1 < n_it;
            bool int8[2];
            float dkt[2], dvt[2];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int it = min(2 * j + h, n_it - 1), tile = t0 + it;
                if (it < kMetaTiles) {
                    const float2 mt = meta[it];
                    int8[h] = mt.x >= 0.f; dkt[h] = mt.x; dvt[h] = mt.y;
                } else {
                    int8[h] = route_of(tile); dkt[h] = int8[h] ? dk[tile] : 0.f; dvt[h] = dv[tile];
                }
            }
            if (!wait(&sh.s_ready[g], par, kWS)) break;
            ptx::tc_fence_after_sync();
            uint32_t raw[2][RC];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                if constexpr (RC == 4) ptx::tmem_ld32x32_x4(t_lane + (2 * g + h) * 16, raw[h]);
                else ptx::tmem_ld32x32_x8(t_lane + (2 * g + h) * 16, raw[h]);
            }
            ptx::tmem_wait_ld_dep(raw[0], raw[1]);    // ties the registers to the wait: no use of them moves above it
            ptx::tc_fence_before_sync();
            ptx::mbar_arrive(ptx::smem_u32(&sh.s_free[g]));
            float sc[2][R];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                // keys past the cache (stale rows) and the missing second tile of the last step do not exist
                const bool exists = (h == 0 || two) && (t0 + 2 * j + h) * T + key < len;
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    const float x = int8[h] ? static_cast<float>(static_cast<int>(raw[h][r])) * (a_q[r] * dkt[h])
                                            : __uint_as_float(raw[h][r]) * prm.scale_log2;
                    sc[h][r] = exists ? x : -INFINITY;
                }
            }
            // maximum of the step per row: over the warp (order-preserving integer image of the float), then
            // over the four warps of the stream through shared memory
#pragma unroll
            for (int r = 0; r < R; ++r) {
                int o = __float_as_int(fmaxf(sc[0][r], sc[1][r]));
                o = o >= 0 ? o : o ^ 0x7fffffff;
                o = __reduce_max_sync(0xffffffffu, o);
                o = o >= 0 ? o : o ^ 0x7fffffff;
                if (lane == 0) sh.warp_max[g][wq][r] = __int_as_float(o);
            }
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&sh.xchg[g]));
            if (!wait(&sh.xchg[g], par, kWXchg)) break;
            bool move = false;
            float mt[R];
#pragma unroll
            for (int r = 0; r < R; ++r) {
                mt[r] = fmaxf(fmaxf(sh.warp_max[g][0][r], sh.warp_max[g][1][r]),
                              fmaxf(sh.warp_max[g][2][r], sh.warp_max[g][3][r]));
                move |= mt[r] > m_run[r] + kMoveAbove;      // always on the stream's first step (m = -inf)
            }
            // The PVs of this stream's previous step have retired: they read the P tiles written below and they
            // accumulate into the O that a move of m rescales.  (A barrier per stream whose next phase cannot
            // complete before this step hands P over, so the wait cannot be lapped.)
            if (j >= kStreams && !wait(&sh.pv_pair[g], par ^ 1u, kWPV)) break;
            if (move) {                                      // uniform over the stream
                float alpha_lane = 1.f;
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    const float mn = mt[r] > m_run[r] + kMoveAbove ? mt[r] : m_run[r];
                    const float alpha = exp2f(m_run[r] - mn);    // 0 on the first step
                    z_part[r] *= alpha;
                    m_run[r] = mn;
                    if (lane == r) alpha_lane = alpha;
                }
                if (j >= kStreams && wq == 0) {
                    // rows 0..R-1 of this stream's O (lanes 0..R-1 of tensor memory); the PVs of this step cannot
                    // start before this warp hands P over
                    ptx::tc_fence_after_sync();
#pragma unroll 1
                    for (int c = 0; c < D / 32; ++c) {
                        uint32_t o[32];
                        ptx::tmem_ld32(tmem_base + col_o + 32 * c, o);
                        ptx::tmem_wait_ld_dep(o);
#pragma unroll
                        for (int x = 0; x < 32; ++x) o[x] = __float_as_uint(__uint_as_float(o[x]) * alpha_lane);
                        ptx::tmem_st32(tmem_base + col_o + 32 * c, o);
                    }
                    ptx::tmem_wait_st();
                    ptx::tc_fence_before_sync();
                }
            }
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                uint8_t* pbuf = sm + kOffP + (2 * g + h) * kPTile;
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    float p;
                    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(p) : "f"(sc[h][r] - m_run[r]));
                    z_part[r] += p;
                    *reinterpret_cast<__half*>(pbuf + p_off[r]) = __float2half_rn(p * dvt[h]);
                }
            }
            ptx::fence_proxy_async_smem();
            ptx::mbar_arrive(ptx::smem_u32(&sh.p_ready[g]));
            if (j + kStreams >= n_pairs) {
                // ---- the stream's last step: (m, z, O~) to the workspace
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    float z = z_part[r];
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
                    if (lane == 0) sh.zsum[g][wq][r] = z;
                }
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&sh.zbar[g]));
                if (wq != 0) break;
                if (!wait(&sh.zbar[g], 0, kWXchg)) break;
                if (!wait(&sh.pv_pair[g], par, kWPV)) break;      // the PVs of this step
                ptx::tc_fence_after_sync();
#pragma unroll 1
                for (int c = 0; c < D / 32; ++c) {
                    uint32_t o[32];
                    ptx::tmem_ld32(tmem_base + col_o + 32 * c, o);
                    ptx::tmem_wait_ld_dep(o);
                    if (lane < R) {
                        float4* dstp = reinterpret_cast<float4*>(prm.o_part + orow * D + 32 * c);
#pragma unroll
                        for (int x = 0; x < 8; ++x)
                            dstp[x] = make_float4(__uint_as_float(o[4 * x]), __uint_as_float(o[4 * x + 1]),
                                                  __uint_as_float(o[4 * x + 2]), __uint_as_float(o[4 * x + 3]));
                    }
                }
                if (lane < R) {
                    float mine = -INFINITY;
#pragma unroll
                    for (int r = 0; r < R; ++r) if (lane == r) mine = m_run[r];
                    prm.m_part[orow] = mine;
                    prm.z_part[orow] = sh.zsum[g][0][lane] + sh.zsum[g][1][lane] + sh.zsum[g][2][lane] + sh.zsum[g][3][lane];
                }
                ptx::tc_fence_before_sync();
            }
        }
        }
    }

    // ---- every role is out of its loop ---------------------------------------------------------------------
    __syncthreads();
    if (*abort_flag && warp == kProducerWarp && lane == 0) {
        // the copies still in flight land before this CTA's shared memory is given back
        for (int it = max(0, last_issued - kSlots + 1); it <= last_issued; ++it) {
            if (it == prm.test_drop_tile) continue;
            for (int spin = 0; spin < (1 << 16); ++spin)
                if (ptx::mbar_try_wait(ptx::smem_u32(&sh.full[it % kSlots]), (it / kSlots) & 1)) break;
        }
    }
    __syncthreads();
    if (warp == kProducerWarp) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, kTmemCols);
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// Map over a [B, Hk, max_len, 128] cache (innermost first: d, token, head, sequence); box = box_d x 128 tokens.
int encode_cache_map(EncodeTiledFn enc, CUtensorMap* tm, const void* base, int elem_bytes, const DecodeParams& prm,
                     int box_d) {
    const cuuint64_t dims[4] = {static_cast<cuuint64_t>(D), static_cast<cuuint64_t>(prm.max_len),
                                static_cast<cuuint64_t>(prm.Hk), static_cast<cuuint64_t>(prm.B)};
    const cuuint64_t row = static_cast<cuuint64_t>(D) * elem_bytes;
    const cuuint64_t strides[3] = {row, row * prm.max_len, row * prm.max_len * prm.Hk};
    const cuuint32_t box[4] = {static_cast<cuuint32_t>(box_d), static_cast<cuuint32_t>(T), 1u, 1u};
    const cuuint32_t estr[4] = {1u, 1u, 1u, 1u};
    return static_cast<int>(enc(tm, elem_bytes == 2 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_UINT8, 4,
                                const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE));
}

template <int R>
int launch_r(const DecodeParams& prm, const CUtensorMap& tk8, const CUtensorMap& tk16, cudaStream_t stream) {
    auto kernel = prm.k16 != nullptr ? decode_umma_kernel<R, true> : decode_umma_kernel<R, false>;
    // the kernel's shared-memory attribute is set once per device and instance
    constexpr int kMaxDev = 64;
    static std::atomic<int> attr_set[kMaxDev][2];
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return static_cast<int>(e);
    const int which = prm.k16 != nullptr ? 1 : 0;
    if (dev < 0 || dev >= kMaxDev || attr_set[dev][which].load(std::memory_order_acquire) == 0) {
        e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        if (e != cudaSuccess) return static_cast<int>(e);
        if (dev >= 0 && dev < kMaxDev) attr_set[dev][which].store(1, std::memory_order_release);
    }
    const dim3 grid = prm.balanced ? dim3(prm.n_ctas) : dim3(prm.n_splits, prm.Hk, prm.B);
    // programmatic dependent launch: this grid's set-up overlaps the tail of the prepare kernel
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = dim3(kThreads); cfg.dynamicSmemBytes = kSmemBytes; cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    e = cudaLaunchKernelEx(&cfg, kernel, tk8, tk16, prm);
    g_launch_count.fetch_add(1);
    return static_cast<int>(e);
}

}  // namespace

int launch_decode_umma(int R, const DecodeParams& prm, cudaStream_t stream) {
    static std::atomic<void*> encoder{nullptr};      // the driver's tensor-map encoder, looked up once
    void* sym = encoder.load(std::memory_order_acquire);
    if (sym == nullptr) {
        cudaDriverEntryPointQueryResult qres;
        const cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres);
        if (e != cudaSuccess) return static_cast<int>(e);
        if (qres != cudaDriverEntryPointSuccess || sym == nullptr) return static_cast<int>(cudaErrorNotSupported);
        encoder.store(sym, std::memory_order_release);
    }
    EncodeTiledFn enc = reinterpret_cast<EncodeTiledFn>(sym);
    CUtensorMap tk8, tk16;
    int rc = encode_cache_map(enc, &tk8, prm.k8, 1, prm, 128);
    if (rc) return rc;
    if (prm.k16 != nullptr) {
        if ((rc = encode_cache_map(enc, &tk16, prm.k16, 2, prm, 64))) return rc;
    } else {
        tk16 = tk8;
    }
    switch (R) {
        case 1: return launch_r<1>(prm, tk8, tk16, stream);
        case 2: return launch_r<2>(prm, tk8, tk16, stream);
        case 4: return launch_r<4>(prm, tk8, tk16, stream);
        case 8: return launch_r<8>(prm, tk8, tk16, stream);
        default: return TILEMIX_ERR_UNSUPPORTED;
    }
}

}  // namespace tilemix
