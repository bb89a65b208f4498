// Fused TileMix attention forward for sm_100a (Sec. 4.1 loops, Sec. 4.3 "Tile-group dispatch",
// Sec. 3.1 online softmax, App. C score formulas).
//
// One CTA owns two adjacent query tiles (A = 2p, B = 2p+1) of one (batch, query head) and
// streams the key/value tiles 0..B once for both.  Warp roles (w = warp index):
//   warps 0-15  softmax warps: tile (w >> 2) & 1, 16 query rows each -- TMEM lanes 32 (w & 3) + 16 (w >> 3)
//               .. + 15 (a warp may only touch the lane quarter w & 3), read in the 16-lane shapes so that the
//               four warps of a scheduler work on four disjoint sets of rows
//   warp  16    TMA producer: Q16/Q8 once, then per key tile the K operand(s) the routing bits ask for
//               (FP16 and/or INT8) and V, into a ring of equally sized shared-memory chunks
//   warps 17,18 MMA issuers, one per query tile: tcgen05.mma kind::f16 or kind::i8 for S = Q K^T per the
//               routing bit, then kind::f16 for O += P V with P read from tensor memory; warp 17 also owns
//               the TMEM allocation.  The whole warp runs the loop, one elected lane issues.
//   warp  19    idle
//   warps 20-23 only in the on-the-fly operand mode: the on-chip quantiser, which makes the INT8 copies of
//               the query tiles and of the key tiles routed to INT8 in shared memory from the FP16 tiles
// Tensor memory: S_A | S_B | O_A | O_B (FP32 / INT32 accumulators).  A score tile is produced and consumed in
// two halves of T/2 key columns; the FP16 probabilities P of a half overwrite the start of that half.  While
// the softmax warps of a tile turn one half into P, the tensor pipe runs the PV of the other half and the
// QK^T of the next key tile into it.
//
// Every wait is bounded: when one runs out the CTA records a status, raises an abort flag all
// roles poll, drains what is in flight and returns.
#include <cuda.h>
#include <cuda_fp16.h>

#include "common.cuh"
#include "ptx_sm100.cuh"
#include "quant8.cuh"
#include "softmax_tile.cuh"

namespace tilemix {

namespace {

constexpr int kSoftmaxWarps = 16;         // 8 per query tile, 16 rows each
constexpr int kProducerWarp = 16;
constexpr int kMmaWarp = 17;
// setmaxnreg only moves registers inside what the block was launched with (threads x registers per thread); an
// increase beyond that waits for ever.  640 threads start with 96 registers: 512*104 + 128*64 = 61440 = 640*96.
constexpr int kThreads = 640;
constexpr int kLaunchRegs = 96;
constexpr int kRegsSoftmax = 104, kRegsOther = 64;
// On-the-fly operand mode: a sixth warpgroup, the on-chip quantiser (32 rows of a tile per warp).  768 threads
// start with 80 registers: 512*96 + 256*48 = 61440 = 768*80.
constexpr int kQuantWarp0 = 20, kQuantWarps = 4;
constexpr int kThreadsOtf = 768;
constexpr int kLaunchRegsOtf = 80;
constexpr int kRegsSoftmaxOtf = 96, kRegsOtherOtf = 48;
static_assert(kSoftmaxWarps * 32 * kRegsSoftmax + (kThreads - kSoftmaxWarps * 32) * kRegsOther <= kThreads * kLaunchRegs, "setmaxnreg split");
static_assert(kSoftmaxWarps * 32 * kRegsSoftmaxOtf + (kThreadsOtf - kSoftmaxWarps * 32) * kRegsOtherOtf <= kThreadsOtf * kLaunchRegsOtf, "setmaxnreg split");
constexpr uint32_t kQuantBar = 9;         // named barrier of the quantiser warps
constexpr int kMaxHeadGroup = 8;   // (batch, head) rows whose CTAs are interleaved in the grid order, at most
constexpr int kRing = 8;
constexpr int kBundles = 4;        // operand bundles in flight at most (each has a "landed" and a "consumed" barrier)
constexpr int kWorkspaceClearBytes = 4096;  // status record
constexpr int kMaxTiles = 2048;           // key tiles per row the shared-memory schedule table holds
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
// Lazy running maximum.  P = 2^(score - m) is handed to the tensor pipe in FP16 (largest finite value just
// below 2^16), z and O are FP32, so m may lag the true row maximum.  An interior step is done in one pass with
// the current m and is accepted when this thread's part of each row sum stays below 2^kAccept (no probability
// of the step can then exceed 2^kAccept).  Otherwise the step is redone from the accumulators in the generic
// two-pass form, which moves m to kMargin above the step's maximum whenever that maximum is more than kMove above
// m (a rejected step always is: 2^kAccept spread over at most 16 values) and rescales z and O.  After a move
// P tops out at 2^-kMargin, 18 binades above the smallest FP16 subnormal, and a later score has to beat
// everything before it by 2^(kMove + kMargin) to move m again.
constexpr float kAccept = 8.0f, kMove = 4.0f, kMargin = 6.0f;
// the INT8 route leaves the conversion bias to the scaling FMA while a * 1.5*2^23 <= kFoldLimit: the addend
// m + a*1.5*2^23 is then below 2^13 and its rounding moves a score by at most 2^-12 (a relative 1.7e-4 in P)
constexpr float kFoldLimit = 4096.0f;

enum Role : int { kRoleSoftmaxA = 0, kRoleSoftmaxB = 1, kRoleProducer = 2, kRoleMma = 3, kRoleQuant = 4 };
enum Bar : int { kBarQ = 0, kBarRingFull = 1, kBarRingEmpty = 2, kBarS = 3, kBarP = 4, kBarO = 5, kBarDrain = 6, kBarPV = 7,
                 kBarRaw = 8, kBarQ8 = 9 };

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
    static constexpr int kTH = T / 2;                 // key columns per half step
    static constexpr int kNumBars = 2 + 2 * kRing + 4 + 4 + 2 + 2 + 1 + kBundles + 2;
    static constexpr int kOffMisc = kOffBars + kNumBars * 8;       // tmem base, abort flag; on-chip scales
    static constexpr int kOffWords = kOffMisc + 64;
    static constexpr int kSmemBytes = kOffWords + kMaxTiles / 2;   // 4-bit schedule entries
    static constexpr int kSmemAlloc = kSmemBytes + 1024;           // slack to align the base
    static_assert(kK8Bytes <= kChunk, "INT8 key tile must fit one ring chunk");
    static_assert(kTmemCols == 256 || kTmemCols == 512, "TMEM allocation must be a power of two");
    static_assert(kSmemAlloc <= 232448, "exceeds the 227 KB shared memory of a CTA");
    static_assert(T % 32 == 0 && D % 64 == 0, "tile shape");
};

struct Params {
    int B, Hq, Hk, L, G, T_m, W, nb;
    int kv_off, mask_T_m, ks_blocks;   // chunked prefill: see Geometry (0, T_m, T_m for a plain prefill)
    int k_half_blocks;                 // 1: delta_K per half key tile (quantisation block = tile_n / 2), 0: per key tile
    unsigned long long wait_limit_ns;  // limit of every bounded wait
    int test_drop_bundle;              // testing aid: the producer leaves out the copies of this operand bundle (-1: none)
    int head_group;               // (batch, head) rows interleaved in the grid order (>= 1)
    int has_int8;                 // INT8 operands present
    float scale_log2;             // softmax scale * log2(e)
    const float* q_scale;         // [B,Hq,T_m]; variable-length batch: [sum T_m, Hq]
    const float* k_scale;         // [B,Hk,T_n]; variable-length batch: [sum T_n, Hk]
    const float* v_scale;         // [B,Hk,vs_blocks] block scales of an INT8 value cache (VS instances), else null
    int vs_blocks;                // key tiles of the context
    const uint32_t* words;        // [nb,Hk,T_m,W] or null (all FP16)
    // Variable-length batch (null = one dense batch): prefix sums over the sequences.  Then B = 1,
    // L = total tokens and T_m = total query-tile rows of the packed batch.
    const int32_t* vl_tok;        // [n_seqs+1] first token of each sequence
    const int32_t* vl_tile;       // [n_seqs+1] query-tile rows before each sequence
    const int32_t* vl_blkk;       // [n_seqs+1] quantisation blocks of K before each sequence
    const int32_t* vl_item_seq;   // [total_pairs] work item -> sequence (longest rows first)
    const int32_t* vl_item_pair;  // [total_pairs] work item -> pair of query tiles of that sequence
    int n_seqs, total_pairs;
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
    unsigned long long wait_limit_ns;
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
            if (ptx::globaltimer_ns() - t0 > cx.wait_limit_ns) {
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

// VL: variable-length batch (the work item is found in the sequence prefix sums).
// OTF: on-the-fly operand generation (App. D, "fused on-the-fly" mode): there are no INT8 copies of Q and K
// and no scales in global memory; a quantiser warp makes them in shared memory from the FP16 tiles, for
// the key tiles some query tile of the CTA routes to INT8 only.
// DBG: the instance that can write the raw accumulators of requested tiles (every step then takes the generic form).
// A kernel of its own, because every instruction in the softmax warps' loop that is not executed still costs: the loop
// of the other instances is ~1 % faster without that code in it.
template <int D, int T, bool VL, bool OTF, bool VS = false, bool DBG = false>
__global__ void __launch_bounds__(OTF ? kThreadsOtf : kThreads, 1)
attention_kernel(const Params prm, const __grid_constant__ CUtensorMap tm_q16,
                 const __grid_constant__ CUtensorMap tm_k16, const __grid_constant__ CUtensorMap tm_v16,
                 const __grid_constant__ CUtensorMap tm_q8, const __grid_constant__ CUtensorMap tm_k8) {
    using C = Cfg<D, T>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sbase = ptx::smem_u32(smem);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    // An earlier CTA of this launch already failed: do nothing (decided once per CTA; the status word is read
    // here and looked at behind the set-up barrier, so that its latency hides behind the set-up).
    __shared__ int s_skip;
    int skip_word = 0;
    if (threadIdx.x == 0) skip_word = *reinterpret_cast<volatile int*>(prm.status);

    // ---- work item -------------------------------------------------------------------
    // b: batch coordinate of the tensor maps; seq: sequence index (== b for a dense batch);
    // tok0 / len: first token and length of the sequence; row0: its first row among the mask rows
    // and scale blocks; m, n below count tiles inside the sequence.
    int b, hq, pr, seq, tok0 = 0, len = prm.L, row0 = VL ? 0 : prm.kv_off, n_rows = prm.T_m;
    int kblk0 = 0, n_kblk = prm.ks_blocks;   // first quantisation block of K of this sequence and their number
    // Order of the grid: (batch, head) rows in groups of head_group; inside a group the longest work items
    // first, and the heads of the group side by side for each item.  The host sizes the group so that its
    // K/V fits in L2 while its CTAs run; the grid then ends with the shortest items of the last group instead
    // of with the long items of the last head, and the SMs finish close together.
    const int kHeadGroup = prm.head_group;
    if constexpr (!VL) {
        const int n_pairs = (prm.T_m + 1) >> 1;
        const int n_bh = prm.B * prm.Hq;
        const int grp = blockIdx.x / (kHeadGroup * n_pairs);
        const int in_grp = blockIdx.x - grp * (kHeadGroup * n_pairs);
        const int g_heads = min(kHeadGroup, n_bh - grp * kHeadGroup);    // the last group may be smaller
        const int item = in_grp / g_heads;
        const int bh = grp * kHeadGroup + (in_grp - item * g_heads);
        pr = n_pairs - 1 - item;                            // longest rows first
        b = bh / prm.Hq;
        hq = bh - b * prm.Hq;
        seq = b;
    } else {
        const int grp = blockIdx.x / (kHeadGroup * prm.total_pairs);
        const int in_grp = blockIdx.x - grp * (kHeadGroup * prm.total_pairs);
        const int g_heads = min(kHeadGroup, prm.Hq - grp * kHeadGroup);
        const int item = in_grp / g_heads;                  // items are sorted by length on the host
        hq = grp * kHeadGroup + (in_grp - item * g_heads);
        seq = prm.vl_item_seq[item];
        pr = prm.vl_item_pair[item];
        b = 0;
        tok0 = prm.vl_tok[seq];
        len = prm.vl_tok[seq + 1] - tok0;
        row0 = prm.vl_tile[seq];
        n_rows = prm.vl_tile[seq + 1] - row0;
        kblk0 = prm.vl_blkk[seq];
        n_kblk = prm.vl_blkk[seq + 1] - kblk0;
    }
    constexpr bool varlen = VL;
    const int hk = hq / (prm.Hq / prm.Hk);
    // m: query-tile rows of this CTA (inside the sequence / the chunk); k: the key tile on their diagonal
    // (m + the chunk's offset in the context)
    const int kv_off = VL ? 0 : prm.kv_off;
    const int mA = 2 * pr, mB = 2 * pr + 1;
    const bool hasB = mB < n_rows;
    const int kA = mA + kv_off, kB = mB + kv_off;
    const int nkv = (hasB ? kB : kA) + 1;

    // ---- shared memory ------------------------------------------------------------------
    const uint32_t bar0 = sbase + C::kOffBars;
    auto bar_q = [&](int t) { return bar0 + 8u * t; };
    // Operands travel in bundles: bundle 0 = the K copies of key tile 0, bundle j + 1 = V_j and the K copies
    // of key tile j + 1 -- exactly what an MMA issuer needs for its iteration j.  One "landed" barrier and
    // one "consumed" barrier per bundle (kBundles of each, used round robin), whatever the number of
    // chunks, so an issuer pays one wait and one commit per key tile.
    auto bar_full = [&](int i) { return bar0 + 8u * (2 + i); };            // bundle i % kBundles landed
    auto bar_empty = [&](int i) { return bar0 + 8u * (2 + kRing + i); };   // ... consumed by every issuer
    // per query tile t and half h of the score tile: "S half ready", "P half ready"; per tile: "PV retired"
    auto bar_s = [&](int t, int h) { return bar0 + 8u * (2 + 2 * kRing + 2 * t + h); };
    auto bar_p = [&](int t, int h) { return bar0 + 8u * (6 + 2 * kRing + 2 * t + h); };
    auto bar_pv = [&](int t) { return bar0 + 8u * (10 + 2 * kRing + t); };   // the last-but-one PV of tile t
    auto bar_o = [&](int t) { return bar0 + 8u * (12 + 2 * kRing + t); };    // the last PV of tile t
    const uint32_t bar_drain = bar0 + 8u * (14 + 2 * kRing);
    // on-the-fly mode: "FP16 K tile of bundle i landed and its INT8 chunk is free" (producer -> quantiser),
    // "INT8 copy and scale of query tile t are in shared memory" (quantiser -> issuers, softmax groups)
    auto bar_raw = [&](int i) { return bar0 + 8u * (15 + 2 * kRing + i); };
    auto bar_q8 = [&](int t) { return bar0 + 8u * (15 + 2 * kRing + kBundles + t); };
    uint32_t* misc = reinterpret_cast<uint32_t*>(smem + C::kOffMisc);   // [0] tmem base, [1] abort
    // on-the-fly mode: delta_K of bundle n at otf_dk[n % (2 kBundles)] (a slot is rewritten only after
    // bundle n + kBundles has been consumed, i.e. long after both groups finished key tile n), delta_Q of
    // query tile t at otf_dq[t]
    volatile float* otf_dk = reinterpret_cast<volatile float*>(misc + 4);
    volatile float* otf_dq = reinterpret_cast<volatile float*>(misc + 12);
    uint32_t* sched_s = reinterpret_cast<uint32_t*>(smem + C::kOffWords);
    Ctx cx{reinterpret_cast<volatile int*>(&misc[1]), prm.status, prm.wait_limit_ns};

    // Set-up, shared out so that no thread does two things in a row: lane 0 of warp 0 initialises the two "Q landed"
    // barriers and starts the copies of the query tiles at once (they depend on nothing else and land while the rest
    // is set up), the other lanes of warp 0 initialise one barrier each, the warps behind it build the schedule
    // table, the first issuer warp allocates the tensor memory.
    if (warp == 0) {
        if (lane == 0) {
            ptx::mbar_init(bar_q(0), 1);
            ptx::mbar_init(bar_q(1), 1);
            misc[1] = 0;
        } else if (lane <= 3 * kBundles) {
            // on-the-fly mode: one more arrival per quantiser warp on "landed" (after it made its rows of the bundle's
            // INT8 tile, if there is one to make); "raw": K16 bytes expected + "INT8 chunk claimed"
            const int i = (lane - 1) / 3, which = (lane - 1) % 3;
            if (which == 0) ptx::mbar_init(bar_full(i), OTF ? 1 + kQuantWarps : 1);
            else if (which == 1) ptx::mbar_init(bar_empty(i), hasB ? 2 : 1);   // one arrival per MMA issuer
            else ptx::mbar_init(bar_raw(i), 2);
        } else if (lane <= 3 * kBundles + 2) {
            ptx::mbar_init(bar_q8(lane - 3 * kBundles - 1), kQuantWarps);
        } else if (lane <= 3 * kBundles + 6) {
            const int th = lane - 3 * kBundles - 3;
            ptx::mbar_init(bar_s(th >> 1, th & 1), 1);
        } else if (lane <= 3 * kBundles + 10) {
            const int th = lane - 3 * kBundles - 7;
            ptx::mbar_init(bar_p(th >> 1, th & 1), kSoftmaxWarps / 2 * 32);
        } else if (lane <= 3 * kBundles + 12) {
            ptx::mbar_init(bar_pv(lane - 3 * kBundles - 11), 1);
        } else if (lane <= 3 * kBundles + 14) {
            ptx::mbar_init(bar_o(lane - 3 * kBundles - 13), 1);
        } else if (lane == 3 * kBundles + 15) {
            ptx::mbar_init(bar_drain, hasB ? 2 : 1);
        }
        static_assert(3 * kBundles + 15 < 32, "one barrier per lane of warp 0");
        ptx::fence_mbar_init();
        if (lane == 0) {
            // The copies start whatever the status word says (its load is still on its way): a CTA that then finds
            // it has nothing to do waits for them before it leaves.
            for (int t = 0; t < (hasB ? 2 : 1); ++t) {
                const int m = t ? mB : mA;
                const uint32_t bytes = C::kQ16Tile + ((prm.has_int8 && !OTF) ? C::kQ8Tile : 0);
                ptx::mbar_arrive_expect_tx(bar_q(t), bytes);
                for (int c = 0; c < C::kHalves; ++c)
                    ptx::tma_load_4d(sbase + C::kOffQ16 + t * C::kQ16Tile + c * C::kQ16Slab, &tm_q16,
                                     bar_q(t), c * 64, tok0 + m * T, hq, b);
                if (prm.has_int8 && !OTF)
                    ptx::tma_load_4d(sbase + C::kOffQ8 + t * C::kQ8Tile, &tm_q8, bar_q(t), 0, tok0 + m * T, hq, b);
            }
            s_skip = skip_word;
        }
    }
    // Schedule table, one 4-bit entry per key tile j (Sec. 4.2 lookup done once per CTA):
    //   bit0 / bit1: tile A / tile B takes the INT8 route at key tile j  (R = (b >> floor(j/G)) & 1)
    //   bit2 / bit3: the FP16 / the INT8 copy of K_j has to be staged
    // A thread makes eight consecutive entries.  Their groups lie in at most two mask words per row: the four words
    // are loaded up front, so that the thread waits for one round trip, not for one per entry.
    for (int i = static_cast<int>(threadIdx.x) - 32; i >= 0 && i * 8 < nkv; i += static_cast<int>(blockDim.x) - 32) {
        const int j0 = i * 8, j_last = min(j0 + 7, nkv - 1);
        int g = 0, in_g = 0, w_lo = 0;
        uint32_t wa[2] = {0u, 0u}, wb[2] = {0u, 0u};
        if (prm.words != nullptr) {
            g = j0 / prm.G;
            in_g = j0 - g * prm.G;
            w_lo = g >> 5;
            const int w_hi = (j_last / prm.G) >> 5;
            const int nbi = (prm.nb == 1) ? 0 : b;
            const uint32_t* rowA = prm.words + ((static_cast<int64_t>(nbi) * prm.Hk + hk) * prm.mask_T_m + row0 + mA) * prm.W;
            wa[0] = rowA[w_lo];
            wa[1] = rowA[w_hi];
            if (hasB) { wb[0] = rowA[prm.W + w_lo]; wb[1] = rowA[prm.W + w_hi]; }
        }
        uint32_t packed = 0u;
        for (int jj = 0; jj < 8; ++jj) {
            const int j = j0 + jj;
            if (j > j_last) break;
            const bool hi = (g >> 5) != w_lo;              // (no mask words: all bits 0)
            uint32_t e = ((hi ? wa[1] : wa[0]) >> (g & 31)) & 1u;
            if (hasB) e |= (((hi ? wb[1] : wb[0]) >> (g & 31)) & 1u) << 1;
            if (++in_g == prm.G) { in_g = 0; ++g; }
            const bool useA = j <= kA;
            if ((useA && !(e & 1u)) || (hasB && !(e & 2u))) e |= 4u;
            if ((useA && (e & 1u)) || (hasB && (e & 2u))) e |= 8u;
            if (OTF && (e & 8u)) e |= 4u;   // the INT8 copy is made from the FP16 tile
            packed |= e << (4 * jj);
        }
        sched_s[i] = packed;
    }
    if (warp == kMmaWarp) {
        ptx::tmem_alloc(ptx::smem_u32(&misc[0]), C::kTmemCols);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = misc[0];
    if (s_skip != 0) {   // only the query tiles are in flight: let them land, give the tensor memory back and leave
        if (threadIdx.x == 0)
            for (int t = 0; t < (hasB ? 2 : 1); ++t)
                for (int it = 0; it < (1 << 20); ++it)
                    if (ptx::mbar_try_wait(bar_q(t), 0)) break;
        if (warp == kMmaWarp) ptx::tmem_dealloc(tmem_base, C::kTmemCols);
        return;
    }
    auto sched = [&](int j) -> uint32_t { return (sched_s[j >> 3] >> ((j & 7) * 4)) & 15u; };

    if (OTF && warp >= kQuantWarp0) {
        // ================================================================ on-chip quantiser (on-the-fly mode)
        // Four warps make the INT8 copies the tensor pipe reads: of a query tile before the first key tile it
        // routes to INT8, then of every key tile some query tile of the CTA routes to INT8.  A tile is 128
        // rows = one quantisation block (App. C): delta = max|x| / 127 over the tile, codes by the quantiser's
        // own arithmetic; each warp takes 32 rows, the four partial maxima meet in shared memory.  Source and
        // destination are the shared-memory images TMA would have written: FP16 tiles as D/64 slabs of
        // 128-byte rows, INT8 tiles as 128-byte rows, both with the 128-byte swizzle (16-byte chunk c of row r
        // sits at chunk c ^ (r & 7)).
        ptx::setmaxnreg_dec<OTF ? kRegsOtherOtf : kRegsOther>();
        static_assert(!OTF || (D == 128 && T == 128), "the on-chip quantiser handles 128 x 128 tiles");
        const int cw = warp - kQuantWarp0;
        volatile uint32_t* xch = misc + 2;   // partial maxima of the four warps: words 2, 3, 14, 15 of misc
        auto xch_slot = [&](int w) -> volatile uint32_t& { return xch[w < 2 ? w : w + 10]; };
        // `ok` turns false when a bounded wait ran out or the CTA is aborting; a warp then skips the work but
        // keeps meeting the others at the named barrier (every warp runs the same number of tiles).
        bool ok = true;
        auto quantise_tile = [&](uint32_t src_off, uint32_t dst_off) -> float {
            const uint8_t* src = smem + src_off;
            uint8_t* dst = smem + dst_off;
            constexpr int kRowsW = 128 / kQuantWarps, kVecW = kRowsW * 8;   // rows / 16-byte vectors per warp and slab
            uint32_t amax2 = 0u;
            if (ok) {
#pragma unroll
                for (int sl = 0; sl < C::kHalves; ++sl) {
                    uint4 v[kVecW / 32];   // eight loads in flight per lane
#pragma unroll
                    for (int u = 0; u < kVecW / 32; ++u)
                        v[u] = *reinterpret_cast<const uint4*>(src + (sl * 1024 + cw * kVecW + lane + 32 * u) * 16);
#pragma unroll
                    for (int u = 0; u < kVecW / 32; ++u)
                        amax2 = umax2(amax2, umax2(umax2(habs2_bits(v[u].x), habs2_bits(v[u].y)),
                                                   umax2(habs2_bits(v[u].z), habs2_bits(v[u].w))));
                }
            }
            uint32_t amax = max(amax2 & 0xffffu, amax2 >> 16);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) amax = max(amax, __shfl_xor_sync(0xffffffffu, amax, o));
            if (lane == 0) xch_slot(cw) = amax;
            ptx::bar_sync_named(kQuantBar, kQuantWarps * 32);
            amax = max(max(xch_slot(0), xch_slot(1)), max(xch_slot(2), xch_slot(3)));
            ptx::bar_sync_named(kQuantBar, kQuantWarps * 32);   // all have read: the slots may be written again
            const float amax_f = __half2float(__ushort_as_half(static_cast<unsigned short>(amax)));
            const float delta = __fdiv_rn(amax_f, 127.0f);
            if (!ok) return delta;
            if (amax == 0u) {   // zero block: delta = 0, every code 0
                for (int i = lane; i < kRowsW * D / 16; i += 32)
                    *reinterpret_cast<uint4*>(dst + cw * kRowsW * 128 + i * 16) = make_uint4(0u, 0u, 0u, 0u);
                return delta;
            }
            const float rdelta = __frcp_rn(delta);
#pragma unroll
            for (int sl = 0; sl < C::kHalves; ++sl) {
#pragma unroll
                for (int u0 = 0; u0 < kVecW / 32; u0 += 4) {   // four vectors in flight per lane
                    uint4 v[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u)
                        v[u] = *reinterpret_cast<const uint4*>(src + (sl * 1024 + cw * kVecW + lane + 32 * (u0 + u)) * 16);
                    uint2 qv[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) qv[u] = quant8_div(v[u], delta, rdelta);
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const int i = cw * kVecW + lane + 32 * (u0 + u);          // vector of the slab
                        const int r = i >> 3, cl = (i & 7) ^ (r & 7);             // row, logical chunk of the slab
                        // elements 64 sl + 8 cl .. + 7 of row r: byte column 64 sl + 8 cl of the INT8 row
                        const int c16 = sl * 4 + (cl >> 1);
                        *reinterpret_cast<uint2*>(dst + r * 128 + ((c16 ^ (r & 7)) << 4) + (cl & 1) * 8) = qv[u];
                    }
                }
            }
            return delta;
        };
        // hand-over to the async proxy (the tensor pipe reads shared memory through it), then one arrival per warp
        auto publish = [&](uint32_t bar) {
            ptx::fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(bar);
        };
        // The quantiser arrives on the "landed" barrier of EVERY bundle, with or without an INT8 tile to
        // make, so that the issuers (and with them the producer) can never run more than kBundles bundles
        // ahead of it and the phase it waits for is unambiguous.
        Ring ring;   // the producer's sequence of chunks
        uint32_t q8_made = 0u;
        for (int n = 0; n < nkv; ++n) {
            const uint32_t e = sched(n);
            uint32_t s16 = 0, s8 = 0;
            if (n >= 1) ring.take(C::kHalves);
            if (e & 4u) s16 = ring.take(C::kHalves);
            if (e & 8u) s8 = ring.take(1);
            for (int t = 0; t < 2; ++t) {
                if (!((e >> t) & 1u) || ((q8_made >> t) & 1u)) continue;
                if (ok) ok = wait_bar(cx, bar_q(t), 0, kRoleQuant, t, kBarQ);
                ok = __all_sync(0xffffffffu, ok);
                const float dq = quantise_tile(C::kOffQ16 + t * C::kQ16Tile, C::kOffQ8 + t * C::kQ8Tile);
                if (cw == 0 && lane == 0) otf_dq[t] = dq;
                publish(bar_q8(t));
                q8_made |= 1u << t;
            }
            if (ok) ok = wait_bar(cx, bar_raw(n % kBundles), (n / kBundles) & 1, kRoleQuant, n, kBarRaw);
            ok = __all_sync(0xffffffffu, ok);
            if (e & 8u) {
                const float dk = quantise_tile(C::kOffRing + s16 * C::kChunk, C::kOffRing + s8 * C::kChunk);
                if (cw == 0 && lane == 0) otf_dk[n % (2 * kBundles)] = dk;
            }
            publish(bar_full(n % kBundles));
        }
    } else if (warp >= kMmaWarp + 2 || (warp == kMmaWarp + 1 && !hasB)) {
        ptx::setmaxnreg_dec<OTF ? kRegsOtherOtf : kRegsOther>();   // idle warps of the third warpgroup
    } else if (warp == kProducerWarp) {
        // ================================================================ TMA producer
        ptx::setmaxnreg_dec<OTF ? kRegsOtherOtf : kRegsOther>();
        if (lane == 0) {
            ptx::tma_prefetch_desc(&tm_q16);
            ptx::tma_prefetch_desc(&tm_k16);
            ptx::tma_prefetch_desc(&tm_v16);
            if (prm.has_int8 && !OTF) {
                ptx::tma_prefetch_desc(&tm_q8);
                ptx::tma_prefetch_desc(&tm_k8);
            }
            // Chunks are taken from the ring in the order K16_j?, K8_j?, V_j (j = 0, 1, ...), the same
            // order in which the issuers count them.  A chunk may be refilled once the bundle that used it
            // last has been consumed; `last_user` remembers that bundle per chunk.
            Ring ring;
            bool ok = true;
            int consumed = 0;                       // bundles 0 .. consumed-1 are known to be consumed
            int last_user[kRing];
            for (int s = 0; s < kRing; ++s) last_user[s] = -1;
            auto wait_consumed = [&](int bundle, int j) {   // until `bundle` has been consumed
                while (ok && consumed <= bundle) {
                    if (!wait_bar(cx, bar_empty(consumed % kBundles), (consumed / kBundles) & 1, kRoleProducer, j, kBarRingEmpty)) ok = false;
                    ++consumed;
                }
            };
            int armed = 0;                          // bundles whose copies have been issued
            int dropped = -1;                       // (testing aid) the bundle that was left out
            for (int n = 0; n <= nkv && ok; ++n) {
                // bundle n: V of key tile n - 1 (n >= 1) and the K copies of key tile n (n < nkv)
                const uint32_t e = n < nkv ? sched(n) : 0u;
                const bool has_v = n >= 1;
                uint32_t s16 = 0, s8 = 0, sv = 0, bytes = 0, raw_bytes = 0;
                // On-the-fly mode: the FP16 K tile of a bundle with an INT8 tile to make is announced to the
                // quantiser (bar_raw), not to the issuers; the INT8 chunk is only claimed, not filled.
                const bool make8 = OTF && (e & 8u);
                // chunk order inside the sequence: ..., V_{n-1}, K16_n, K8_n, V_n, ...
                if (has_v) { sv = ring.take(C::kHalves); bytes += C::kHalves * C::kChunk; }
                if (e & 4u) { s16 = ring.take(C::kHalves); (make8 ? raw_bytes : bytes) += C::kHalves * C::kChunk; }
                if (e & 8u) { s8 = ring.take(1); if (!OTF) bytes += C::kK8Bytes; }
                if (bytes == 0u && raw_bytes == 0u) break;             // nothing after the last V
                if (n == prm.test_drop_bundle) {   // testing aid: this bundle never lands, an issuer's bounded wait runs out
                    dropped = n;
                    continue;
                }
                if (n >= kBundles) wait_consumed(n - kBundles, n);     // its barriers are free again
                // the barrier is armed for the whole bundle first; every operand is then copied as soon as
                // its own chunks are free, so a V tile does not wait for the room of the K tile behind it
                const uint32_t bar = bar_full(n % kBundles);
                if (bytes != 0u) ptx::mbar_arrive_expect_tx(bar, bytes);
                else ptx::mbar_arrive(bar);
                if (OTF) {
                    if (n == nkv)                          // the last bundle (V only) is not the quantiser's
                        for (int w = 0; w < kQuantWarps; ++w) ptx::mbar_arrive(bar);
                    if (n < nkv) {
                        if (raw_bytes != 0u) ptx::mbar_arrive_expect_tx(bar_raw(n % kBundles), raw_bytes);
                        else ptx::mbar_arrive(bar_raw(n % kBundles));
                    }
                }
                armed = n + 1;
                auto claim = [&](uint32_t slot, int chunks) {
                    for (int c = 0; c < chunks; ++c) {
                        if (last_user[slot + c] >= 0) wait_consumed(last_user[slot + c], n);
                        last_user[slot + c] = n;
                    }
                };
                if (has_v) {
                    claim(sv, C::kHalves);
                    if (!ok) break;
                    for (int c = 0; c < C::kHalves; ++c)
                        ptx::tma_load_4d(sbase + C::kOffRing + (sv + c) * C::kChunk, &tm_v16, bar, c * 64, tok0 + (n - 1) * T, hk, b);
                }
                if (e & 4u) {
                    claim(s16, C::kHalves);
                    if (!ok) break;
                    const uint32_t bar16 = make8 ? bar_raw(n % kBundles) : bar;
                    for (int c = 0; c < C::kHalves; ++c)
                        ptx::tma_load_4d(sbase + C::kOffRing + (s16 + c) * C::kChunk, &tm_k16, bar16, c * 64, tok0 + n * T, hk, b);
                }
                if (e & 8u) {
                    claim(s8, 1);
                    if (!ok) break;
                    if (!OTF) ptx::tma_load_4d(sbase + C::kOffRing + s8 * C::kChunk, &tm_k8, bar, 0, tok0 + n * T, hk, b);
                }
                // on-the-fly mode, second arrival: the INT8 chunk (if any) is the quantiser's to write
                if (OTF && n < nkv) ptx::mbar_arrive(bar_raw(n % kBundles));
            }
            if (!ok || *cx.abort_flag) {
                // let copies that are still in flight land before the CTA's memory is released
                for (int n = armed > kBundles ? armed - kBundles : 0; n < armed; ++n) {
                    if (n == dropped) continue;
                    for (int it = 0; it < (1 << 20); ++it)
                        if (ptx::mbar_try_wait(bar_full(n % kBundles), (n / kBundles) & 1)) break;
                    if (OTF && n < nkv)
                        for (int it = 0; it < (1 << 20); ++it)
                            if (ptx::mbar_try_wait(bar_raw(n % kBundles), (n / kBundles) & 1)) break;
                }
            }
        }
    } else if (warp == kMmaWarp || warp == kMmaWarp + 1) {
        // ================================================================ MMA issuers
        // One issuing warp per query tile (warp kMmaWarp: tile A, the next warp: tile B); the whole warp runs this
        // loop with warp-uniform values and stays converged, one elected lane issues each tcgen05 instruction.
        // Both issuers walk the same sequence of ring items; an item goes back to the producer when both have
        // committed it.
        ptx::setmaxnreg_dec<OTF ? kRegsOtherOtf : kRegsOther>();
        {
            const int t = warp - kMmaWarp;
            const int m_t = t ? kB : kA;       // last key tile of this issuer's query tile
            constexpr int TH = C::kTH;
            constexpr uint32_t kIdescQK16 = ptx::instr_desc(1, 0, 0, 0, C::kM, TH);
            constexpr uint32_t kIdescQK8 = ptx::instr_desc(2, 1, 0, 0, C::kM, TH);
            constexpr uint32_t kIdescPV = ptx::instr_desc(1, 0, 0, 1, C::kM, D);
            Ring ring;
            bool ok = true;
            bool q8_there = !OTF;   // on-the-fly mode: the INT8 copy of Q is waited for before its first use
            // Wait until bundle n has landed.  An issuer waits for EVERY bundle, also one whose data it
            // does not read: its arrival on the bundle's "consumed" barrier must not run a round of the
            // barriers ahead of the other issuer's, or two arrivals of one issuer would release it.
            auto acquire = [&](int n) {
                if (!ok) return;
                if (!wait_bar(cx, bar_full(n % kBundles), (n / kBundles) & 1, kRoleMma, n, kBarRingFull)) ok = false;
            };
            // Descriptor words that do not change: the high words, and the low words of the
            // resident Q operands.  One K step advances a K-major operand by 32 bytes inside its
            // swizzle atom (+2 in the low word) and the MN-major V operand by 16 keys = 2048 bytes.
            constexpr uint32_t kHi16 = ptx::desc_hi(1024, 2);
            constexpr uint32_t kHi8 = ptx::desc_hi(C::kI8Sbo, C::kI8Layout);
            const uint32_t ring_lo = ptx::desc_lo(sbase + C::kOffRing, 16);
            const uint32_t ring_lo_v = ptx::desc_lo(sbase + C::kOffRing, C::kChunk);
            constexpr uint32_t kChunkLo = C::kChunk >> 4;
            // Half h of S_t = Q_t K_j^T on the route of tile t: keys [h*TH, (h+1)*TH) of the key tile, i.e.
            // the rows of the K-major operand from byte h*TH*(row pitch) on (a whole number of swizzle atoms).
            auto issue_qk = [&](int t, int h, uint32_t int8_route, uint32_t s16, uint32_t s8) {
                const uint32_t d_tmem = tmem_base + t * C::kSCols + h * TH;
                if (int8_route) {
                    if constexpr (OTF) {
                        if (!q8_there) {
                            if (!wait_bar(cx, bar_q8(t), 0, kRoleMma, t, kBarQ8)) { ok = false; return; }
                            q8_there = true;
                        }
                    }
                    const uint32_t a_lo = ptx::desc_lo(sbase + C::kOffQ8 + t * C::kQ8Tile, 16);
                    const uint32_t b_lo = ring_lo + s8 * kChunkLo + ((h * TH * C::kI8RowBytes) >> 4);
                    ptx::mma_i8_ss<false>(d_tmem, a_lo, kHi8, b_lo, kHi8, kIdescQK8);
#pragma unroll
                    for (int k = 1; k < D / 32; ++k)
                        ptx::mma_i8_ss<true>(d_tmem, a_lo + 2 * k, kHi8, b_lo + 2 * k, kHi8, kIdescQK8);
                } else {
#pragma unroll
                    for (int c = 0; c < C::kHalves; ++c) {
                        const uint32_t a_lo = ptx::desc_lo(sbase + C::kOffQ16 + t * C::kQ16Tile + c * C::kQ16Slab, 16);
                        const uint32_t b_lo = ring_lo + (s16 + c) * kChunkLo + ((h * TH * 128) >> 4);
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            if (c == 0 && k == 0)
                                ptx::mma_f16_ss<false>(d_tmem, a_lo, kHi16, b_lo, kHi16, kIdescQK16);
                            else
                                ptx::mma_f16_ss<true>(d_tmem, a_lo + 2 * k, kHi16, b_lo + 2 * k, kHi16, kIdescQK16);
                        }
                    }
                }
            };
            // O_t (+)= P_t V_j over the keys of half h, with P in tensor memory (two FP16 per 32-bit
            // column, at the start of its own half of S_t)
            auto issue_pv = [&](int t, int h, uint32_t sv, uint32_t accumulate) {
                const uint32_t d_tmem = tmem_base + 2 * C::kSCols + t * C::kOCols;
                const uint32_t a_tmem = tmem_base + t * C::kSCols + h * TH;
                const uint32_t b_lo = ring_lo_v + sv * kChunkLo + h * (TH / 16) * 128;
                ptx::mma_f16_ts(d_tmem, a_tmem, b_lo, kHi16, kIdescPV, accumulate);
#pragma unroll
                for (int k = 1; k < TH / 16; ++k)
                    ptx::mma_f16_ts(d_tmem, a_tmem + k * 8, b_lo + k * 128, kHi16, kIdescPV, 1u);
            };

            if (!wait_bar(cx, bar_q(t), 0, kRoleMma, t, kBarQ)) ok = false;

            // slots of the K operands of the tile whose QK^T is issued next
            uint32_t e_next = sched(0), k16 = 0, k8 = 0;
            uint32_t r_next = (e_next >> t) & 1u;          // route of this tile at the next key tile
            if (e_next & 4u) k16 = ring.take(C::kHalves);
            if (e_next & 8u) k8 = ring.take(1);
            acquire(0);
            if (ok) {
                ptx::tc_fence_after_sync();
                for (int h = 0; h < 2; ++h) {
                    issue_qk(t, h, r_next, k16, k8);
                    ptx::mma_commit(bar_s(t, h));
                }
                ptx::mma_commit(bar_empty(0));
            }
            for (int j = 0; j < nkv && ok; ++j) {
                const bool mine = j <= m_t;            // tile A has no work at the last key tile of tile B
                const bool more = j + 1 <= m_t;
                const uint32_t sv = ring.take(C::kHalves);
                e_next = (j + 1 < nkv) ? sched(j + 1) : 0u;
                r_next = (e_next >> t) & 1u;
                if (e_next & 4u) k16 = ring.take(C::kHalves);
                if (e_next & 8u) k8 = ring.take(1);
                // operands of this iteration (bundle j + 1): wait for them now, off the P -> PV critical path
                acquire(j + 1);
                if (!ok) break;
                // Half steps: as soon as P of a half has arrived its PV is issued, and right behind it the
                // QK^T of the NEXT key tile into the same half of S_t -- the softmax group is meanwhile
                // working on the other half.
                if (mine) {
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        if (!wait_bar(cx, bar_p(t, h), j & 1, kRoleMma, j, kBarP)) { ok = false; break; }
                        ptx::tc_fence_after_sync();
                        issue_pv(t, h, sv, (j > 0 || h > 0) ? 1u : 0u);
                        if (j == m_t && h == 0) ptx::mma_commit(bar_pv(t));   // the last-but-one PV (a rescale in the last step waits for it)
                        if (j == m_t && h == 1) ptx::mma_commit(bar_o(t));
                        if (more) {
                            issue_qk(t, h, r_next, k16, k8);
                            ptx::mma_commit(bar_s(t, h));
                        }
                    }
                }
                if (!ok) break;
                ptx::mma_commit(bar_empty((j + 1) % kBundles));
            }
            // every MMA issued by this thread has retired before TMEM / shared memory go away
            ptx::mma_commit(bar_drain);
            wait_bar(cx, bar_drain, 0, kRoleMma, nkv, kBarDrain);
        }
    } else {
        // ================================================================ softmax warps
        ptx::setmaxnreg_inc<OTF ? kRegsSoftmaxOtf : kRegsSoftmax>();
        const int quarter = warp & 3, t = (warp >> 2) & 1, sub = warp >> 3;
        const int m_t = t ? mB : mA;           // query-tile row
        const int k_t = t ? kB : kA;           // its diagonal key tile
        if (t == 0 || hasB) {
            constexpr int TH = C::kTH;         // key columns per half step
            constexpr int NB = TH / 8;         // blocks of 8 columns per half step
            // This thread holds two columns (cq, cq + 1 of every block of 8) of the rows rw[0] and rw[1] = rw[0] + 8
            // of the tile; the four lanes of a quad share a row.
            const int cq = 2 * (lane & 3);
            const int rw[2] = {quarter * 32 + sub * 16 + (lane >> 2), quarter * 32 + sub * 16 + (lane >> 2) + 8};
            const uint32_t lane_base = tmem_base + (static_cast<uint32_t>(quarter * 32 + sub * 16) << 16);
            const uint32_t t_s = lane_base + t * C::kSCols;
            const uint32_t t_o = lane_base + 2 * C::kSCols + t * C::kOCols;
            // scales: dense [B,H,T_m] (unit stride over blocks), variable-length [blocks, H]
            const int64_t dk_step = varlen ? prm.Hk : 1;
            float dq = 0.f;
            const float* dk_row = nullptr;
            if constexpr (!OTF) {
                if (prm.has_int8) {
                    dq = varlen ? prm.q_scale[static_cast<int64_t>(row0 + m_t) * prm.Hq + hq]
                                : prm.q_scale[(static_cast<int64_t>(b) * prm.Hq + hq) * prm.T_m + m_t];
                    dk_row = varlen ? prm.k_scale + static_cast<int64_t>(kblk0) * prm.Hk + hk
                                    : prm.k_scale + (static_cast<int64_t>(b) * prm.Hk + hk) * prm.ks_blocks;
                }
            }
            // Shared online-softmax state (Sec. 3.1), log2 domain, per row: running maximum m (identical in the four
            // lanes of the row's quad) and this lane's part of the normaliser z.
            float m_run[2] = {-INFINITY, -INFINITY}, z[2] = {0.f, 0.f};
            bool ok = true;
            const int role = t ? kRoleSoftmaxB : kRoleSoftmaxA;
            bool dq_there = !OTF;   // on-the-fly mode: this tile's scale comes from the on-chip quantiser
            // delta_K of the quantisation block a step's keys lie in (App. C "Quantization Granularity": a block is a
            // key tile or, with the paper's BLK_K = BLOCK_N / 2, one half of it -- exactly one step); the next block's
            // scale is read ahead of its use.  A block beyond the end of a ragged sequence holds no legal key.
            const bool k_half = prm.k_half_blocks != 0;
            auto load_dk = [&](int blk) { return (prm.has_int8 && !OTF && blk < n_kblk) ? dk_row[blk * dk_step] : 0.f; };
            float dk_cur = 0.f, dk_next = load_dk(0);
            // VS: delta_V of the key tile (block = key tile) of the INT8 value cache the FP16 V operand was made from
            const float* dv_row = nullptr;
            if constexpr (VS) dv_row = prm.v_scale + (static_cast<int64_t>(b) * prm.Hk + hk) * prm.vs_blocks;
            float dv = 1.f;
            float a = prm.scale_log2;
            uint32_t int8_route = 0u;
            const int n_steps = 2 * (k_t + 1);
            // One step = one half (TH key columns) of a score tile: while the warps of this tile work on one half of
            // S_t, the tensor pipe runs the PV of the previous half and the QK^T of the next one into the other
            // half.  u = 2*j + h.
            for (int u = 0; u < n_steps; ++u) {
                const int j = u >> 1, h = u & 1;
                if (h == 0) int8_route = (sched(j) >> t) & 1u;
                if constexpr (VS) { if (h == 0) dv = dv_row[j]; }
                if (h == 0 || k_half) {
                    dk_cur = dk_next;
                    dk_next = load_dk(k_half ? u + 1 : j + 1);
                    a = prm.scale_log2;
                    if (int8_route) {
                        a *= dq * dk_cur;
                        if (a == 0.f) a = 1.f;   // a zero block: every accumulator is 0 already
                    }
                }
                const uint32_t t_sh = t_s + h * TH;
                ok = wait_bar(cx, bar_s(t, h), j & 1, role, j, kBarS);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                ptx::tc_fence_after_sync();
                uint32_t s[4 * NB];
                if constexpr (NB == 8) ptx::tmem_ld16x256_x8(t_sh, s);
                else ptx::tmem_ld16x256_x4(t_sh, s);
                if constexpr (OTF) {
                    // the key tile's scale was written by the quantiser before the issuer could start the
                    // MMAs whose result has just been seen
                    if (h == 0 && int8_route) {
                        if (!dq_there) {
                            ok = wait_bar(cx, bar_q8(t), 0, role, m_t, kBarQ8);   // long over: S of an INT8 tile is there
                            ok = __all_sync(0xffffffffu, ok);
                            if (!ok) break;
                            dq = otf_dq[t];
                            dq_there = true;
                        }
                        a = prm.scale_log2 * (dq * otf_dk[j % (2 * kBundles)]);   // same rounding order as with scales from memory
                        if (a == 0.f) a = 1.f;
                    }
                }

                // P = 2^(a*raw - m) is rounded to FP16, one pair per register.
                const bool diag = (j == k_t);
                bool redo = diag || u == 0 || DBG;
                bool stored = false;      // P of the one-pass form has been sent to tensor memory
                float alpha[2] = {1.f, 1.f}, sum[2] = {0.f, 0.f};
                bool grow = false;
                uint32_t p[2 * NB];
                ptx::tmem_wait_ld_dep(s);     // ties the registers to the wait: no use of them moves above it
                if (!redo) {
                    if (!int8_route) {
                        const float addend[2] = {-m_run[0], -m_run[1]};
                        softmax_step_fast<NB, kFp32, VS>(s, a, addend, p, sum, dv);
                    } else if (a * kInt8Bias <= kFoldLimit) {
                        // one explicit FMA: every instantiation of the kernel rounds the addend the same way
                        const float addend[2] = {-__fmaf_rn(a, kInt8Bias, m_run[0]), -__fmaf_rn(a, kInt8Bias, m_run[1])};
                        softmax_step_fast<NB, kInt8Folded, VS>(s, a, addend, p, sum, dv);
                    } else {
                        const float addend[2] = {-m_run[0], -m_run[1]};
                        softmax_step_fast<NB, kInt8Exact, VS>(s, a, addend, p, sum, dv);
                    }
                    // The store of P goes out before the vote, so that the vote's latency hides behind it; a rejected
                    // step stores again below, after this store has been waited for.
                    if constexpr (NB == 8) ptx::tmem_st16x128_x8(t_sh, p);
                    else ptx::tmem_st16x128_x4(t_sh, p);
                    stored = true;
                    redo = __any_sync(0xffffffffu, !(sum[0] <= exp2f(kAccept) && sum[1] <= exp2f(kAccept)));   // also true for a NaN
                }
                if (redo) {
                    // Generic two-pass form: the very first step, the diagonal tile, steps that move the maximum, and
                    // every step in debug mode.
                    if constexpr (DBG) {   // debug mode: raw accumulators of the requested tiles
                        int idx = -1;
                        if (lane == 0) {
                            for (int e = 0; e < prm.dbg_n; ++e) {
                                const int32_t* qd = prm.dbg_tiles + 4 * e;
                                if (qd[0] == seq && qd[1] == hq && qd[2] == m_t && qd[3] == j) { idx = e; break; }
                            }
                        }
                        idx = __shfl_sync(0xffffffffu, idx, 0);
                        if (idx >= 0) {
#pragma unroll
                            for (int k = 0; k < 2; ++k) {
                                if (rw[k] >= T) continue;
                                int32_t* dst = prm.dbg_raw + (static_cast<int64_t>(idx) * T + rw[k]) * T + h * TH + cq;
#pragma unroll
                                for (int i = 0; i < NB; ++i)
                                    *reinterpret_cast<uint2*>(dst + 8 * i) = make_uint2(s[4 * i + 2 * k], s[4 * i + 2 * k + 1]);
                            }
                            if (rw[0] == 0 && cq == 0) prm.dbg_kind[idx] = static_cast<uint8_t>(int8_route);
                        }
                    }
                    // Common FP32 score domain (App. C), causal legality on the diagonal tile (App. B:
                    // enforced kernel-side, independent of R), row maximum, then the exponentials.
                    float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
                    for (int i = 0; i < NB; ++i) {
#pragma unroll
                        for (int k = 0; k < 2; ++k) {
#pragma unroll
                            for (int e = 0; e < 2; ++e) {
                                const int c = 4 * i + 2 * k + e;
                                float v = int8_route ? __int2float_rn(static_cast<int>(s[c])) : __uint_as_float(s[c]);
                                if (diag && h * TH + 8 * i + cq + e > rw[k]) v = -INFINITY;
                                s[c] = __float_as_uint(v);
                                mx[k] = fmaxf(mx[k], v);
                            }
                        }
                    }
#pragma unroll
                    for (int k = 0; k < 2; ++k) {
                        const float m_step = quad_max(mx[k] * a);     // a >= 0, so max(a*raw) = a*max(raw)
                        if (m_step > m_run[k] + kMove) {
                            alpha[k] = fast_exp2(m_run[k] - (m_step + kMargin));
                            m_run[k] = m_step + kMargin;
                            z[k] *= alpha[k];
                            grow = true;
                        }
                    }
                    const float2 a2 = make_float2(a, a);
                    float2 acc[2] = {{0.f, 0.f}, {0.f, 0.f}};
#pragma unroll
                    for (int i = 0; i < NB; ++i) {
#pragma unroll
                        for (int k = 0; k < 2; ++k) {
                            const float2 t2 = __ffma2_rn(make_float2(__uint_as_float(s[4 * i + 2 * k]), __uint_as_float(s[4 * i + 2 * k + 1])),
                                                         a2, make_float2(-m_run[k], -m_run[k]));
                            const float2 pp = make_float2(fast_exp2(t2.x), fast_exp2(t2.y));
                            acc[k] = __fadd2_rn(acc[k], pp);
                            if constexpr (VS) p[2 * i + k] = pack_half2(pp.x * dv, pp.y * dv);
                            else p[2 * i + k] = pack_half2(pp.x, pp.y);
                        }
                    }
                    sum[0] = acc[0].x + acc[0].y;
                    sum[1] = acc[1].x + acc[1].y;
                }
                z[0] += sum[0];
                z[1] += sum[1];

                if (redo && u > 0 && __any_sync(0xffffffffu, grow)) {
                    // O~ *= alpha.  The PV of the previous step may still be accumulating into O~: wait
                    // until it has retired (the PV of this step is not issued before P arrives below).
                    // The issuer puts the QK^T of step u+1 behind PV(u-1) and commits both to "S(u+1) ready",
                    // so that barrier -- the one the next step waits on anyway -- says PV(u-1) has retired; the
                    // last step has no successor and waits on the commit behind the last-but-one PV instead.
                    if (u + 1 < n_steps) ok = wait_bar(cx, bar_s(t, h ^ 1), ((u + 1) >> 1) & 1, role, j, kBarS);
                    else ok = wait_bar(cx, bar_pv(t), 0, role, j, kBarPV);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                    ptx::tc_fence_after_sync();
#pragma unroll 1                     // (rare: kept small, see DBG above)
                    for (int c = 0; c < D / 32; ++c) {
                        uint32_t o[16];
                        ptx::tmem_ld16x256_x4(t_o + c * 32, o);
                        ptx::tmem_wait_ld_dep(o);
#pragma unroll
                        for (int e = 0; e < 16; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha[(e >> 1) & 1]);
                        ptx::tmem_st16x256_x4(t_o + c * 32, o);
                    }
                }
                if (redo) {
                    if (stored) ptx::tmem_wait_st();      // (the rejected one-pass store, before the same columns are stored again)
                    if constexpr (NB == 8) ptx::tmem_st16x128_x8(t_sh, p);
                    else ptx::tmem_st16x128_x4(t_sh, p);
                }
                ptx::tmem_wait_st();
                ptx::tc_fence_before_sync();
                ptx::mbar_arrive(bar_p(t, h));
            }

            if (ok) {
                ok = wait_bar(cx, bar_o(t), 0, role, k_t + 1, kBarO);
                ok = __all_sync(0xffffffffu, ok);
            }
            if (ok) {
                // Finalise (Sec. 3.1): O = O~ / z in FP16; LSE = m + ln z.
                ptx::tc_fence_after_sync();
#pragma unroll
                for (int k = 0; k < 2; ++k) {
                    const float z_row = quad_sum(z[k]);
                    const int i_loc = m_t * T + rw[k];                            // row inside the sequence
                    const int64_t i_glob = static_cast<int64_t>(tok0) + i_loc;    // row on the token axis
                    const bool row_valid = rw[k] < T && i_loc < len;
                    z[k] = row_valid ? 1.f / z_row : 0.f;
                    if (row_valid && cq == 0 && prm.lse != nullptr)
                        prm.lse[(static_cast<int64_t>(b) * prm.Hq + hq) * prm.L + i_glob] = (m_run[k] + log2f(z_row)) * kLn2;
                }
                __half* dst0 = prm.out + b * prm.os[0] + hq * prm.os[1] + (static_cast<int64_t>(tok0) + m_t * T) * prm.os[2] + cq;
#pragma unroll
                for (int c = 0; c < D / 32; ++c) {
                    uint32_t o[16];
                    ptx::tmem_ld16x256_x4(t_o + c * 32, o);
                    ptx::tmem_wait_ld_dep(o);
#pragma unroll
                    for (int k = 0; k < 2; ++k) {
                        if (z[k] == 0.f) continue;     // a row beyond the sequence (or the 64-row tile): not written
                        __half* dst = dst0 + rw[k] * prm.os[2] + c * 32;
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const __half2 hv = __floats2half2_rn(__uint_as_float(o[4 * i + 2 * k]) * z[k],
                                                                 __uint_as_float(o[4 * i + 2 * k + 1]) * z[k]);
                            *reinterpret_cast<__half2*>(dst + 8 * i) = hv;
                        }
                    }
                }
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
                float* lse, void* workspace, const tilemix_debug_t* dbg, cudaStream_t stream,
                const VarlenDev* vl, int total_pairs, const float* v_scale) {
    using C = Cfg<D, T>;
    EncodeTiledFn enc = nullptr;
    int rc = get_encoder(&enc);
    if (rc) return rc;
    const bool otf = (g.flags & TILEMIX_QUANT_ON_THE_FLY) != 0;
    if (otf && (vl != nullptr || !(D == 128 && T == 128) || g.blk_k != g.tile_n)) return TILEMIX_ERR_UNSUPPORTED;
    if (v_scale != nullptr && (otf || vl != nullptr)) return TILEMIX_ERR_UNSUPPORTED;   // value-cache scales: dense, quantise-once
    const bool has8 = !(g.flags & TILEMIX_FORCE_FP16) && (q8 != nullptr || otf);
    CUtensorMap tq, tk, tv, tq8, tk8;
    if ((rc = encode_map(enc, &tq, q, 2, g.d, g.L, g.Hq, g.B, g.qs, 64, C::kM, CU_TENSOR_MAP_SWIZZLE_128B))) return rc;
    if ((rc = encode_map(enc, &tk, k, 2, g.d, g.Lk, g.Hk, g.B, g.ks, 64, T, CU_TENSOR_MAP_SWIZZLE_128B))) return rc;
    if ((rc = encode_map(enc, &tv, v, 2, g.d, g.Lk, g.Hk, g.B, g.vs, 64, T, CU_TENSOR_MAP_SWIZZLE_128B))) return rc;
    if (has8 && !otf) {
        const CUtensorMapSwizzle sw8 = (D == 128) ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B;
        const int64_t dq[3] = {static_cast<int64_t>(g.Hq) * g.L * g.d, static_cast<int64_t>(g.L) * g.d, g.d};
        const int64_t dk[3] = {static_cast<int64_t>(g.Hk) * g.Lk * g.d, static_cast<int64_t>(g.Lk) * g.d, g.d};
        if ((rc = encode_map(enc, &tq8, q8, 1, g.d, g.L, g.Hq, g.B, dq, D, C::kM, sw8))) return rc;
        if ((rc = encode_map(enc, &tk8, k8, 1, g.d, g.Lk, g.Hk, g.B, dk, D, T, sw8))) return rc;
    } else {
        tq8 = tq;
        tk8 = tk;
    }
    Params prm{};
    prm.B = g.B; prm.Hq = g.Hq; prm.Hk = g.Hk; prm.L = g.L; prm.G = g.G; prm.T_m = g.T_m; prm.W = g.W;
    prm.kv_off = g.kv_off; prm.mask_T_m = g.mask_T_m; prm.ks_blocks = g.ks_blocks;
    prm.k_half_blocks = (g.blk_k * 2 == g.tile_n) ? 1 : 0;
    prm.wait_limit_ns = g_wait_limit_ns.load();
    prm.test_drop_bundle = g_test_drop.load() == 1 ? 1 : -1;
    {
        // heads per group: as many as keep the group's K and V (FP16; adjacent query heads of a GQA group share
        // theirs) within 72 MB of the 126 MB L2
        const int64_t kv_bytes = 2 * static_cast<int64_t>(g.Lk) * g.d * 2;
        const int rep = g.Hq / g.Hk;
        int hg = 1;
        while (hg < kMaxHeadGroup && ceil_div(2 * hg, rep) * kv_bytes <= (72ll << 20)) hg *= 2;
        prm.head_group = hg;
    }
    prm.nb = g.nb;
    prm.has_int8 = has8 ? 1 : 0;
    prm.scale_log2 = g.scale * kLog2e;
    prm.q_scale = qs; prm.k_scale = ks;
    prm.v_scale = v_scale; prm.vs_blocks = g.T_n;
    prm.words = has8 ? words : nullptr;
    prm.out = static_cast<__half*>(out);
    prm.os[0] = g.os[0]; prm.os[1] = g.os[1]; prm.os[2] = g.os[2];
    prm.lse = lse;
    prm.status = static_cast<int*>(workspace);
    if (vl != nullptr) {
        prm.vl_tok = vl->tok; prm.vl_tile = vl->tile; prm.vl_blkk = vl->blkk; prm.vl_item_seq = vl->item_seq; prm.vl_item_pair = vl->item_pair;
        prm.n_seqs = vl->n; prm.total_pairs = total_pairs;
    }
    if (dbg != nullptr && dbg->n_tiles > 0) {
        prm.dbg_tiles = dbg->tiles; prm.dbg_n = dbg->n_tiles; prm.dbg_raw = dbg->raw; prm.dbg_kind = dbg->kind;
    }
    cudaError_t e = cudaMemsetAsync(workspace, 0, kWorkspaceClearBytes, stream);
    if (e != cudaSuccess) return static_cast<int>(e);
    const bool dbg_on = prm.dbg_n > 0;
    auto kernel = vl ? (dbg_on ? attention_kernel<D, T, true, false, false, true> : attention_kernel<D, T, true, false>)
                     : (dbg_on ? attention_kernel<D, T, false, false, false, true> : attention_kernel<D, T, false, false>);
    if constexpr (D == 128 && T == 128) {
        if (otf) kernel = dbg_on ? attention_kernel<D, T, false, true, false, true> : attention_kernel<D, T, false, true>;
    }
    if (v_scale != nullptr) {
        if (dbg_on) return TILEMIX_ERR_UNSUPPORTED;     // (the chunk against an INT8 value cache has no debug instance)
        kernel = attention_kernel<D, T, false, false, true>;
    }
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemAlloc);
    if (e != cudaSuccess) return static_cast<int>(e);
    const int64_t ctas = vl ? static_cast<int64_t>(g.Hq) * total_pairs
                            : static_cast<int64_t>(g.B) * g.Hq * ((g.T_m + 1) / 2);
    if (ctas == 0) return TILEMIX_OK;   // only zero-length sequences
    if (ctas > 0x7fffffffLL) return static_cast<int>(cudaErrorInvalidConfiguration);
    // The register split inside the kernel (setmaxnreg) assumes what the block is launched with; a build that
    // gave the kernel fewer registers must not run (an increase beyond the block's allotment never returns).
    cudaFuncAttributes fa;
    e = cudaFuncGetAttributes(&fa, kernel);
    if (e != cudaSuccess) return static_cast<int>(e);
    if (fa.numRegs < (otf ? kLaunchRegsOtf : kLaunchRegs)) return TILEMIX_ERR_UNSUPPORTED;
    kernel<<<static_cast<unsigned>(ctas), otf ? kThreadsOtf : kThreads, C::kSmemAlloc, stream>>>(prm, tq, tk, tv, tq8, tk8);
    g_launch_count.fetch_add(1);
    return static_cast<int>(cudaGetLastError());
}

}  // namespace

int launch_attention(const Geometry& g, const void* q, const void* k, const void* v, const int8_t* q8,
                     const int8_t* k8, const float* qs, const float* ks, const uint32_t* words, void* out,
                     float* lse, void* workspace, const tilemix_debug_t* dbg, cudaStream_t stream,
                     const VarlenDev* vl, int total_pairs, const float* v_scale) {
    if (g.d == 128 && g.tile_m == 128)
        return launch_impl<128, 128>(g, q, k, v, q8, k8, qs, ks, words, out, lse, workspace, dbg, stream, vl,
                                     total_pairs, v_scale);
    if (g.d == 64 && g.tile_m == 64)
        return launch_impl<64, 64>(g, q, k, v, q8, k8, qs, ks, words, out, lse, workspace, dbg, stream, vl,
                                   total_pairs, v_scale);
    return TILEMIX_ERR_UNSUPPORTED;
}

}  // namespace tilemix

// ---------------------------------------------------------------------------------- no-allocation entry
// Scratch for callers that cannot allocate device memory: the status/workspace record of
// tilemix_attention_fwd, held in a fixed array that lives in the library image.
namespace tilemix {
namespace {

constexpr size_t kStaticWorkspaceBytes = 4096;
static __device__ __align__(256) unsigned char g_static_workspace[kStaticWorkspaceBytes];

constexpr int kMaxDevices = 64;
std::atomic<void*> g_static_workspace_addr[kMaxDevices];

// Device address of g_static_workspace on the current device.  In host code the array's name is only
// a handle, not a device address, so the address is asked for once per device (that device current).
int static_workspace(void** out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return static_cast<int>(e);
    if (dev < 0 || dev >= kMaxDevices) return TILEMIX_ERR_UNSUPPORTED;
    void* ptr = g_static_workspace_addr[dev].load(std::memory_order_acquire);
    if (ptr == nullptr) {
        e = cudaGetSymbolAddress(&ptr, g_static_workspace);
        if (e != cudaSuccess) return static_cast<int>(e);
        if (ptr == nullptr) return static_cast<int>(cudaErrorInvalidSymbol);
        g_static_workspace_addr[dev].store(ptr, std::memory_order_release);   // same value from any thread
    }
    *out = ptr;
    return TILEMIX_OK;
}

}  // namespace
}  // namespace tilemix

extern "C" int tilemix_attention_fwd_noalloc(const tilemix_problem_t* p, const void* q_f16, const void* k_f16,
                                             const void* v_f16, const int8_t* q_i8, const int8_t* k_i8,
                                             const float* q_scale, const float* k_scale,
                                             const uint32_t* mask_words, void* out_f16, float* lse,
                                             const tilemix_debug_t* dbg, void** workspace_out, void* stream) {
    using namespace tilemix;
    if (p == nullptr || !q_f16 || !k_f16 || !v_f16 || !out_f16) return TILEMIX_ERR_NULL;
    Geometry g;
    const int bad = resolve(p, &g);      // the codes tilemix_attention_fwd returns for the same problem
    if (bad) return bad;
    if (tilemix_workspace_size(p) > kStaticWorkspaceBytes) return TILEMIX_ERR_WORKSPACE;   // beyond the fixed scratch
    void* ws = nullptr;
    const int rc = static_workspace(&ws);
    if (rc != TILEMIX_OK) return rc;
    if (workspace_out != nullptr) *workspace_out = ws;
    return tilemix_attention_fwd(p, q_f16, k_f16, v_f16, q_i8, k_i8, q_scale, k_scale, mask_words, out_f16, lse,
                                 ws, kStaticWorkspaceBytes, dbg, stream);
}
