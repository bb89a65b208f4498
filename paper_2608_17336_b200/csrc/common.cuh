// Internal helpers shared by the translation units of libtilemix (host-side validation,
// resolved geometry, launch counting).  Not part of the public ABI.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>
#include <vector>

#include "tilemix.h"

namespace tilemix {

extern std::atomic<uint64_t> g_launch_count;

// Testing aid (tilemix_test_drop_copy): which producer leaves out one copy, and the limit of the bounded waits.
constexpr uint64_t kDefaultWaitLimitNs = 2000000000ull;
extern std::atomic<int> g_test_drop;                 // 0 none, 1 attention kernel, 2 decode step, 3 streaming quantiser
extern std::atomic<uint64_t> g_wait_limit_ns;

inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }

// Problem with defaults resolved and derived tile counts.
struct Geometry {
    int B, Hq, Hk, L, d;
    int tile_m, tile_n, G;
    int blk_q, blk_k;
    int nb;                 // mask batch
    int T_m, T_n, T_mask, W;
    // Chunked prefill (queries = the last L tokens of an Lk-token context): K/V length, the chunk's
    // first tile row in the context, rows per head of the mask words, blocks per head of k_scale.
    // For a plain prefill: Lk = L, kv_off = 0, mask_T_m = T_m, ks_blocks = T_n.
    int Lk, kv_off, mask_T_m, ks_blocks;
    float scale;            // softmax scale (natural-log domain)
    uint32_t flags;
    int64_t qs[3], ks[3], vs[3], os[3];   // element strides (batch, head, token)
};

// Fills `g`; returns TILEMIX_OK or a negative error.  Checks sizes only (no pointers).
int resolve(const tilemix_problem_t* p, Geometry* g);

// Variable-length batch: host-side prefix sums over the sequences and their device copy.
struct VarlenTable {
    int n = 0;                 // sequences
    int max_len = 0;           // longest sequence (or the caller's bound)
    int total_tiles = 0, total_pairs = 0, total_blk_q = 0, total_blk_k = 0;
    // four arrays of n + 1 entries (tok, tile, blkq, blkk), then two of total_pairs entries: the
    // attention kernel's work items (sequence, pair of query tiles), longest first
    std::vector<int32_t> tab;
};
struct VarlenDev {
    const int32_t* tok = nullptr;    // first token of sequence s (cu_seqlens)
    const int32_t* tile = nullptr;   // query-tile rows before sequence s
    const int32_t* blkq = nullptr;   // quantiser blocks of Q before sequence s
    const int32_t* blkk = nullptr;   // quantiser blocks of K before sequence s
    const int32_t* item_seq = nullptr;   // work item -> sequence
    const int32_t* item_pair = nullptr;  // work item -> pair of query tiles (2p, 2p+1) of that sequence
    int n = 0;
};
constexpr size_t kStatusAreaBytes = 4096;   // status record, timers, trace: start of every workspace

// Fills `g` for the packed batch (B = 1, L = total tokens, T_m = sum of tile rows, T_mask / W of the
// longest sequence, T_n = key tiles of the longest sequence) and the prefix sums.
int resolve_varlen(const tilemix_problem_t* p, const tilemix_varlen_t* vl, Geometry* g, VarlenTable* t);
// Copies the tables behind the status area of `workspace` on `stream` and points `dev` at them.
int upload_varlen(const VarlenTable& t, void* workspace, cudaStream_t stream, VarlenDev* dev);

#ifdef __CUDACC__
// Sequence s with off[s] <= x < off[s+1] (off non-decreasing, off[0] <= x < off[n]).
__device__ __forceinline__ int find_seq(const int32_t* __restrict__ off, int n, int x) {
    int lo = 0, hi = n;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (off[mid] <= x) lo = mid; else hi = mid;
    }
    return lo;
}
#endif

inline bool aligned16(const void* ptr) { return (reinterpret_cast<uintptr_t>(ptr) & 15u) == 0; }

// Launchers implemented in the .cu files (all enqueue on `stream`, return cudaError_t as int).
// `vl` (nullable) switches a launcher to the variable-length layouts; `blk_off` / `total_blk` are the
// block prefix sums of the operand being quantised.
int launch_quantize(const void* x, const int64_t stride[3], int B, int H, int L, int d, int blk,
                    int8_t* out, float* scale, cudaStream_t stream, const VarlenDev* vl = nullptr,
                    const int32_t* blk_off = nullptr, int total_blk = 0);
int launch_quantize_pair(const void* q, const int64_t qstride[3], int Hq, int blk_q, int8_t* q8, float* qs,
                         const void* k, const int64_t kstride[3], int Hk, int blk_k, int8_t* k8, float* ks,
                         int B, int L, int d, cudaStream_t stream);
int launch_pack(const Geometry& g, const uint8_t* route, uint32_t pack_flags, uint32_t* words,
                unsigned long long* counts, cudaStream_t stream, const VarlenDev* vl = nullptr);
int launch_attention(const Geometry& g, const void* q, const void* k, const void* v,
                     const int8_t* q8, const int8_t* k8, const float* qs, const float* ks,
                     const uint32_t* words, void* out, float* lse, void* workspace,
                     const tilemix_debug_t* dbg, cudaStream_t stream, const VarlenDev* vl = nullptr,
                     int total_pairs = 0, const float* v_scale = nullptr);
// `v_scale` (nullable; dense batches only): `v` is the exact FP16 image of an INT8 value cache and the block scale
// of key tile j is folded into the probabilities of that tile before they are rounded to FP16.

}  // namespace tilemix
