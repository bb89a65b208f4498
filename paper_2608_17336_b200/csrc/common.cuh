// Internal helpers shared by the translation units of libtilemix (host-side validation,
// resolved geometry, launch counting).  Not part of the public ABI.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "tilemix.h"

namespace tilemix {

extern std::atomic<uint64_t> g_launch_count;

inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }

// Problem with defaults resolved and derived tile counts.
struct Geometry {
    int B, Hq, Hk, L, d;
    int tile_m, tile_n, G;
    int blk_q, blk_k;
    int nb;                 // mask batch
    int T_m, T_n, T_mask, W;
    float scale;            // softmax scale (natural-log domain)
    uint32_t flags;
    int64_t qs[3], ks[3], vs[3], os[3];   // element strides (batch, head, token)
};

// Fills `g`; returns TILEMIX_OK or a negative error.  Checks sizes only (no pointers).
int resolve(const tilemix_problem_t* p, Geometry* g);

inline bool aligned16(const void* ptr) { return (reinterpret_cast<uintptr_t>(ptr) & 15u) == 0; }

// Launchers implemented in the .cu files (all enqueue on `stream`, return cudaError_t as int).
int launch_quantize(const void* x, const int64_t stride[3], int B, int H, int L, int d, int blk,
                    int8_t* out, float* scale, cudaStream_t stream);
int launch_pack(const Geometry& g, const uint8_t* route, uint32_t pack_flags, uint32_t* words,
                unsigned long long* counts, cudaStream_t stream);
int launch_attention(const Geometry& g, const void* q, const void* k, const void* v,
                     const int8_t* q8, const int8_t* k8, const float* qs, const float* ks,
                     const uint32_t* words, void* out, float* lse, void* workspace,
                     const tilemix_debug_t* dbg, cudaStream_t stream);

}  // namespace tilemix
