// Launch parameters of the decode step, shared by its two kernels (decode.cu: warp-level MMAs, every supported
// shape; decode_umma.cu: tcgen05 MMAs, head dimension 128 with 128-key tiles).  Not part of the public ABI.
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace tilemix {

struct DecodeParams {
    int B, Hq, Hk, max_len, G, nb, W, n_splits, n_blk;
    int tile_n;      // tokens per scale block and per routing key tile (a multiple of the kernel's chunk)
    int n_parts;     // partial results per query head in the workspace
    // tcgen05 form, automatic split count: n_ctas CTAs (one wave) are shared out over the n_rows = B * Hk rows by
    // their cost, at most split_cap to a row (n_parts = 2 * split_cap); n_splits is then not used
    int balanced, n_rows, n_ctas, split_cap;
    float scale_log2;
    const __half* q;
    const __half* k16;
    const int8_t* k8;
    const float* k_scale;
    const int8_t* v8;
    const float* v_scale;
    const uint32_t* words;
    const int32_t* cache_len;       // clamped copy in the workspace (written by the prepare kernel)
    const int32_t* cache_len_raw;   // the caller's array
    float* o_part;   // [B, Hq, n_parts, D]
    float* m_part;   // [B, Hq, n_parts]
    float* z_part;
    int8_t* q8_out;
    float* qs_out;
    int* status;     // 4 ints at the start of the workspace (same record as the attention kernel's)
    unsigned long long wait_limit_ns;   // limit of the bounded waits
    int test_drop_tile;                 // testing aid: the producer leaves out the copies of this tile of every split (-1: none)
};

// The tcgen05 form of the step for head_dim 128, tile_n 128 (R = Hq / Hk in {1, 2, 4, 8}): enqueues the kernel
// that writes (m, z, O~) of every split to the workspace; the caller launches the merge.  Returns a cudaError_t
// or a TILEMIX_ERR_* code.
int launch_decode_umma(int R, const DecodeParams& prm, cudaStream_t stream);

}  // namespace tilemix
