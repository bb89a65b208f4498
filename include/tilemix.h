/*
 * tilemix.h -- C ABI of the TileMix hot path for NVIDIA B200 (sm_100a).
 *
 * TileMix (arxiv 2608.17336) is causal prefill attention in which every group of G adjacent
 * key tiles of a query-tile row is routed, by one bit of a packed mask, to an FP16 or an
 * INT8 QK^T score computation; both routes feed one shared online-softmax state, and the PV
 * product stays FP16.  This library holds the three steps of that path:
 *
 *   tilemix_quantize_qk        blockwise symmetric INT8 quantiser for Q and K
 *   tilemix_pack_routing_mask  routing map R -> packed words (+ coverage counters)
 *   tilemix_attention_fwd      the fused mixed-precision attention kernel
 *   tilemix_prefill_host       the three steps on HOST buffers (copies included)
 *
 * Conventions shared by every entry point
 *   - Unless a parameter says "host", every pointer is a DEVICE pointer on the current CUDA
 *     device; the caller owns every buffer; outputs are fully overwritten.
 *   - Work is enqueued on `stream` (a cudaStream_t passed as void*; NULL = default stream).
 *     No entry point allocates device memory or synchronises, except where stated.
 *   - Return value: 0 = TILEMIX_OK; negative = a contract violation found on the host
 *     BEFORE anything was launched; positive = the cudaError_t / CUresult of a failed
 *     launch or tensor-map encode.  Nothing is printed, nothing throws.
 *   - Indices are 0-based.  T_m = ceil(L/tile_m), T_n = ceil(L/tile_n),
 *     T_mask = ceil(L/(G*tile_n)), W = ceil(T_mask/32).
 */
#ifndef TILEMIX_H_
#define TILEMIX_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define TILEMIX_OK 0
#define TILEMIX_ERR_NULL (-1)        /* a required pointer is NULL                          */
#define TILEMIX_ERR_SHAPE (-2)       /* non-positive size, heads_q % heads_kv != 0, ...      */
#define TILEMIX_ERR_UNSUPPORTED (-3) /* tile/head_dim combination or device not supported    */
#define TILEMIX_ERR_ALIGN (-4)       /* base pointer or stride not 16-byte aligned           */
#define TILEMIX_ERR_WORKSPACE (-5)   /* workspace / arena smaller than required              */
#define TILEMIX_ERR_DEVICE_TIMEOUT (-6) /* reported by tilemix_read_status only              */

/* flags of tilemix_problem_t */
#define TILEMIX_FORCE_FP16 1u /* ignore the mask: every tile takes the FP16 route; the INT8
                                 operands, scales and mask may then be NULL               */
#define TILEMIX_QUANT_ON_THE_FLY 2u /* tilemix_attention_fwd, _chunk and tilemix_prefill_host (App. D, the "fused on-the-fly" operand
                                      mode): q_i8, k_i8, q_scale and k_scale are not read and may be NULL;
                                      the kernel makes the INT8 tiles and their scales in shared memory from
                                      the FP16 tiles, for the key tiles routed to INT8 only, with the
                                      arithmetic of tilemix_quantize_qk -- same result, bit for bit, no INT8
                                      scratch in device memory.  128x128 tiles with head_dim 128.          */
/* pack_flags of tilemix_pack_routing_mask */
#define TILEMIX_PIN_DIAGONAL_FP16 1u

/* Shape of one attention call, in the paper's notation (Sec. 3.1, Sec. 4.1): B, H_q, H_k,
 * L = L_q = L_k, d, BLOCK_M x BLOCK_N score tiles, g key tiles per routing bit.
 * Strides are in elements, for (batch, head, token); the head_dim axis is contiguous.  A
 * stride triple of all zeros means dense [B, H, L, d].  INT8 operands, scales, mask words
 * and the routing map are always dense. */
typedef struct tilemix_problem {
    int32_t batch, heads_q, heads_kv, seqlen, head_dim;
    int32_t tile_m, tile_n;           /* routing / quantisation tile; supported: 64x64 with
                                         head_dim 64, 128x128 with head_dim 128             */
    int32_t group;                    /* G >= 1                                              */
    int32_t quant_blk_q, quant_blk_k; /* rows per scale; 0 = tile_m / tile_n                 */
    int32_t mask_batch;               /* 1 = one mask shared by the batch, or == batch       */
    uint32_t flags;
    float softmax_scale;              /* <= 0 means 1/sqrt(head_dim)                         */
    int32_t reserved;
    int64_t q_stride[3], k_stride[3], v_stride[3], o_stride[3];
} tilemix_problem_t;

/* Debug request for tilemix_attention_fwd: the raw score accumulators of the listed tiles. */
typedef struct tilemix_debug {
    const int32_t* tiles; /* [n_tiles, 4] = (b, h_q, m, n), legal tiles (n <= m)            */
    int32_t n_tiles;
    int32_t* raw;         /* [n_tiles, tile_m, tile_n]: INT8-routed tile: the INT32
                             accumulator Q8_m K8_n^T exactly as the tensor core produced it
                             (before scaling and masking; rows/cols beyond L are 0);
                             FP16-routed tile: the bit pattern of the FP32 accumulator      */
    uint8_t* kind;        /* [n_tiles]: 1 = INT32 written, 0 = FP32 bits written             */
} tilemix_debug_t;

/* Blockwise symmetric INT8 quantisation of Q and K (App. C, "Blockwise INT8 Quantization"
 * and "Quantization Granularity"): for every block r of quant_blk rows of one head,
 * delta = max|x| / 127 and xhat = round(x / delta) in {-127..127}, computed in FP32 with
 * IEEE division and round-half-to-even; a zero block gives delta = 0, xhat = 0; a tail block
 * takes its maximum over the rows that exist.
 *   q_f16 [B,Hq,L,d], k_f16 [B,Hk,L,d]  FP16, strided per the problem
 *   q_i8, k_i8                          INT8, dense, same shapes
 *   q_scale [B,Hq,ceil(L/blk_q)], k_scale [B,Hk,ceil(L/blk_k)]  FP32
 * Either operand may be skipped by passing all three of its pointers as NULL. */
int tilemix_quantize_qk(const tilemix_problem_t* p, const void* q_f16, const void* k_f16,
                        int8_t* q_i8, int8_t* k_i8, float* q_scale, float* k_scale,
                        void* stream);

/* Packed routing words (Sec. 4.2, "Bitmask packing"): for every (nb, h_k, m) the word row
 * b = sum_g R[g] * 2^g, stored as W little-endian uint32 words (group g -> word g>>5,
 * bit g&31; for T_mask <= 64 this is the paper's one 64-bit word).  1 = INT8, 0 = FP16.
 * Bits of groups with no legal (query, key) pair, of pad positions >= T_mask and -- with
 * TILEMIX_PIN_DIAGONAL_FP16 -- of groups holding a key tile that straddles the diagonal are
 * written as 0.
 *   route      uint8 [nb, Hk, T_m, T_mask], non-zero = INT8
 *   mask_words uint32 [nb, Hk, T_m, W]
 *   counts     nullable uint64 [nb, Hk, 2] = {legal groups, INT8-routed legal groups}
 *              (App. B, "Coverage Accounting") */
int tilemix_pack_routing_mask(const tilemix_problem_t* p, const uint8_t* route,
                              uint32_t pack_flags, uint32_t* mask_words, uint64_t* counts,
                              void* stream);

/* The fused kernel (Sec. 4.1 loops, Sec. 4.3 "Tile-group dispatch", App. C): for every query
 * tile m it streams key tiles n <= m; bit floor(n/G) of row (h_k, m) selects
 *   S = Q_m K_n^T / sqrt(d)                                   (FP16 route, bit 0) or
 *   S = delta_Q[m] delta_K[n] (Q8_m K8_n^T) / sqrt(d)         (INT8 route, bit 1),
 * both update one FP32 online-softmax state (Sec. 3.1), P is rounded to FP16 for the PV
 * product, and O = O~/z is written as FP16.  h_k = h_q / (H_q/H_k).
 *   lse        nullable float [B,Hq,L]: max + ln(sum) of the scaled scores of each row
 *   workspace  >= tilemix_workspace_size(p) bytes, 16-byte aligned; its first 16 bytes are a
 *              status record (see tilemix_read_status) which this call clears on the stream
 *   dbg        nullable; see tilemix_debug_t
 * Requires quant_blk_q == tile_m; quant_blk_k == tile_n or tile_n / 2 (App. C "Quantization Granularity": the
 * paper's BLK_Q = 128, BLK_K = 64 with 128 x 128 tiles; one delta_K then serves each half of a key tile; not in the
 * on-the-fly operand mode, which quantises whole key tiles); 16-byte aligned bases and strides; a device of compute
 * capability 10.0. */
int tilemix_attention_fwd(const tilemix_problem_t* p, const void* q_f16, const void* k_f16,
                          const void* v_f16, const int8_t* q_i8, const int8_t* k_i8,
                          const float* q_scale, const float* k_scale,
                          const uint32_t* mask_words, void* out_f16, float* lse,
                          void* workspace, size_t workspace_bytes, const tilemix_debug_t* dbg,
                          void* stream);

/* Chunked prefill: the queries are the LAST p->seqlen tokens of a context of kv_len tokens whose keys
 * and values are all present (earlier chunks, a prefix cache); query i attends to keys
 * 0 .. kv_len - p->seqlen + i.  The result equals the corresponding rows of tilemix_attention_fwd over
 * the whole context, bit for bit.  kv_len - p->seqlen must be a multiple of the tile (so that query
 * tiles, quantisation blocks and mask rows line up with the context's).
 *   q_f16, q_i8, out_f16   [B,Hq,seqlen,d];  q_scale [B,Hq,ceil(seqlen/tile)];  lse [B,Hq,seqlen]
 *   k_f16, v_f16, k_i8     [B,Hk,kv_len,d] (dense strides are taken with kv_len);  k_scale [B,Hk,ceil(kv_len/tile)]
 *   mask_words             the words of the WHOLE context, uint32 [nb,Hk,ceil(kv_len/tile),W(kv_len)], as
 *                          tilemix_pack_routing_mask writes them for seqlen = kv_len; the chunk reads its rows
 * Everything else as for tilemix_attention_fwd (the workspace needs 4096 bytes). */
int tilemix_attention_fwd_chunk(const tilemix_problem_t* p, int32_t kv_len, const void* q_f16,
                                const void* k_f16, const void* v_f16, const int8_t* q_i8,
                                const int8_t* k_i8, const float* q_scale, const float* k_scale,
                                const uint32_t* mask_words, void* out_f16, float* lse, void* workspace,
                                size_t workspace_bytes, const tilemix_debug_t* dbg, void* stream);

/* Chunked prefill against an INT8 VALUE cache (App. C, "Additional Execution Interfaces": cached V8 is
 * converted to FP16 on chip and its block scale is folded into the probability tile before the PV product).
 * As tilemix_attention_fwd_chunk, but the values are INT8 with one FP32 scale per block of tile_n tokens
 * (the cache layout of tilemix_decode_int8kv):
 *   o_i = sum_j softmax(s_i)_j * delta_V[blk(j)] * v8_j  over the keys j <= kv_len - p->seqlen + i,
 * computed as P' V with P'_ij = FP16(softmax numerator * delta_V[blk(j)]) and V the exact FP16 image of V8,
 * FP32 accumulation (the row sum is of the unscaled numerators).  The scores are those of
 * tilemix_attention_fwd_chunk (routed FP16 / INT8 QK^T).  With kv_len == p->seqlen it is a prefill that writes
 * against a freshly quantised value cache; with p->seqlen == tile it is one tile of new queries.
 *   v_i8     INT8 [B,Hk,kv_len,d], dense;  v_scale FP32 [B,Hk,ceil(kv_len/tile_n)]
 *   workspace  tilemix_chunk_v8_workspace_size(p, kv_len) bytes: the status record and an FP16 image of the value
 *            cache.  The conversion is a kernel of its own in front of the attention kernel (two launches): the
 *            image passes through device memory once per call (3 bytes per cached element, ~1 % of the attention
 *            kernel's time at a 4096-token chunk of a 32K context) instead of being made tile by tile in shared
 *            memory; the arithmetic is the same.
 * Dense batches, quantise-once operands (no TILEMIX_QUANT_ON_THE_FLY); the v_stride of `p` is ignored.
 * Everything else as for tilemix_attention_fwd_chunk. */
size_t tilemix_chunk_v8_workspace_size(const tilemix_problem_t* p, int32_t kv_len);
int tilemix_attention_fwd_chunk_v8(const tilemix_problem_t* p, int32_t kv_len, const void* q_f16,
                                   const void* k_f16, const int8_t* v_i8, const float* v_scale,
                                   const int8_t* q_i8, const int8_t* k_i8, const float* q_scale,
                                   const float* k_scale, const uint32_t* mask_words, void* out_f16,
                                   float* lse, void* workspace, size_t workspace_bytes, void* stream);

/* Same computation as tilemix_attention_fwd for callers that cannot hand it a workspace because
 * they cannot allocate device memory at all: a process whose whole GPU memory was claimed at
 * start-up by another allocator or memory pool (any later cudaMalloc fails), or a code path that
 * must not synchronise the device, which cudaMalloc and cudaFree do.  (The paper has no
 * counterpart; this is a convenience of this library.)  The workspace is a fixed array of
 * 4096 bytes inside the library image; every GPU on which the library is used holds its own copy
 * until the process exits.  This call allocates nothing -- no cudaMalloc, no cudaFree, no
 * allocating library routine -- and all inputs and outputs are still the caller's.
 *   - A problem whose tilemix_workspace_size() exceeds 4096 bytes is rejected with
 *     TILEMIX_ERR_WORKSPACE before anything is launched.
 *   - The first call on each device looks up the device address of the array (a host-side query, that
 *     device must be current); make that first call before any stream capture begins.
 *   - Every call on a device shares the one array, which keeps what the last call left in it; this
 *     call clears the status record on `stream` before the kernel.  Two calls that overlap on the
 *     GPU (different streams, or different host threads on different streams) race on the status
 *     record: serialise them, or use tilemix_attention_fwd with one workspace per stream.
 *   workspace_out  nullable; receives the device address of the array, e.g. for tilemix_read_status
 * All other parameters, the return values and the error behaviour are those of
 * tilemix_attention_fwd. */
int tilemix_attention_fwd_noalloc(const tilemix_problem_t* p, const void* q_f16, const void* k_f16,
                                  const void* v_f16, const int8_t* q_i8, const int8_t* k_i8,
                                  const float* q_scale, const float* k_scale,
                                  const uint32_t* mask_words, void* out_f16, float* lse,
                                  const tilemix_debug_t* dbg, void** workspace_out, void* stream);

/* Whole path on HOST buffers: copies Q, K, V and the routing map to the device arena,
 * quantises, packs, runs the fused kernel and copies O back (use pinned host memory for the
 * copies to be asynchronous).  The batch -- for a single sequence, its KV heads -- is cut into up
 * to 8 chunks that are pipelined: host->device copies and device->host copies run on two helper
 * streams of the library (created on the first call on a device, kept until exit) while the
 * kernels run on `stream`.  All of it is ordered after the work `stream` held on entry, and
 * `stream` is made to wait for the last copy, so synchronising `stream` completes the call.
 *   q_host,k_host,v_host  host FP16, dense [B,H,L,d];  route_host host uint8 [nb,Hk,T_m,T_mask]
 *   out_host              host FP16, dense [B,Hq,L,d]
 *   arena                 device scratch of >= tilemix_arena_size(p) bytes, 256-byte aligned
 * Host threads: the helper streams and events are one set per device, and a call holds a per-device lock of
 * the library while it enqueues, so calls from several host threads on one device (each with its own arena,
 * output buffer and stream) are safe and are enqueued one whole call after the other; their copies share the
 * two helper streams and therefore run in that order.  The call does not synchronise anything. */
int tilemix_prefill_host(const tilemix_problem_t* p, const void* q_host, const void* k_host,
                         const void* v_host, const uint8_t* route_host, uint32_t pack_flags,
                         void* out_host, void* arena, size_t arena_bytes, void* stream);

/* ---- variable-length batches (Sec. 4.1, "grouped-query attention and variable-length batching";
 * App. C, scale shapes for variable-length batches) -------------------------------------------
 * n_seqs sequences are packed back to back along the token axis with no padding.  Sequence s
 * owns tokens [cu_seqlens[s], cu_seqlens[s+1]) and is an independent causal attention problem
 * with its own tiles: T_m(s) = ceil(L_s/tile_m) query-tile rows, blocks of the quantiser that
 * restart at the sequence's first token, and its own mask rows.  Prefix sums over the sequences
 * (built by the library from cu_seqlens) place each sequence's tile rows and scale blocks:
 *   tile_off[s] = sum_{t<s} ceil(L_t/tile_m),  blkq_off / blkk_off likewise with the quantiser
 *   block sizes.
 * The problem struct describes the packed batch: batch = 1, seqlen = total tokens
 * (= cu_seqlens[n_seqs]), mask_batch = 1.  An all-zero stride triple means the flattened
 * token-major layout [total, H, d] (head stride d, token stride H*d); any other layout is given
 * by explicit strides (the batch stride is ignored).  Layouts of the derived buffers:
 *   q_i8, k_i8   INT8 [H, total, d] (head-major, dense)
 *   q_scale      FP32 [sum_s ceil(L_s/blk_q), Hq]    (block-major, as in App. C)
 *   k_scale      FP32 [sum_s ceil(L_s/blk_k), Hk]
 *   route        uint8 [Hk, sum_s T_m(s), T_mask_max], T_mask_max = ceil(max_seqlen/(G*tile_n));
 *                row tile_off[s]+m is query-tile row m of sequence s; entries beyond the
 *                sequence's own T_mask(s) are ignored
 *   mask_words   uint32 [Hk, sum_s T_m(s), W], W = ceil(T_mask_max/32)
 *   lse          FP32 [Hq, total]
 * Zero-length sequences are allowed and produce nothing. */
typedef struct tilemix_varlen {
    int32_t n_seqs;            /* >= 1                                                         */
    int32_t max_seqlen;        /* 0 = take the longest sequence of cu_seqlens; otherwise it must
                                  be >= the longest sequence (fixes T_mask_max and W)          */
    const int32_t* cu_seqlens; /* HOST pointer, n_seqs + 1 entries, non-decreasing,
                                  cu_seqlens[0] = 0, cu_seqlens[n_seqs] = p->seqlen; read
                                  before the call returns                                      */
} tilemix_varlen_t;

/* Derived sizes of a variable-length batch, out = {total tokens, sum T_m, sum blocks of Q,
 * sum blocks of K, T_mask_max, W, longest sequence}.  Returns TILEMIX_OK or a negative error. */
int tilemix_varlen_counts(const tilemix_problem_t* p, const tilemix_varlen_t* vl, int64_t out[7]);
/* The three calls below copy their prefix-sum tables from a host buffer of the call (pageable memory) to the
 * workspace with cudaMemcpyAsync: do not call them while `stream` is being captured into a CUDA graph (the graph
 * would keep a pointer to memory that is gone when the call returns), and expect the copy to be staged by the
 * driver like any copy from pageable memory.
 * Bytes of `workspace` the three calls below need (0 on invalid arguments): the 4096-byte
 * status area of tilemix_attention_fwd followed by the prefix-sum tables and the attention
 * kernel's work list (two int32 per pair of query tiles).  Every call copies
 * the tables into its workspace on `stream`, so one workspace may serve all three calls in
 * stream order, and the tables of the last call stay there. */
size_t tilemix_varlen_workspace_size(const tilemix_problem_t* p, const tilemix_varlen_t* vl);
/* tilemix_quantize_qk over a variable-length batch: blocks never cross a sequence boundary;
 * the tail block of every sequence takes its maximum over the rows that exist. */
int tilemix_quantize_qk_varlen(const tilemix_problem_t* p, const tilemix_varlen_t* vl,
                               const void* q_f16, const void* k_f16, int8_t* q_i8, int8_t* k_i8,
                               float* q_scale, float* k_scale, void* workspace,
                               size_t workspace_bytes, void* stream);
/* tilemix_pack_routing_mask over a variable-length batch; legality of a group is judged with
 * the length of the row's own sequence.  counts: nullable uint64 [Hk, 2]. */
int tilemix_pack_routing_mask_varlen(const tilemix_problem_t* p, const tilemix_varlen_t* vl,
                                     const uint8_t* route, uint32_t pack_flags,
                                     uint32_t* mask_words, uint64_t* counts, void* workspace,
                                     size_t workspace_bytes, void* stream);
/* tilemix_attention_fwd over a variable-length batch: every sequence is attended causally on
 * its own; no score crosses a sequence boundary.  dbg tiles are (sequence, h_q, m, n) with m, n
 * counted inside the sequence.  Requires every sequence to have at most 2048 key tiles. */
int tilemix_attention_fwd_varlen(const tilemix_problem_t* p, const tilemix_varlen_t* vl,
                                 const void* q_f16, const void* k_f16, const void* v_f16,
                                 const int8_t* q_i8, const int8_t* k_i8, const float* q_scale,
                                 const float* k_scale, const uint32_t* mask_words, void* out_f16,
                                 float* lse, void* workspace, size_t workspace_bytes,
                                 const tilemix_debug_t* dbg, void* stream);

/* ---- decode step over an INT8 key/value cache (App. C, "Additional Execution Interfaces") ------
 * One new query token per sequence attends to the first cache_len[b] keys of a cache that holds,
 * per KV head, K in FP16 and in INT8 and V in INT8, with one FP32 scale per block of tile_n tokens
 * (the blockwise quantiser above; V is quantised like K, e.g. by passing it to
 * tilemix_quantize_qk as the K operand).  Bit g of the mask row of (nb, h_k) routes the keys
 * [g*G*tile_n, (g+1)*G*tile_n):
 *   bit 1:  s_j = delta_q delta_K[blk(j)] (q8 . k8_j) * scale   -- INT8 dot products, INT32 sums;
 *           q8, delta_q = the blockwise quantiser applied to the query row, done in the kernel
 *   bit 0:  s_j = (q . k16_j) * scale                           -- FP16 inputs, FP32 sums
 * and  o = sum_j softmax(s)_j * delta_V[blk(j)] * v8_j : V8 is converted on chip and its block
 * scale is folded into the probability before the PV sum (FP32 accumulation), O is written as FP16.
 * Only the K copy a group is routed to is read, so the bytes per cached token are 2*d (INT8 route)
 * or 3*d (FP16 route).  The keys are split over n_splits CTAs per (b, h_k); every CTA serves the
 * H_q/H_k query heads of its KV head; a second kernel merges the partial results.
 * Supported: head_dim 64 or 128, tile_n 64 or 128, H_q/H_k in {1, 2, 4, 8}.  Two forms of the step
 * kernel: head_dim 128 with tile_n 128 runs on tcgen05 MMAs (keys are the rows of S^T = K Q^T, one CTA
 * per SM, one wave of CTAs when n_splits is left to the library, two partial results per split); the
 * other shapes run on warp-level MMAs (the query rows fill a 16-row tile).  Same arithmetic, same
 * results up to the order of the FP32 sums. */
typedef struct tilemix_decode {
    int32_t batch, heads_q, heads_kv, head_dim;
    int32_t max_len;       /* token capacity of the caches (their token stride)             */
    int32_t tile_n, group; /* key tile = scale block; G key tiles per routing bit           */
    int32_t mask_batch;    /* 1 = one mask row per KV head shared by the batch, or == batch */
    int32_t n_splits;      /* CTAs per (b, h_k); 0 = chosen by the library, the same for every (b, h_k);
                            * -1 = chosen by the kernel per (b, h_k), for batches of unequal cache lengths: in
                            * the tcgen05 form with batch * heads_kv <= 148 the CTAs of one wave are shared out
                            * so that the largest number of cache bytes a CTA reads is as small as it can be
                            * (a row gets clamp(ceil(bytes / tau), 1, cap) CTAs for the smallest tau that fits
                            * the wave); elsewhere -1 means 0 */
    float softmax_scale;   /* <= 0 means 1/sqrt(head_dim)                                   */
} tilemix_decode_t;

/* Bytes of `workspace` for tilemix_decode_int8kv: the status record, the clamped copy of the cache lengths
 * and the partial results of the splits (0 on an invalid problem). */
size_t tilemix_decode_workspace_size(const tilemix_decode_t* p);
/*   q_f16      FP16 [B, Hq, d]
 *   k_f16      FP16 [B, Hk, max_len, d]   (may be NULL if every group inside the cache lengths is
 *                                          INT8-routed; a 0 bit there is then found by the kernel before it
 *                                          reads anything: no access is made, the status record of the
 *                                          workspace reads TILEMIX_ERR_NULL and the outputs are undefined)
 *   k_i8, v_i8 INT8 [B, Hk, max_len, d];  k_scale, v_scale FP32 [B, Hk, ceil(max_len/tile_n)]
 *   mask_words uint32 [nb, Hk, W], W = ceil(ceil(max_len/(G*tile_n))/32); NULL = all FP16
 *   cache_len  int32 [B] on the DEVICE, 0 <= cache_len[b] <= max_len (values outside are clamped to that
 *              range by the kernel); a sequence of length 0
 *              gets an all-zero output row and lse = -inf
 *   out_f16    FP16 [B, Hq, d];  lse nullable FP32 [B, Hq]
 *   q_i8_out / q_scale_out  nullable INT8 [B, Hq, d] / FP32 [B, Hq]: the quantised query the
 *              kernel used (for checking)
 * Three kernels are enqueued on `stream` (preparation of the lengths and the status record, the step over the
 * splits, the merge; in the tcgen05 form the last two are programmatic dependent launches, so that their set-up
 * overlaps the kernel before them).  Errors as for the other entry points; tilemix_read_status on the workspace reports what the
 * kernel itself found (a bounded wait that ran out, or the missing FP16 cache above). */
int tilemix_decode_int8kv(const tilemix_decode_t* p, const void* q_f16, const void* k_f16,
                          const int8_t* k_i8, const float* k_scale, const int8_t* v_i8,
                          const float* v_scale, const uint32_t* mask_words,
                          const int32_t* cache_len, void* out_f16, float* lse, int8_t* q_i8_out,
                          float* q_scale_out, void* workspace, size_t workspace_bytes,
                          void* stream);

/* W = ceil(ceil(L / (G*tile_n)) / 32); <= 0 on invalid arguments. */
int tilemix_mask_words_per_row(int seqlen, int tile_n, int group);
/* Bytes of `workspace` needed by tilemix_attention_fwd (0 on an invalid problem). */
size_t tilemix_workspace_size(const tilemix_problem_t* p);
/* Bytes of the quantize-once scratch of App. D's accounting: INT8 Q and K, their FP32
 * scales and the packed words (0 on an invalid problem). */
size_t tilemix_scratch_bytes(const tilemix_problem_t* p);
/* Bytes of `arena` needed by tilemix_prefill_host (0 on an invalid problem). */
size_t tilemix_arena_size(const tilemix_problem_t* p);
/* Synchronises `stream`, then copies the 4-word status record of the last
 * tilemix_attention_fwd on that workspace to host `out`: {code, role, tile index, barrier}.
 * Returns out[0]: TILEMIX_OK or TILEMIX_ERR_DEVICE_TIMEOUT (a bounded wait inside the kernel
 * ran out; the outputs of that call are then undefined). */
int tilemix_read_status(const void* workspace, int32_t out[4], void* stream);
const char* tilemix_status_string(int code);
/* Number of kernels this library has launched since it was loaded (all entry points). */
uint64_t tilemix_launch_count(void);
/* Measurement aid (the paper has no counterpart): the issue rate of the tensor pipe for the instruction shape the
 * fused kernel's full score tile uses, the denominator of its roofline measured on the same GPU in the same run.  One
 * CTA per SM issues n_mma back-to-back tcgen05.mma M128 N128 (K16 kind::f16 if int8 == 0, K32 kind::i8 otherwise)
 * with both operands in shared memory, into one accumulator, and returns when they have retired.  Time the call with
 * events on `stream`: operations = *n_ctas * n_mma * 2*128*128*K.  workspace: >= 16 device bytes, receives a status
 * record (tilemix_read_status).  Returns TILEMIX_OK, TILEMIX_ERR_SHAPE or a CUDA error. */
int tilemix_tensor_peak_probe(int int8, int n_mma, int* n_ctas, void* workspace, void* stream);
/* Testing aid for the bounded waits (the paper has no counterpart).  Every wait inside the kernels is bounded: when
 * one runs out the CTA records {TILEMIX_ERR_DEVICE_TIMEOUT, role, tile, barrier} in the status record, every role
 * stops, what is in flight is waited for, and the kernel RETURNS -- nothing faults and nothing spins for ever.  This
 * switch, process-wide and read at launch time, lets a test see that path run:
 *   which = 1  the attention kernel's producer leaves out the copies of operand bundle 1 (V of key tile 0 and K of key
 *              tile 1) of every CTA, so an MMA issuer's wait for that bundle runs out after wait_limit_ns
 *   which = 2  the decode step's producer leaves out the second tile of every split
 *   which = 3  the streaming quantiser's producer leaves out the second block of every CTA; the quantiser has no
 *              status record: a CTA that gives up writes NaN into the scales of the blocks it did not finish
 *   which = 0  normal operation, limit back to the default of 2 s (wait_limit_ns is ignored)
 * Returns TILEMIX_OK or TILEMIX_ERR_SHAPE. */
int tilemix_test_drop_copy(int which, uint64_t wait_limit_ns);

#ifdef __cplusplus
}
#endif
#endif /* TILEMIX_H_ */
