/*
 * TileMix CPU oracle -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain, slow, obviously-correct CPU statement of what the TileMix hot path computes
 * (causal prefill attention whose QK^T score tiles are routed, per packed bit, to an FP16
 * or an INT8 score formula).  It shares no code, header, table or helper with the CUDA
 * path; only tests, the smoke check and the bench's cpu_baseline leg may call it.
 *
 * The method is exact up to the stated quantisation: the online-softmax recurrence of
 * Sec. 3.1 reaches plain softmax, and routing only chooses which of the two score
 * formulas of Sec. 4.3 / App. C a tile uses.  So the oracle is the *definition* written
 * out -- no key tiles in the loop structure, no running maximum, no FP16 probabilities:
 *
 *   quantise (App. C "Blockwise INT8 Quantization")      oracle_quantize
 *   pack     (Sec. 4.2 "Bitmask packing", App. B)          oracle_pack
 *   scores -> full softmax -> PV  (Sec. 3.1, Sec. 4.3)     oracle_attention_rows
 *   raw INT32 score tile (App. C "INT8 Score Computation") oracle_int32_tile
 *
 * Arithmetic: FP32 where the paper fixes it (the quantiser), exact int32 for the INT8 dot
 * products, IEEE double for everything else.  Compile with -O2 -ffp-contract=off and no
 * fast-math flags; OpenMP is used only over independent query rows / blocks.
 *
 * Layouts (all dense, row-major, innermost index last):
 *   q16/k16/v16  uint16 (IEEE binary16 bit patterns)  [B, H, L, d]
 *   q8/k8        int8                                  [B, H, L, d]
 *   q_scale      float [B, Hq, ceil(L/blk_q)],  k_scale float [B, Hk, ceil(L/blk_k)]
 *   words        uint32 [nb, Hk, T_m, W],  W = ceil(T_mask/32), T_mask = ceil(L/(G*tile_n))
 *   route        uint8  [nb, Hk, T_m, T_mask]  (non-zero = INT8)
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
    int32_t batch, heads_q, heads_kv, seqlen, head_dim;
    int32_t tile_m, tile_n, group;
    int32_t blk_q, blk_k;   /* quantisation block rows for Q and K                     */
    int32_t mask_batch;     /* 1 (mask shared over the batch) or batch                 */
    double softmax_scale;   /* <= 0 means 1/sqrt(head_dim)                              */
} oracle_problem_t;

/* IEEE binary16 -> binary32, exact (every half is representable as a float). */
static float decode_half(uint16_t h) {
    uint32_t sign = (uint32_t)(h >> 15) & 1u;
    uint32_t expo = (uint32_t)(h >> 10) & 0x1fu;
    uint32_t frac = (uint32_t)h & 0x3ffu;
    float v;
    if (expo == 0) {
        v = ldexpf((float)frac, -24);              /* zero and subnormals */
    } else if (expo == 31) {
        v = frac ? NAN : INFINITY;
    } else {
        v = ldexpf((float)(frac | 0x400u), (int)expo - 25);
    }
    return sign ? -v : v;
}

/* The 65536 decoded values, tabulated once (decode_half is the definition). */
static float g_half_table[65536];
static int g_half_table_ready = 0;

void oracle_init(void) {
    if (g_half_table_ready) return;
    for (uint32_t h = 0; h < 65536u; ++h) g_half_table[h] = decode_half((uint16_t)h);
    g_half_table_ready = 1;
}

static float half_bits_to_float(uint16_t h) { return g_half_table[h]; }

static int64_t ceil_div64(int64_t a, int64_t b) { return (a + b - 1) / b; }

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* App. C, "Blockwise INT8 Quantization": for each block r of `blk` consecutive rows of one
 * head, delta = max|x| / 127 and xhat = round(x / delta) in {-127..127}, computed in FP32.
 * Readings: round = IEEE round-half-to-even of the FP32 quotient x/delta; a tail block
 * takes its absmax over the valid rows only; an all-zero block gets delta = 0, xhat = 0.
 *   x     [n_heads, L, d] half bits     out [n_heads, L, d] int8
 *   scale [n_heads, ceil(L/blk)] float                                                   */
void oracle_quantize(const uint16_t* x, int64_t n_heads, int32_t L, int32_t d, int32_t blk,
                     int8_t* out, float* scale) {
    const int64_t n_blk = ceil_div64(L, blk);
#pragma omp parallel for schedule(static)
    for (int64_t hb = 0; hb < n_heads * n_blk; ++hb) {
        const int64_t h = hb / n_blk, r = hb % n_blk;
        const int64_t row0 = r * blk;
        const int64_t row1 = (row0 + blk < L) ? row0 + blk : L;
        const uint16_t* src = x + (h * L + row0) * d;
        int8_t* dst = out + (h * L + row0) * d;
        const int64_t n = (row1 - row0) * d;
        float amax = 0.0f;
        for (int64_t e = 0; e < n; ++e) {
            float a = fabsf(half_bits_to_float(src[e]));
            if (a > amax) amax = a;
        }
        const float delta = amax / 127.0f;
        scale[hb] = delta;
        for (int64_t e = 0; e < n; ++e) {
            int v = 0;
            if (amax > 0.0f) {
                float t = half_bits_to_float(src[e]) / delta;
                float rnd = nearbyintf(t);          /* default mode: ties to even */
                if (rnd > 127.0f) rnd = 127.0f;
                if (rnd < -127.0f) rnd = -127.0f;
                v = (int)rnd;
            }
            dst[e] = (int8_t)v;
        }
    }
}

/* Geometry of one query-tile row (0-based indices everywhere). */
static int64_t last_row_of_tile(const oracle_problem_t* p, int64_t m) {
    int64_t e = (m + 1) * (int64_t)p->tile_m;
    if (e > p->seqlen) e = p->seqlen;
    return e - 1;
}

/* A routing group (m, g) is legal iff it holds at least one legal (query, key) pair, i.e.
 * its first key index does not exceed the last query index of tile row m (causality) and
 * lies inside the sequence (App. B "Coverage Accounting"; the printed set-builder lost its
 * predicate, this is the reading taken).                                                  */
static int group_is_legal(const oracle_problem_t* p, int64_t m, int64_t g) {
    int64_t first_key = g * (int64_t)p->group * p->tile_n;
    return first_key <= last_row_of_tile(p, m);
}

/* A group is "diagonal" for row m iff it holds a key tile n that straddles the diagonal
 * of that row: n*tile_n <= last query row of m  and  (n+1)*tile_n - 1 >= m*tile_m.        */
static int group_is_diagonal(const oracle_problem_t* p, int64_t m, int64_t g) {
    int64_t n0 = g * (int64_t)p->group, n1 = n0 + p->group;
    int64_t T_n = ceil_div64(p->seqlen, p->tile_n);
    if (n1 > T_n) n1 = T_n;
    for (int64_t n = n0; n < n1; ++n) {
        if (n * p->tile_n <= last_row_of_tile(p, m) &&
            (n + 1) * (int64_t)p->tile_n - 1 >= m * (int64_t)p->tile_m)
            return 1;
    }
    return 0;
}

/* Sec. 4.2 "Bitmask packing": b[h_k,m] = sum_g R[h_k,m,g] * 2^g, stored as W little-endian
 * uint32 words (group g -> word g>>5, bit g&31).  Bits of illegal groups, of pad positions
 * beyond T_mask and (if pin_diagonal) of diagonal groups are written as 0.
 * counts [nb, Hk, 2] = {legal groups, INT8-routed legal groups} (App. B coverage).        */
void oracle_pack(const oracle_problem_t* p, const uint8_t* route, int32_t pin_diagonal,
                 uint32_t* words, uint64_t* counts) {
    const int64_t T_m = ceil_div64(p->seqlen, p->tile_m);
    const int64_t T_mask = ceil_div64(p->seqlen, (int64_t)p->group * p->tile_n);
    const int64_t W = ceil_div64(T_mask, 32);
    for (int64_t bh = 0; bh < (int64_t)p->mask_batch * p->heads_kv; ++bh) {
        uint64_t n_legal = 0, n_int8 = 0;
        for (int64_t m = 0; m < T_m; ++m) {
            uint32_t* row = words + (bh * T_m + m) * W;
            for (int64_t w = 0; w < W; ++w) row[w] = 0u;
            for (int64_t g = 0; g < T_mask; ++g) {
                if (!group_is_legal(p, m, g)) continue;
                ++n_legal;
                if (pin_diagonal && group_is_diagonal(p, m, g)) continue;
                if (route[(bh * T_m + m) * T_mask + g]) {
                    row[g >> 5] |= (uint32_t)1u << (g & 31);
                    ++n_int8;
                }
            }
        }
        if (counts) {
            counts[bh * 2 + 0] = n_legal;
            counts[bh * 2 + 1] = n_int8;
        }
    }
}

/* Sec. 4.2 "Constant-time lookup" with the grouping index of Sec. 4.3:
 * g_j = floor(n / G), R = (b >> g_j) & 1.                                                 */
static int route_bit(const oracle_problem_t* p, const uint32_t* words, int64_t b, int64_t hk,
                     int64_t m, int64_t n) {
    const int64_t T_m = ceil_div64(p->seqlen, p->tile_m);
    const int64_t T_mask = ceil_div64(p->seqlen, (int64_t)p->group * p->tile_n);
    const int64_t W = ceil_div64(T_mask, 32);
    const int64_t nb = (p->mask_batch == 1) ? 0 : b;
    const int64_t g = n / p->group;
    const uint32_t* row = words + ((nb * p->heads_kv + hk) * T_m + m) * W;
    return (int)((row[g >> 5] >> (g & 31)) & 1u);
}

/* Attention output for a list of query rows; each row is independent.
 *   rows [n_rows, 3] = (b, h_q, i);  out [n_rows, d] double;  lse [n_rows] double or NULL
 *   row_sum [n_rows] double or NULL: sum_j p_j / Z (should be 1).
 * Per row i (Sec. 3.1 definition, S = QK^T/sqrt(d), P = softmax(S) over keys j <= i,
 * O = PV), with the score of pair (i, j) taken from the route of its tile (Sec. 4.3):
 *   bit 1: S = delta_Q[r] * delta_K[s] * C / sqrt(d),  C = sum_c q8[i,c]*k8[j,c] in int32
 *   bit 0: S = (sum_c q[i,c]*k[j,c]) / sqrt(d)
 * GQA head map h_k = floor(h_q / (H_q/H_k)) (Sec. 4.1).                                    */
void oracle_attention_rows(const oracle_problem_t* p, const uint16_t* q16, const uint16_t* k16,
                           const uint16_t* v16, const int8_t* q8, const int8_t* k8,
                           const float* q_scale, const float* k_scale, const uint32_t* words,
                           int64_t n_rows, const int64_t* rows, double* out, double* lse,
                           double* row_sum) {
    const int64_t L = p->seqlen, d = p->head_dim;
    const int64_t Hq = p->heads_q, Hk = p->heads_kv;
    const int64_t nbq = ceil_div64(L, p->blk_q), nbk = ceil_div64(L, p->blk_k);
    const double scale = (p->softmax_scale > 0.0) ? p->softmax_scale : 1.0 / sqrt((double)d);
#pragma omp parallel
    {
        double* s = (double*)malloc(sizeof(double) * (size_t)L);
        double* qrow = (double*)malloc(sizeof(double) * (size_t)d);
#pragma omp for schedule(dynamic, 1)
        for (int64_t r = 0; r < n_rows; ++r) {
            const int64_t b = rows[3 * r], hq = rows[3 * r + 1], i = rows[3 * r + 2];
            const int64_t hk = hq / (Hq / Hk);
            const int64_t m = i / p->tile_m;
            const uint16_t* qi = q16 + ((b * Hq + hq) * L + i) * d;
            const int8_t* qi8 = q8 ? q8 + ((b * Hq + hq) * L + i) * d : NULL;
            for (int64_t c = 0; c < d; ++c) qrow[c] = (double)half_bits_to_float(qi[c]);
            double mx = -INFINITY;
            for (int64_t j = 0; j <= i; ++j) {
                const int64_t n = j / p->tile_n;
                double sv;
                if (route_bit(p, words, b, hk, m, n)) {
                    const int8_t* kj8 = k8 + ((b * Hk + hk) * L + j) * d;
                    int32_t acc = 0;
                    for (int64_t c = 0; c < d; ++c) acc += (int32_t)qi8[c] * (int32_t)kj8[c];
                    const double dq = (double)q_scale[(b * Hq + hq) * nbq + i / p->blk_q];
                    const double dk = (double)k_scale[(b * Hk + hk) * nbk + j / p->blk_k];
                    sv = dq * dk * (double)acc * scale;
                } else {
                    const uint16_t* kj = k16 + ((b * Hk + hk) * L + j) * d;
                    double acc = 0.0;
                    for (int64_t c = 0; c < d; ++c)
                        acc += qrow[c] * (double)half_bits_to_float(kj[c]);
                    sv = acc * scale;
                }
                s[j] = sv;
                if (sv > mx) mx = sv;
            }
            double Z = 0.0;
            for (int64_t j = 0; j <= i; ++j) {
                s[j] = exp(s[j] - mx);
                Z += s[j];
            }
            double* o = out + r * d;
            for (int64_t c = 0; c < d; ++c) o[c] = 0.0;
            for (int64_t j = 0; j <= i; ++j) {
                const uint16_t* vj = v16 + ((b * Hk + hk) * L + j) * d;
                const double pj = s[j];
                for (int64_t c = 0; c < d; ++c) o[c] += pj * (double)half_bits_to_float(vj[c]);
            }
            double psum = 0.0;
            for (int64_t j = 0; j <= i; ++j) psum += s[j] / Z;
            for (int64_t c = 0; c < d; ++c) o[c] /= Z;
            if (lse) lse[r] = mx + log(Z);
            if (row_sum) row_sum[r] = psum;
        }
        free(s);
        free(qrow);
    }
}

/* App. C "INT8 Score Computation": the raw tile C = Q8_m K8_n^T in int32 for one
 * (b, h_q, m, n), *including* positions above the diagonal (what the tensor core produces
 * before any mask); rows/columns at or beyond the sequence end are 0.
 *   out [tile_m, tile_n] int32                                                           */
void oracle_int32_tile(const oracle_problem_t* p, const int8_t* q8, const int8_t* k8, int64_t b,
                       int64_t hq, int64_t m, int64_t n, int32_t* out) {
    const int64_t L = p->seqlen, d = p->head_dim;
    const int64_t hk = hq / (p->heads_q / p->heads_kv);
    for (int64_t ii = 0; ii < p->tile_m; ++ii) {
        for (int64_t jj = 0; jj < p->tile_n; ++jj) {
            const int64_t i = m * p->tile_m + ii, j = n * p->tile_n + jj;
            int32_t acc = 0;
            if (i < L && j < L) {
                const int8_t* a = q8 + ((b * p->heads_q + hq) * L + i) * d;
                const int8_t* c8 = k8 + ((b * p->heads_kv + hk) * L + j) * d;
                for (int64_t c = 0; c < d; ++c) acc += (int32_t)a[c] * (int32_t)c8[c];
            }
            out[ii * p->tile_n + jj] = acc;
        }
    }
}

/* The FP16-route raw tile Q_m K_n^T (before the 1/sqrt(d) scaling), in double, same
 * conventions as oracle_int32_tile.   out [tile_m, tile_n] double                          */
void oracle_fp_tile(const oracle_problem_t* p, const uint16_t* q16, const uint16_t* k16,
                    int64_t b, int64_t hq, int64_t m, int64_t n, double* out) {
    const int64_t L = p->seqlen, d = p->head_dim;
    const int64_t hk = hq / (p->heads_q / p->heads_kv);
    for (int64_t ii = 0; ii < p->tile_m; ++ii) {
        for (int64_t jj = 0; jj < p->tile_n; ++jj) {
            const int64_t i = m * p->tile_m + ii, j = n * p->tile_n + jj;
            double acc = 0.0;
            if (i < L && j < L) {
                const uint16_t* a = q16 + ((b * p->heads_q + hq) * L + i) * d;
                const uint16_t* c16 = k16 + ((b * p->heads_kv + hk) * L + j) * d;
                for (int64_t c = 0; c < d; ++c)
                    acc += (double)half_bits_to_float(a[c]) * (double)half_bits_to_float(c16[c]);
            }
            out[ii * p->tile_n + jj] = acc;
        }
    }
}
