// Routing-mask packer (Sec. 4.2, "Bitmask packing"; App. B, "Coverage Accounting"): turns the
// byte map R[nb, h_k, m, g] into rows of W little-endian uint32 words with bit g = R, and
// counts legal and INT8-routed groups per (nb, h_k).  Causal legality is applied here so the
// packed form is canonical: groups with no legal pair, pad bits and (optionally) diagonal
// groups are written as 0.
#include "common.cuh"

namespace tilemix {

namespace {

constexpr int kThreads = 256;

__global__ void __launch_bounds__(kThreads)
pack_kernel(const uint8_t* __restrict__ route, int L, int tile_m, int tile_n, int G, int T_m,
            int T_mask, int W, int pin_diag, uint32_t* __restrict__ words,
            unsigned long long* __restrict__ counts, const int32_t* __restrict__ tok,
            const int32_t* __restrict__ tile_off, int n_seqs) {
    const int64_t bh = blockIdx.x;
    const uint8_t* r_in = route + bh * T_m * static_cast<int64_t>(T_mask);
    uint32_t* w_out = words + bh * T_m * static_cast<int64_t>(W);
    unsigned int n_legal = 0, n_int8 = 0;
    for (int idx = threadIdx.x; idx < T_m * W; idx += kThreads) {
        const int m_row = idx / W, w = idx - m_row * W;
        // variable-length batch: row m_row of the packed batch is row m of its own sequence of length L
        int m = m_row;
        if (tok != nullptr) {
            const int s = find_seq(tile_off, n_seqs, m_row);
            m = m_row - tile_off[s];
            L = tok[s + 1] - tok[s];
        }
        const int64_t last_row = min(static_cast<int64_t>(m + 1) * tile_m, static_cast<int64_t>(L)) - 1;
        // key tiles that straddle the diagonal of row m: [n_lo, n_hi]
        const int64_t n_lo = static_cast<int64_t>(m) * tile_m / tile_n;
        const int64_t n_hi = last_row / tile_n;
        uint32_t word = 0u;
        for (int t = 0; t < 32; ++t) {
            const int64_t g = 32 * w + t;
            if (g >= T_mask) break;
            const int64_t first_tile = g * G;
            if (first_tile * tile_n > last_row) break;  // this and all later groups are illegal
                                                        // (also every group beyond the sequence's own T_mask)
            ++n_legal;
            const bool diag = first_tile <= n_hi && first_tile + G - 1 >= n_lo;
            if (pin_diag && diag) continue;
            if (r_in[static_cast<int64_t>(m_row) * T_mask + g] != 0) {
                word |= 1u << t;
                ++n_int8;
            }
        }
        w_out[idx] = word;
    }
    if (counts == nullptr) return;
    __shared__ unsigned int s_legal, s_int8;
    if (threadIdx.x == 0) { s_legal = 0; s_int8 = 0; }
    __syncthreads();
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        n_legal += __shfl_xor_sync(0xffffffffu, n_legal, o);
        n_int8 += __shfl_xor_sync(0xffffffffu, n_int8, o);
    }
    if ((threadIdx.x & 31) == 0) { atomicAdd(&s_legal, n_legal); atomicAdd(&s_int8, n_int8); }
    __syncthreads();
    if (threadIdx.x == 0) {
        counts[bh * 2 + 0] = s_legal;
        counts[bh * 2 + 1] = s_int8;
    }
}

}  // namespace

int launch_pack(const Geometry& g, const uint8_t* route, uint32_t pack_flags, uint32_t* words,
                unsigned long long* counts, cudaStream_t stream, const VarlenDev* vl) {
    const int ctas = g.nb * g.Hk;
    pack_kernel<<<ctas, kThreads, 0, stream>>>(route, g.L, g.tile_m, g.tile_n, g.G, g.T_m, g.T_mask,
                                               g.W, (pack_flags & TILEMIX_PIN_DIAGONAL_FP16) ? 1 : 0,
                                               words, counts, vl ? vl->tok : nullptr, vl ? vl->tile : nullptr,
                                               vl ? vl->n : 0);
    g_launch_count.fetch_add(1);
    return static_cast<int>(cudaGetLastError());
}

}  // namespace tilemix
