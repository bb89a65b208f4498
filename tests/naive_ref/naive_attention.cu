// Naive CUDA reference of the TileMix hot path -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
//
// The middle rung between the CPU oracle (too slow for every row of the large configurations) and the fused
// kernel: one warp per query row, FP32 arithmetic on the CUDA cores, the INT8 dot products with __dp4a, plain
// loads, no tensor cores, no TMA, no tensor memory.  It shares no code, header or table with libtilemix; it reads
// the UNPACKED routing map (bytes), decides legality and the diagonal pin itself, and has its own quantiser.
// The tests check it against the oracle (all rows of small cases, sampled rows of the large ones) and then check
// the fused kernel against it on every row.
//
//   scores (Sec. 4.3 / App. C):  bit 1: S = delta_Q[r] delta_K[s] (q8 . k8) / sqrt(d)     bit 0: S = (q . k) / sqrt(d)
//   softmax over the keys j <= i (Sec. 3.1), running maximum / sum per row, O = P V
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

namespace {

constexpr int kRowsPerBlock = 8;     // one warp per query row
constexpr int kChunk = 32;           // keys per step: one key per lane

// Blockwise INT8 quantiser (App. C): delta = max|x| / 127 over the block's rows of one head, code =
// round-half-even(x / delta), both in FP32 with IEEE division; a zero block gives delta = 0 and codes 0.
__global__ void naive_quantize_kernel(const __half* __restrict__ x, int L, int d, int blk, int n_blk,
                                      int8_t* __restrict__ out, float* __restrict__ scale) {
    const int64_t head = blockIdx.y;
    const int r = blockIdx.x;
    const int row0 = r * blk, row1 = min(row0 + blk, L);
    const int64_t n = static_cast<int64_t>(row1 - row0) * d;
    const __half* src = x + (head * L + row0) * d;
    int8_t* dst = out + (head * L + row0) * d;
    __shared__ unsigned int amax_bits;
    if (threadIdx.x == 0) amax_bits = 0u;
    __syncthreads();
    unsigned int local = 0u;
    for (int64_t e = threadIdx.x; e < n; e += blockDim.x)
        local = max(local, __float_as_uint(fabsf(__half2float(src[e]))));     // non-negative floats order like their bits
    atomicMax(&amax_bits, local);
    __syncthreads();
    const float amax = __uint_as_float(amax_bits);
    const float delta = __fdiv_rn(amax, 127.0f);
    if (threadIdx.x == 0) scale[head * n_blk + r] = delta;
    for (int64_t e = threadIdx.x; e < n; e += blockDim.x) {
        int v = 0;
        if (amax > 0.0f) {
            float t = rintf(__fdiv_rn(__half2float(src[e]), delta));
            t = fminf(fmaxf(t, -127.0f), 127.0f);
            v = static_cast<int>(t);
        }
        dst[e] = static_cast<int8_t>(v);
    }
}

struct AttnArgs {
    const __half *q, *k, *v;          // [B, H, L, d] dense
    const int8_t *q8, *k8;            // [B, H, L, d] dense
    const float *qs, *ks;             // [B, Hq, ceil(L/blk_q)], [B, Hk, ceil(L/blk_k)]
    const uint8_t* route;             // [nb, Hk, T_m, T_mask] bytes, non-zero = INT8
    int B, Hq, Hk, L, tile, G, blk_q, blk_k, nb, pin;
    float scale;
    float *out, *lse;                 // [B, Hq, L, d] FP32, [B, Hq, L] (nullable)
};

template <int D>
__global__ void __launch_bounds__(kRowsPerBlock * 32) naive_attention_kernel(const AttnArgs a) {
    constexpr int CPL = D / 32;                       // output columns per lane
    __shared__ __align__(16) __half k16_s[kChunk][D + 8];
    __shared__ __align__(16) int8_t k8_s[kChunk][D + 16];
    __shared__ __align__(16) __half v_s[kChunk][D];
    __shared__ __align__(16) float q_s[kRowsPerBlock][D];
    __shared__ __align__(16) int8_t q8_s[kRowsPerBlock][D];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int b = blockIdx.z, hq = blockIdx.y, hk = hq / (a.Hq / a.Hk);
    const int i0 = (gridDim.x - 1 - blockIdx.x) * kRowsPerBlock;      // long rows first
    const int i = i0 + warp;
    const bool row_ok = i < a.L;
    const int T_m = (a.L + a.tile - 1) / a.tile, T_mask = (a.L + a.G * a.tile - 1) / (a.G * a.tile);
    const int m = i0 / a.tile;                                          // the block's rows share a query tile
    const int nbq = (a.L + a.blk_q - 1) / a.blk_q, nbk = (a.L + a.blk_k - 1) / a.blk_k;
    const __half* qrow = a.q + ((static_cast<int64_t>(b) * a.Hq + hq) * a.L + (row_ok ? i : 0)) * D;
    const int8_t* q8row = a.q8 ? a.q8 + ((static_cast<int64_t>(b) * a.Hq + hq) * a.L + (row_ok ? i : 0)) * D : nullptr;
    for (int c = lane; c < D; c += 32) {
        q_s[warp][c] = __half2float(qrow[c]);
        q8_s[warp][c] = q8row ? q8row[c] : 0;
    }
    const float dq = (a.qs && row_ok) ? a.qs[(static_cast<int64_t>(b) * a.Hq + hq) * nbq + i / a.blk_q] : 0.f;
    const uint8_t* route_row = a.route + ((static_cast<int64_t>(a.nb == 1 ? 0 : b) * a.Hk + hk) * T_m + m) * T_mask;
    const int64_t kv_base = (static_cast<int64_t>(b) * a.Hk + hk) * a.L;

    float m_run = -INFINITY, z = 0.f, o[CPL];
#pragma unroll
    for (int c = 0; c < CPL; ++c) o[c] = 0.f;
    const int i_last = min(i0 + kRowsPerBlock, a.L) - 1;
    for (int c0 = 0; c0 <= i_last; c0 += kChunk) {
        // routing decision of this chunk (Sec. 4.2 lookup on the unpacked map; App. B: the diagonal group of a
        // row of square tiles is the one that holds key tile m)
        const int n = c0 / a.tile, g = n / a.G;
        const bool int8 = route_row[g] != 0 && !(a.pin && g == m / a.G);
        __syncthreads();       // the previous chunk has been consumed
        for (int e = threadIdx.x; e < kChunk * (D / 8); e += blockDim.x) {
            const int r = e / (D / 8), c8 = e % (D / 8);
            const int j = c0 + r;
            uint4 vv = make_uint4(0u, 0u, 0u, 0u), kk = vv;
            if (j < a.L) {
                vv = *reinterpret_cast<const uint4*>(a.v + (kv_base + j) * D + c8 * 8);
                if (!int8) kk = *reinterpret_cast<const uint4*>(a.k + (kv_base + j) * D + c8 * 8);
            }
            *reinterpret_cast<uint4*>(&v_s[r][c8 * 8]) = vv;
            if (!int8) *reinterpret_cast<uint4*>(&k16_s[r][c8 * 8]) = kk;
        }
        if (int8) {
            for (int e = threadIdx.x; e < kChunk * (D / 16); e += blockDim.x) {
                const int r = e / (D / 16), c16 = e % (D / 16);
                const int j = c0 + r;
                uint4 kk = make_uint4(0u, 0u, 0u, 0u);
                if (j < a.L) kk = *reinterpret_cast<const uint4*>(a.k8 + (kv_base + j) * D + c16 * 16);
                *reinterpret_cast<uint4*>(&k8_s[r][c16 * 16]) = kk;
            }
        }
        __syncthreads();
        // score of (row i, key c0 + lane)
        const int j = c0 + lane;
        float s = -INFINITY;
        if (row_ok && j <= i) {
            if (int8) {
                int acc = 0;
                for (int c = 0; c < D; c += 4)
                    acc = __dp4a(*reinterpret_cast<const int*>(&q8_s[warp][c]), *reinterpret_cast<const int*>(&k8_s[lane][c]), acc);
                const float dk = a.ks[(static_cast<int64_t>(b) * a.Hk + hk) * nbk + j / a.blk_k];
                s = dq * dk * static_cast<float>(acc) * a.scale;
            } else {
                float acc = 0.f;
                for (int c = 0; c < D; ++c) acc = fmaf(q_s[warp][c], __half2float(k16_s[lane][c]), acc);
                s = acc * a.scale;
            }
        }
        float mx = s;
        for (int off = 16; off > 0; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
        if (mx == -INFINITY) continue;                 // (uniform per warp) no legal key of this row in the chunk
        const float m_new = fmaxf(m_run, mx);
        const float corr = expf(m_run - m_new);         // 0 on the first chunk
        const float p = expf(s - m_new);                // 0 for an excluded key
        float psum = p;
        for (int off = 16; off > 0; off >>= 1) psum += __shfl_xor_sync(0xffffffffu, psum, off);
        z = z * corr + psum;
#pragma unroll
        for (int c = 0; c < CPL; ++c) o[c] *= corr;
        for (int l = 0; l < kChunk; ++l) {
            const float pl = __shfl_sync(0xffffffffu, p, l);
#pragma unroll
            for (int c = 0; c < CPL; ++c) o[c] = fmaf(pl, __half2float(v_s[l][lane * CPL + c]), o[c]);
        }
        m_run = m_new;
    }
    if (row_ok) {
        float* dst = a.out + ((static_cast<int64_t>(b) * a.Hq + hq) * a.L + i) * D + lane * CPL;
#pragma unroll
        for (int c = 0; c < CPL; ++c) dst[c] = o[c] / z;
        if (a.lse && lane == 0) a.lse[(static_cast<int64_t>(b) * a.Hq + hq) * a.L + i] = m_run + logf(z);
    }
}

}  // namespace

extern "C" {

// x [n_heads, L, d] FP16 (device) -> out INT8 same shape, scale [n_heads, ceil(L/blk)]
int naive_quantize(const void* x_f16, int64_t n_heads, int L, int d, int blk, int8_t* out, float* scale, void* stream) {
    const int n_blk = (L + blk - 1) / blk;
    dim3 grid(n_blk, static_cast<unsigned>(n_heads));
    naive_quantize_kernel<<<grid, 256, 0, static_cast<cudaStream_t>(stream)>>>(static_cast<const __half*>(x_f16), L, d, blk, n_blk, out, scale);
    return static_cast<int>(cudaGetLastError());
}

// Dense [B, H, L, d] tensors on the device; route: bytes [nb, Hk, T_m, T_mask] (square tiles); out FP32.
int naive_attention(const void* q, const void* k, const void* v, const int8_t* q8, const int8_t* k8, const float* qs,
                    const float* ks, const uint8_t* route, int B, int Hq, int Hk, int L, int d, int tile, int G,
                    int blk_q, int blk_k, int nb, int pin, float scale, float* out, float* lse, void* stream) {
    if (tile % kChunk != 0 || (d != 64 && d != 128) || Hq % Hk != 0) return -1;
    AttnArgs a{static_cast<const __half*>(q), static_cast<const __half*>(k), static_cast<const __half*>(v), q8, k8, qs, ks,
               route, B, Hq, Hk, L, tile, G, blk_q, blk_k, nb, pin, scale, out, lse};
    dim3 grid((L + kRowsPerBlock - 1) / kRowsPerBlock, Hq, B);
    if (d == 128) naive_attention_kernel<128><<<grid, kRowsPerBlock * 32, 0, static_cast<cudaStream_t>(stream)>>>(a);
    else naive_attention_kernel<64><<<grid, kRowsPerBlock * 32, 0, static_cast<cudaStream_t>(stream)>>>(a);
    return static_cast<int>(cudaGetLastError());
}

}  // extern "C"
