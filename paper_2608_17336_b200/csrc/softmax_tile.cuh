// Per-thread softmax arithmetic of the attention kernel (Sec. 3.1 recurrence in the log2 domain; App. C common
// score domain).  A softmax warp owns 16 query rows of a score tile and reads them from tensor memory in the
// 16-lane "256-bit" shape: per block of 8 key columns a thread holds two adjacent columns of row r and the
// same two columns of row r + 8 (r = lane / 4, columns 2 * (lane % 4) and + 1), i.e. registers
// 4i .. 4i+3 = (r, c), (r, c + 1), (r + 8, c), (r + 8, c + 1) of block i.  The two adjacent columns of a row
// become one FP16 pair of P, which is exactly one 32-bit column of the 16-lane "128-bit" store shape.
#pragma once

#include <cuda_fp16.h>
#include <limits.h>
#include <stdint.h>

#include "ptx_sm100.cuh"

namespace tilemix {

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ float fmax3(float a, float b, float c) {
    float r;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}

__device__ __forceinline__ uint32_t pack_half2(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

// Maximum / sum over the four threads that share a row (lanes 4k .. 4k+3).
__device__ __forceinline__ float quad_max(float v) {
    v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 1));
    return fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 2));
}
__device__ __forceinline__ float quad_sum(float v) {
    v += __shfl_xor_sync(0xffffffffu, v, 1);
    return v + __shfl_xor_sync(0xffffffffu, v, 2);
}

// How the raw accumulators of a step become floats: FP32 scores as they are; INT32 scores by the bias trick --
// bits(1.5*2^23) + i is the float 1.5*2^23 + i for |i| < 2^22 (here |i| <= 127*127*D) -- either with the bias
// removed by an exact subtraction before the scaling (kInt8Exact), or left in and cancelled by the addend of the
// scaling FMA, a*(1.5*2^23 + i) - (m + a*1.5*2^23) (kInt8Folded: one instruction less per pair; the addend is
// rounded once per step, so the caller uses it only while that rounding is negligible).
enum ScoreKind : int { kFp32 = 0, kInt8Exact = 1, kInt8Folded = 2 };
constexpr float kInt8Bias = 12582912.f;   // 1.5 * 2^23

// One interior step (NB blocks of 8 key columns, no causal mask) in one pass with the current running
// maxima: raw accumulators s -> P = 2^(a*raw - m) rounded to FP16 (p[2i + k] = the pair of row k in block
// i) and this thread's part of the FP32 row sums.  addend[k] = -m_k (kFp32, kInt8Exact) or -(m_k + a*1.5*2^23)
// (kInt8Folded).  VS: the probabilities are multiplied by `dv` (the block scale of an INT8 value cache, App. C:
// folded into the probability tile) before they are rounded to FP16; the row sums are of the unscaled values.
template <int NB, int KIND, bool VS = false>
__device__ __forceinline__ void softmax_step_fast(const uint32_t (&s)[4 * NB], float a, const float (&addend)[2],
                                                  uint32_t (&p)[2 * NB], float (&sum)[2], float dv = 1.f) {
    const float2 a2 = make_float2(a, a);
    const float2 unbias = make_float2(-kInt8Bias, -kInt8Bias);
    float2 acc[2] = {{0.f, 0.f}, {0.f, 0.f}};
#pragma unroll
    for (int i = 0; i < NB; ++i) {
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            const uint32_t r0 = s[4 * i + 2 * k], r1 = s[4 * i + 2 * k + 1];
            float2 x;
            if (KIND == kFp32) {
                x = make_float2(__uint_as_float(r0), __uint_as_float(r1));
            } else {
                x = make_float2(__uint_as_float(r0 + 0x4B400000u), __uint_as_float(r1 + 0x4B400000u));
                if (KIND == kInt8Exact) x = __fadd2_rn(x, unbias);
            }
            const float2 t2 = __ffma2_rn(x, a2, make_float2(addend[k], addend[k]));
            const float2 e = make_float2(fast_exp2(t2.x), fast_exp2(t2.y));
            acc[k] = __fadd2_rn(acc[k], e);
            if constexpr (VS) {
                const float2 ev = __fmul2_rn(e, make_float2(dv, dv));
                p[2 * i + k] = pack_half2(ev.x, ev.y);
            } else {
                p[2 * i + k] = pack_half2(e.x, e.y);
            }
        }
    }
    sum[0] = acc[0].x + acc[0].y;
    sum[1] = acc[1].x + acc[1].y;
}

}  // namespace tilemix
