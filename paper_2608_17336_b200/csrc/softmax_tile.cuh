// Per-thread softmax arithmetic of the attention kernel: one thread owns one query row of a score
// tile (Sec. 3.1 recurrence in the log2 domain; App. C common score domain).
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

// One interior step (T score columns) in one pass: raw accumulators in tensor memory at t_s ->
// P = 2^(a*raw - m) rounded to FP16 and packed two per word into p2, the FP32 row sum of P and the row
// maximum of the raw values.  The 32-column chunks are double-buffered (the next one is in flight
// while this one is processed; the FIRST one was put in flight into `first` by the caller), and the
// per-pair work is software-pipelined in program order -- exponentials of pair k, conversion of pair
// k + kD1, sum and packing of pair k - (kD2 - kD1) -- because a warp issues in order: the
// special-function unit takes 16 clocks per pair and the other ~7 instructions of a pair fit in its
// shadow only if they belong to other pairs.  `late()` is called once, when `first` is free again (its
// last chunk has been consumed): the caller may start the NEXT step's first chunk into it there, so
// that the latency of that load hides behind the rest of this step.
template <int T, bool INT8, class Late>
__device__ __forceinline__ void softmax_tile_fast(uint32_t t_s, uint32_t (&first)[32], float a, float m_run,
                                                  uint32_t (&p2)[T / 2], float& sum, float& mx, Late&& late) {
    // Pipeline depth in pairs: pair k is read (and, INT8, re-biased) in iteration k, made a float in
    // k + 1, scaled in k + 2, exponentiated in k + kE and summed / packed in k + kS.  No instruction
    // uses a result produced in its own iteration.
    #ifndef TILEMIX_KE
#define TILEMIX_KE 3
#define TILEMIX_KS 7
#endif
    constexpr int NP = T / 2, kE = TILEMIX_KE, kS = TILEMIX_KS;
    const float2 a2 = make_float2(a, a), nm2 = make_float2(-m_run, -m_run);
    const float2 unbias = make_float2(-12582912.f, -12582912.f);
    float2 acc[4] = {{0.f, 0.f}, {0.f, 0.f}, {0.f, 0.f}, {0.f, 0.f}};
    int mi[4] = {INT_MIN, INT_MIN, INT_MIN, INT_MIN};
    float mf[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
    float2 xb[4], tb[4], eb[8];       // rings: biased / float raw values, scaled values, exponentials
#ifndef TILEMIX_LATE_BEFORE_END
#define TILEMIX_LATE_BEFORE_END 8
#endif
    // iteration at which late() runs: not before the last even chunk (held in `first`) is consumed
    constexpr int kFirstFree = ((((T / 32) - 1) & ~1) + 1) * 16;
    constexpr int kLateAt = (NP - TILEMIX_LATE_BEFORE_END > kFirstFree) ? NP - TILEMIX_LATE_BEFORE_END : kFirstFree;
    uint32_t buf[32];                 // odd chunks; even chunks land in `first`
#pragma unroll
    for (int i = 0; i < NP + kS; ++i) {
        if (i == kLateAt) late();
        if (i >= kE && i - kE < NP) {                         // exponentials of pair i - kE
            const int k = i - kE;
            eb[k & 7] = make_float2(fast_exp2(tb[k & 3].x), fast_exp2(tb[k & 3].y));
        }
        if (i >= 2 && i - 2 < NP) {                           // a*raw - m of pair i - 2
            const int k = i - 2;
            tb[k & 3] = __ffma2_rn(xb[k & 3], a2, nm2);
        }
        if (INT8 && i >= 1 && i - 1 < NP) {                   // remove the bias of pair i - 1 (exact)
            const int k = i - 1;
            xb[k & 3] = __fadd2_rn(xb[k & 3], unbias);
        }
        if (i < NP) {                                         // read pair i
            const int c = i / 16, e = (i % 16) * 2;
            if (e == 0) {
                if (c & 1) {
                    ptx::tmem_wait_ld_dep(buf);
                    if (c + 1 < T / 32) ptx::tmem_ld32(t_s + (c + 1) * 32, first);
                } else {
                    ptx::tmem_wait_ld_dep(first);
                    if (c + 1 < T / 32) ptx::tmem_ld32(t_s + (c + 1) * 32, buf);
                }
            }
            const uint32_t r0 = (c & 1) ? buf[e] : first[e], r1 = (c & 1) ? buf[e + 1] : first[e + 1];
            if (INT8) {
                // int -> float without the conversion unit: bits(1.5*2^23) + i is the float
                // 1.5*2^23 + i for |i| < 2^22 (here |i| <= 127*127*D); subtracting 1.5*2^23 is exact.
                mi[i & 3] = __vimax3_s32(mi[i & 3], static_cast<int>(r0), static_cast<int>(r1));
                xb[i & 3] = make_float2(__uint_as_float(r0 + 0x4B400000u), __uint_as_float(r1 + 0x4B400000u));
            } else {
                mf[i & 3] = fmax3(mf[i & 3], __uint_as_float(r0), __uint_as_float(r1));
                xb[i & 3] = make_float2(__uint_as_float(r0), __uint_as_float(r1));
            }
        }
        if (i >= kS) {                                        // row sum and FP16 packing of pair i - kS
            const int k = i - kS;
            acc[k & 3] = __fadd2_rn(acc[k & 3], eb[k & 7]);
            p2[k] = pack_half2(eb[k & 7].x, eb[k & 7].y);
        }
    }
    mx = INT8 ? __int2float_rn(max(max(mi[0], mi[1]), max(mi[2], mi[3])))
              : fmaxf(fmaxf(mf[0], mf[1]), fmaxf(mf[2], mf[3]));
    const float2 s01 = __fadd2_rn(acc[0], acc[1]), s23 = __fadd2_rn(acc[2], acc[3]);
    sum = (s01.x + s01.y) + (s23.x + s23.y);
}

}  // namespace tilemix
