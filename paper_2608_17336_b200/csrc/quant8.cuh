// Arithmetic of the blockwise symmetric INT8 quantiser (App. C, "Blockwise INT8 Quantization"), shared by
// the quantise-once kernel and the attention kernel's on-chip quantiser: xhat = round(x / delta) with an
// IEEE FP32 quotient and round-half-to-even, clamped to [-127, 127].
#pragma once

#include <cuda_fp16.h>
#include <stdint.h>

namespace tilemix {

__device__ __forceinline__ uint32_t habs2_bits(uint32_t v) { return v & 0x7fff7fffu; }

// max of two packed pairs of non-negative binary16 values: for non-negative finite halves the
// bit patterns order like unsigned integers.
__device__ __forceinline__ uint32_t umax2(uint32_t a, uint32_t b) { return __vmaxu2(a, b); }

// The definition: IEEE quotient x / delta, rounded to the nearest integer, ties to even.
__device__ __forceinline__ int quant1_exact(float x, float delta) {
    int q = __float2int_rn(__fdiv_rn(x, delta));
    return max(-127, min(127, q));
}

// Same result without a division per element.  t = x * fl(1/delta) is within 2.3e-5 of the IEEE
// quotient (|quotient| <= 127.5), so both round to the same integer unless t lies within 1e-4 of a
// half-integer; only then is the quotient formed exactly.  The rounding itself is done by adding
// 1.5 * 2^23 (round-to-nearest-even puts the integer in the low mantissa bits, so the low byte of the
// sum IS the two's-complement INT8 code).  Eight elements at a time, packed FP32x2 arithmetic; the
// distance of every t from its rounded value is folded into the running maximum `dmax`, which the caller
// checks (once per vector or once per several): above kQuantTieGuard some element is (nearly) a tie and
// quant8_exact has to be used instead.
constexpr float kQuantTieGuard = 0.4999f;

__device__ __forceinline__ uint2 quant8_fast(const uint4& v, float rdelta, float& dmax) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    const float2 r2 = make_float2(rdelta, rdelta);
    const float2 magic = make_float2(12582912.f, 12582912.f), nmagic = make_float2(-12582912.f, -12582912.f);
    float2 y[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float2 x = __half22float2(*reinterpret_cast<const __half2*>(&w[i]));
        const float2 t = __fmul2_rn(x, r2);
        y[i] = __fadd2_rn(t, magic);
        const float2 back = __fadd2_rn(y[i], nmagic);
        const float2 d = __fadd2_rn(t, make_float2(-back.x, -back.y));
        dmax = fmaxf(dmax, fmaxf(fabsf(d.x), fabsf(d.y)));
    }
    // low bytes of the eight sums -> two words
    const uint32_t p0 = __byte_perm(__float_as_uint(y[0].x), __float_as_uint(y[0].y), 0x0040);
    const uint32_t p1 = __byte_perm(__float_as_uint(y[1].x), __float_as_uint(y[1].y), 0x0040);
    const uint32_t p2 = __byte_perm(__float_as_uint(y[2].x), __float_as_uint(y[2].y), 0x0040);
    const uint32_t p3 = __byte_perm(__float_as_uint(y[3].x), __float_as_uint(y[3].y), 0x0040);
    return make_uint2(__byte_perm(p0, p1, 0x5410), __byte_perm(p2, p3, 0x5410));
}

// The definition, element by element.
__device__ __forceinline__ uint2 quant8_exact(const uint4& v, float delta) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    uint32_t o[2] = {0u, 0u};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float2 x = __half22float2(*reinterpret_cast<const __half2*>(&w[i]));
        const uint32_t lo = static_cast<uint32_t>(quant1_exact(x.x, delta)) & 0xffu;
        const uint32_t hi = static_cast<uint32_t>(quant1_exact(x.y, delta)) & 0xffu;
        o[i >> 1] |= (lo | (hi << 8)) << ((i & 1) * 16);
    }
    return make_uint2(o[0], o[1]);
}

// Branch-free form for a caller whose lanes must not diverge (the attention kernel's on-chip quantiser):
// the IEEE quotient itself, by the classical refinement with the exact residual -- q0 = x * r with
// r = RN(1/delta), then twice q <- q + (x - delta * q) * r, the residual being exact in one FMA.  The first
// step leaves q within one unit in the last place of x / delta, the second rounds it correctly (the final
// step of a software division; no operand here is near the underflow or overflow range: |x| is a
// binary16 magnitude, |x / delta| <= 127.5).  The integer rounding is the magic-number add of quant8_fast.
__device__ __forceinline__ uint2 quant8_div(const uint4& v, float delta, float rdelta) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    const float2 r2 = make_float2(rdelta, rdelta), nd2 = make_float2(-delta, -delta);
    const float2 magic = make_float2(12582912.f, 12582912.f);
    float2 y[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float2 x = __half22float2(*reinterpret_cast<const __half2*>(&w[i]));
        float2 q = __fmul2_rn(x, r2);
        float2 e = __ffma2_rn(nd2, q, x);
        q = __ffma2_rn(e, r2, q);
        e = __ffma2_rn(nd2, q, x);
        q = __ffma2_rn(e, r2, q);
        y[i] = __fadd2_rn(q, magic);
    }
    const uint32_t p0 = __byte_perm(__float_as_uint(y[0].x), __float_as_uint(y[0].y), 0x0040);
    const uint32_t p1 = __byte_perm(__float_as_uint(y[1].x), __float_as_uint(y[1].y), 0x0040);
    const uint32_t p2 = __byte_perm(__float_as_uint(y[2].x), __float_as_uint(y[2].y), 0x0040);
    const uint32_t p3 = __byte_perm(__float_as_uint(y[3].x), __float_as_uint(y[3].y), 0x0040);
    return make_uint2(__byte_perm(p0, p1, 0x5410), __byte_perm(p2, p3, 0x5410));
}

__device__ __forceinline__ uint2 quant8(const uint4& v, float delta, float rdelta) {
    float dmax = 0.f;
    const uint2 q = quant8_fast(v, rdelta, dmax);
    if (dmax > kQuantTieGuard) return quant8_exact(v, delta);
    return q;
}

}  // namespace tilemix
