// Decode / quantise routines shared by the tuned kernels (Alg. 2 line 5: e = decode(state);
// line 9: state = C(r), the block absmax quantiser of Sec. 4.2.1), written on bit patterns.
#pragma once
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <float.h>
#include <stdint.h>

#include "conef_internal.h"

namespace conef {

// ------------------------------------------------------------------ decode / quantise, lean forms
// e_j = float(code_j) * scale for 8 consecutive elements.  A code is moved into
// the top mantissa bits of a float f = 1 + (code + bias) / span, so that
// code = span * f - (span + bias) exactly.  With a binary16 scale the product
// code * scale is exact in fp32 and one fused multiply-add gives it; with an
// fp32 scale the code is formed first and one rounded multiply follows.  Both
// equal __fmul_rn((float)code, scale).
template <int CK>
struct ScaleConst {
    float a, b;   // half scales: e = fma(f, a, b); fp32 scales: e = fmul(fma(f, span, -(span+bias)), a)
};
template <int CK, bool HALF>
__device__ __forceinline__ ScaleConst<CK> scale_const(float s)
{
    ScaleConst<CK> k;
    constexpr float span = (CK == CONEF_C_INT4) ? 16.f : 256.f;
    constexpr float off = (CK == CONEF_C_INT4) ? 24.f : 384.f;
    k.a = HALF ? __fmul_rn(s, span) : s;
    k.b = HALF ? __fmul_rn(s, -off) : 0.f;
    return k;
}
// bit patterns of the floats f = 1 + (code + bias) / span of 8 codes
template <int CK>
__device__ __forceinline__ void decode8_bits(uint32_t w0, uint32_t w1, uint32_t (&t)[8])
{
#pragma unroll
    for (int q = 0; q < 8; ++q) {
        if (CK == CONEF_C_INT4) {
            const uint32_t w = q < 4 ? w0 : (w0 >> 16);
            t[q] = ((w << (19 - 4 * (q & 3))) & 0x00780000u) ^ 0x3FC00000u;
        } else {
            const uint32_t w = q < 4 ? w0 : w1;
            const int qq = q & 3;
            const uint32_t sh = qq == 0 ? (w << 15) : qq == 1 ? (w << 7) : qq == 2 ? (w >> 1) : (w >> 9);
            t[q] = (sh & 0x007F8000u) ^ 0x3FC00000u;
        }
    }
}
template <int CK, bool HALF>
__device__ __forceinline__ void decode8(uint32_t w0, uint32_t w1, const ScaleConst<CK> &k, float (&e)[8])
{
    constexpr float span = (CK == CONEF_C_INT4) ? 16.f : 256.f;
    constexpr float off = (CK == CONEF_C_INT4) ? 24.f : 384.f;
    uint32_t t[8];
    decode8_bits<CK>(w0, w1, t);
#pragma unroll
    for (int q = 0; q < 8; ++q) {
        const float f = __uint_as_float(t[q]);
        e[q] = HALF ? __fmaf_rn(f, k.a, k.b) : __fmul_rn(__fmaf_rn(f, span, -off), k.a);
    }
}

// ------------------------------------------------------------------ two fp32 operations per instruction
// sm_100a has packed fp32 arithmetic on register pairs: each half is the IEEE operation of the
// scalar instruction, so results are bit for bit those of two scalar instructions.  (Used for the
// fused multiply-adds and for multiplies that no add follows.)
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 pk2(float lo, float hi)
{
    f32x2 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ f32x2 pk2u(uint32_t lo, uint32_t hi)
{
    f32x2 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(lo), "r"(hi));
    return r;
}
__device__ __forceinline__ void upk2(f32x2 v, float &lo, float &hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v)); }
__device__ __forceinline__ void upk2u(f32x2 v, uint32_t &lo, uint32_t &hi) { asm("mov.b64 {%0, %1}, %2;" : "=r"(lo), "=r"(hi) : "l"(v)); }
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c)
{
    f32x2 d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ f32x2 mul2(f32x2 a, f32x2 b)
{
    f32x2 d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}

template <int CK>
__device__ __forceinline__ void pack_fields8(const uint32_t (&t)[8], uint32_t &w0, uint32_t &w1);

// Two's complement codes of 8 residuals packed into words.  Each value is
// rounded to nearest even by the 1.5 * 2^23 adder trick, shifted to the
// non-negative range, and the fields are combined by exact fp32 Horner steps;
// a final xor turns the offset-binary fields into two's complement.  The
// result equals clamp(rint(r * inv), -qmax, qmax) field by field.
template <int CK, bool CLAMP>
__device__ __forceinline__ void quant_pack8(const float (&r)[8], float inv, uint32_t &w0, uint32_t &w1)
{
    constexpr float qm = (CK == CONEF_C_INT4) ? 7.f : 127.f;
    // t = x + 1.5 * 2^23 is rounded to the nearest-even integer, and its bit pattern is
    // 0x4B400000 + code as a two's-complement integer.  The fields are then combined by integer
    // shift-adds on the raw patterns: sum_q bits_q * 2^(B q) = sum_q code_q * 2^(B q) + K with a
    // constant K (mod 2^32); adding the offset-binary bias and one xor give two's-complement
    // fields.  Equals clamp(rint(r * inv), -qmax, qmax) field by field.
    uint32_t t[8];
#pragma unroll
    for (int q = 0; q < 8; ++q) {
        float x = __fmul_rn(r[q], inv);
        if (CLAMP)
            x = fminf(fmaxf(x, -qm), qm);
        t[q] = __float_as_uint(__fadd_rn(x, 12582912.0f));
    }
    pack_fields8<CK>(t, w0, w1);
}
// t[q] = bit pattern of rint(x_q) + 1.5 * 2^23 -> two's complement fields (see quant_pack8)
template <int CK>
__device__ __forceinline__ void pack_fields8(const uint32_t (&t)[8], uint32_t &w0, uint32_t &w1)
{
    if (CK == CONEF_C_INT4) {
        uint32_t acc = t[7];
#pragma unroll
        for (int q = 6; q >= 0; --q)
            acc = (acc << 4) + t[q];
        constexpr uint32_t K = 0x4B400000u * 0x11111111u;   // sum of the patterns' constant part, mod 2^32
        w0 = (acc - K + 0x88888888u) ^ 0x88888888u;
        w1 = 0;
    } else {
        uint32_t a0 = t[3], a1 = t[7];
#pragma unroll
        for (int q = 2; q >= 0; --q) {
            a0 = (a0 << 8) + t[q];
            a1 = (a1 << 8) + t[q + 4];
        }
        constexpr uint32_t K = 0x4B400000u * 0x01010101u;
        w0 = (a0 - K + 0x80808080u) ^ 0x80808080u;
        w1 = (a1 - K + 0x80808080u) ^ 0x80808080u;
    }
}

template <bool HALF>
__device__ __forceinline__ float load_scale_g(const uint8_t *scales, uint32_t blk)
{
    if (HALF)
        return __half2float(__ushort_as_half(*((const volatile unsigned short *)scales + blk)));
    return *((const volatile float *)scales + blk);
}

// scale and reciprocal of one block from its absmax (same arithmetic as quant_scale)
template <int CK, bool HALF>
__device__ __forceinline__ void block_scale(float amax, float &s, float &inv, unsigned short &hb)
{
    constexpr float qm = (CK == CONEF_C_INT8) ? 127.f : 7.f;
    // amax / qmax, correctly rounded, without the division routine: q = amax * c with
    // c = RN(1 / qmax), one exact remainder, one correction.  For qmax = 7 and 127 this equals
    // the IEEE quotient for every fp32 significand (checked exhaustively by
    // tests/test_division_by_constant.py); exponents do not matter as long as nothing
    // underflows, so tiny non-zero maxima take the division routine.
    // With a binary16 scale a maximum that small stores a zero scale whatever the quotient's last
    // bit is (anything below 2^-25 rounds to zero), so that case needs no branch.
    if (HALF || amax == 0.f || amax > 1e-30f) {
        constexpr float c = 1.0f / qm;
        const float q = __fmul_rn(amax, c);
        const float rem = __fmaf_rn(-qm, q, amax);
        s = __fmaf_rn(rem, c, q);
    } else {
        s = __fdiv_rn(amax, qm);
    }
    hb = 0;
    if (HALF) {
        const __half h = __float2half_rn(fminf(s, 65504.0f));
        hb = __half_as_ushort(h);
        s = __half2float(h);
    }
    const bool zero = !(s >= FLT_MIN);
    inv = __fdiv_rn(1.0f, zero ? 1.0f : s);   // (__frcp_rn gives the same value but was measured slower here)
    inv = zero ? 0.f : inv;
    s = zero ? 0.f : s;
    hb = zero ? (unsigned short)0 : hb;
}

}  // namespace conef
