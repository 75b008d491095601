// Lane-level encoders for HiF4 and MXFP4 (Section 3, "Block-Scaled Quantization").
//
// Thread mapping shared by every quantizer kernel: a lane owns 8 consecutive elements along K
// (one 128-bit load of bf16).  For HiF4 that is exactly one level-2 group and its two level-3
// groups, and the 8 lanes of an aligned octet own one block of 64; for MXFP4 the 4 lanes of an
// aligned quad own one block of 32.  Group maxima are register-local; only the block maximum
// crosses lanes (one redux per block).
#pragma once
#include "common.cuh"

namespace resq {

__device__ __forceinline__ float pow2_from_biased(int biased) {  // 2^(biased-127), biased in 1..254
    return __uint_as_float((uint32_t)biased << 23);
}

// Round |x| * inv to the nearest integer in 0..7, ties to even, saturating at 7.
// `inv` is fl(1/d) * 2^-j for a step d * 2^j with d in {4,5,6,7}: the product carries a relative
// error below 2^-22, so an exact tie can land one ulp off .5.  Inputs have at most 8 significant
// bits (bf16 activations, and residuals of bf16 activations), which keeps every non-tie at least
// 2^-9 away from a half-integer; snapping to a 2^-14 grid first therefore restores exact ties
// without creating new ones.  Returns the float whose low mantissa bits hold q.
__device__ __forceinline__ float rne_magic(float ax, float inv) {
    float r = fminf(__fmul_rn(ax, inv), 7.25f);
    r = __fadd_rn(__fadd_rn(r, 768.0f), -768.0f);  // 1.5 * 2^9: ulp 2^-14
    return __fadd_rn(r, 12582912.0f);              // 1.5 * 2^23: ulp 1, round to nearest even
}

// top-2-of-4 (Section 4.3, item (2)): keys are the 3-bit magnitudes of four codes packed in bits
// 15:0 of c (element i at bits 4i+2:4i, sign bits ignored).  Larger key wins, equal keys keep the
// lower index; exactly two bits of the result are set.
__device__ __forceinline__ uint32_t top2of4(uint32_t c) {
    int k0 = (int)(c & 7u) * 4 + 3;
    int k1 = (int)((c >> 4) & 7u) * 4 + 2;
    int k2 = (int)((c >> 8) & 7u) * 4 + 1;
    int k3 = (int)((c >> 12) & 7u) * 4;
    int g01 = k0 > k1, g02 = k0 > k2, g03 = k0 > k3, g12 = k1 > k2, g13 = k1 > k3, g23 = k2 > k3;
    int w0 = g01 + g02 + g03;
    int w1 = 1 - g01 + g12 + g13;
    int w2 = 2 - g02 - g12 + g23;
    int w3 = 3 - g03 - g13 - g23;
    return (uint32_t)((w0 >= 2) | ((w1 >= 2) << 1) | ((w2 >= 2) << 2) | ((w3 >= 2) << 3));
}

// ------------------------------------------------------------------------------------ HiF4
// x: the lane's 8 values.  grp_mask: the 8 lanes of this block.  lane8: lane index inside the octet.
// Out: codes (8 nibbles, element i at bits 4i+3:4i), meta (whole-block word, same in all 8 lanes),
// deq (signed decoded values, exact in fp32).
__device__ __forceinline__ void hif4_encode_lane(const float (&x)[8], unsigned grp_mask, int lane8,
                                                 uint32_t& codes, uint32_t& meta, float (&deq)[8]) {
    float m4a = fmaxf(fmaxf(fabsf(x[0]), fabsf(x[1])), fmaxf(fabsf(x[2]), fabsf(x[3])));
    float m4b = fmaxf(fmaxf(fabsf(x[4]), fabsf(x[5])), fmaxf(fabsf(x[6]), fabsf(x[7])));
    float m8 = fmaxf(m4a, m4b);
    // block maximum: non-negative floats order like their bit patterns
    uint32_t ab = __reduce_max_sync(grp_mask, __float_as_uint(m8));
    // level 1: smallest E6M2 code with 7*S1 >= amax.  7*S1 takes the values {28,35,42,49} * 2^(E-50),
    // i.e. inside the binade of amax = m * 2^p the candidates are m <= 1.09375, 1.3125, 1.53125, 1.75
    // (codes 4(p+45)+1 .. 4(p+45)+4) and, above 1.75, code 4(p+45)+5.
    int p = (int)(ab >> 23) - 127;
    uint32_t mant = ab & 0x7FFFFFu;
    int s = 4 * (p + 45) + 1 + (mant > 0x0C0000u) + (mant > 0x280000u) + (mant > 0x440000u) + (mant > 0x600000u);
    s = min(max(s, 0), 255);
    int E = s >> 2, Mn = s & 3;
    float d = (float)(4 + Mn);
    float S1 = d * pow2_from_biased(E - 50 + 127);  // (4+Mn) * 2^(E-50)
    // levels 2 and 3: raise an exponent exactly when the group would clip without it
    int e2 = m8 > 3.5f * S1;
    float thr3 = 1.75f * S1 * (e2 ? 2.0f : 1.0f);
    int e3a = m4a > thr3, e3b = m4b > thr3;
    uint32_t mine = ((uint32_t)e2 << (8 + lane8)) | ((uint32_t)(e3a | (e3b << 1)) << (16 + 2 * lane8));
    meta = __reduce_or_sync(grp_mask, mine) | (uint32_t)s;
    // elements: step = (4+Mn) * 2^(E-52+e2+e3)
    float rcp_d = Mn == 0 ? 0.25f : (Mn == 1 ? 0.2f : (Mn == 2 ? (1.0f / 6.0f) : (1.0f / 7.0f)));
    int ja = E - 52 + e2 + e3a, jb = E - 52 + e2 + e3b;
    float step_a = d * pow2_from_biased(ja + 127), step_b = d * pow2_from_biased(jb + 127);
    float inv_a = rcp_d * pow2_from_biased(127 - ja), inv_b = rcp_d * pow2_from_biased(127 - jb);
    uint32_t c = 0;
#pragma unroll
    for (int i = 7; i >= 0; --i) {
        float step = i < 4 ? step_a : step_b;
        float inv = i < 4 ? inv_a : inv_b;
        float t = rne_magic(fabsf(x[i]), inv);
        uint32_t xb = __float_as_uint(x[i]);
        uint32_t nib = (__float_as_uint(t) & 7u) | ((xb >> 28) & 8u);
        c = c * 16u + nib;
        float qf = __fadd_rn(t, -12582912.0f);
        deq[i] = copysignf(__fmul_rn(qf, step), x[i]);
    }
    codes = c;
}

// decode one nibble word with its block meta (used by the dequantize helper)
__device__ __forceinline__ void hif4_decode_lane(uint32_t codes, uint32_t meta, int lane8, float (&v)[8]) {
    int s = meta & 255;
    int E = s >> 2, Mn = s & 3;
    int e2 = (meta >> (8 + lane8)) & 1;
    int e3a = (meta >> (16 + 2 * lane8)) & 1, e3b = (meta >> (17 + 2 * lane8)) & 1;
    float d = (float)(4 + Mn);
    float step_a = d * pow2_from_biased(E - 52 + e2 + e3a + 127), step_b = d * pow2_from_biased(E - 52 + e2 + e3b + 127);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        uint32_t nib = (codes >> (4 * i)) & 15u;
        float mag = (float)(nib & 7u) * (i < 4 ? step_a : step_b);
        v[i] = (nib & 8u) ? -mag : mag;
    }
}

// ------------------------------------------------------------------------------------ MXFP4
__device__ __forceinline__ float e8m0_to_float(int sc) {  // 2^(sc-127); sc = 0 is the fp32 subnormal 2^-127
    return __uint_as_float(sc == 0 ? 0x00400000u : ((uint32_t)sc << 23));
}

// grp_mask: the 4 lanes of this block of 32.  scale: E8M0 code (same in the 4 lanes).
__device__ __forceinline__ void mxfp4_encode_lane(const float (&x)[8], unsigned grp_mask, uint32_t& codes,
                                                  uint32_t& scale, float (&deq)[8]) {
    float m8 = 0.0f;
#pragma unroll
    for (int i = 0; i < 8; ++i) m8 = fmaxf(m8, fabsf(x[i]));
    uint32_t ab = __reduce_max_sync(grp_mask, __float_as_uint(m8));
    // shared exponent: floor(log2 amax) - 2 (2 = exponent of E2M1's largest value), clamped to E8M0
    int sc = max((int)(ab >> 23) - 2, 0);
    scale = (uint32_t)sc;
    float inv = pow2_from_biased(254 - sc);  // 2^(127-sc), exact
    float sf = e8m0_to_float(sc);
    uint32_t c = 0;
#pragma unroll
    for (int i = 3; i >= 0; --i) {
        float lo = __fmul_rn(x[2 * i], inv), hi = __fmul_rn(x[2 * i + 1], inv);  // exact scalings
        uint16_t packed;
        // hardware E2M1 conversion: round to nearest even, saturate to +-6; first source -> high nibble
        asm("{ .reg .b8 t; cvt.rn.satfinite.e2m1x2.f32 t, %1, %2; mov.b16 %0, {t, 0}; }"
            : "=h"(packed) : "f"(hi), "f"(lo));
        uint32_t h2;
        asm("{ .reg .b8 t, z; mov.b16 {t, z}, %1; cvt.rn.f16x2.e2m1x2 %0, t; }" : "=r"(h2) : "h"(packed));
        __half2 hv = *reinterpret_cast<__half2*>(&h2);
        deq[2 * i] = __fmul_rn(__low2float(hv), sf);
        deq[2 * i + 1] = __fmul_rn(__high2float(hv), sf);
        c = (c << 8) | (uint32_t)(packed & 0xFF);
    }
    codes = c;
}

__device__ __forceinline__ void mxfp4_decode_lane(uint32_t codes, uint32_t sc, float (&v)[8]) {
    float sf = e8m0_to_float((int)sc);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        uint32_t nib = (codes >> (4 * i)) & 15u;
        uint32_t k = nib & 7u;
        // E2M1 magnitudes 0, .5, 1, 1.5, 2, 3, 4, 6 as 2*value in a byte table
        float mag = 0.5f * (float)((0x0C08060403020100ull >> (8 * k)) & 0xFFull);
        v[i] = ((nib & 8u) ? -mag : mag) * sf;
    }
}

}  // namespace resq
