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
// without creating new ones.  The snap is the rounding of the fused multiply-add itself
// (768 + r has ulp 2^-14); the second add rounds to an integer with ties to even.
// Returns u = 1.5 * 2^23 + q: the low mantissa bits hold q (bit 3 is clear).
constexpr float kMagicInt = 12582912.0f;  // 1.5 * 2^23
__device__ __forceinline__ float rne_magic(float ax, float inv) {
    float t = fminf(__fmaf_rn(ax, inv, 768.0f), 775.25f);  // 768 = 1.5 * 2^9; clamp keeps q <= 7
    return __fadd_rn(t, kMagicInt - 768.0f);
}
// Sum over i of 16^i (or 8^i for four 3-bit keys) of the magic constant's bit pattern, modulo 2^32: what an
// integer multiply-accumulate over the raw float bits adds on top of the packed digits.
constexpr uint32_t kMagicBits = 0x4B400000u;
constexpr uint32_t kNibbleBias = (uint32_t)(((uint64_t)kMagicBits * 0x11111111ull) & 0xFFFFFFFFull);
constexpr uint32_t kOctalBias = (uint32_t)(((uint64_t)kMagicBits * (1ull + 8ull + 64ull + 512ull)) & 0xFFFFFFFFull);

// top-n-of-4 (Section 4.3, item (2) is n = 2): keys are four 3-bit magnitudes.  Larger key wins, equal keys keep
// the lower index; exactly n bits of the result are set.
__host__ __device__ constexpr uint32_t topnof4_keys(int q0, int q1, int q2, int q3, int n) {
    const int k0 = q0 * 4 + 3, k1 = q1 * 4 + 2, k2 = q2 * 4 + 1, k3 = q3 * 4;
    const int w0 = (k0 > k1) + (k0 > k2) + (k0 > k3);
    const int w1 = (k1 > k0) + (k1 > k2) + (k1 > k3);
    const int w2 = (k2 > k0) + (k2 > k1) + (k2 > k3);
    const int w3 = (k3 > k0) + (k3 > k1) + (k3 > k2);
    const int need = 4 - n;  // an element is kept if it beats at least this many of the others
    return (uint32_t)((w0 >= need) | ((w1 >= need) << 1) | ((w2 >= need) << 2) | ((w3 >= need) << 3));
}
__host__ __device__ constexpr uint32_t top2of4_keys(int q0, int q1, int q2, int q3) { return topnof4_keys(q0, q1, q2, q3, 2); }
// c: four 4-bit codes (element i at bits 4i+2:4i, sign bits ignored).
__device__ __forceinline__ uint32_t top2of4(uint32_t c) {
    return top2of4_keys((int)(c & 7u), (int)((c >> 4) & 7u), (int)((c >> 8) & 7u), (int)((c >> 12) & 7u));
}
// The same as a 4096-entry table indexed by q0 | q1<<3 | q2<<6 | q3<<9, built at compile time: the keep nibbles of
// n = 1, 2, 3 in bits 3:0, 7:4, 11:8 of an entry.
struct TopNTable {
    uint16_t v[4096];
    constexpr TopNTable() : v() {
        for (int i = 0; i < 4096; ++i) {
            const int q0 = i & 7, q1 = (i >> 3) & 7, q2 = (i >> 6) & 7, q3 = (i >> 9) & 7;
            v[i] = (uint16_t)(topnof4_keys(q0, q1, q2, q3, 1) | (topnof4_keys(q0, q1, q2, q3, 2) << 4) |
                              (topnof4_keys(q0, q1, q2, q3, 3) << 8));
        }
    }
};
__device__ const TopNTable kTopNTable{};

// ------------------------------------------------------------------------------------ HiF4
// x: the lane's 8 values.  grp_mask: the 8 lanes of this block.  lane8: lane index inside the octet.
// Out: codes (8 nibbles, element i at bits 4i+3:4i), meta (whole-block word, same in all 8 lanes),
// deq (signed decoded values, exact in fp32), oct (q0 | q1<<3 | q2<<6 | q3<<9 of elements 0..3 in bits 11:0
// and of elements 4..7 in bits 27:16: the indices of the top-2-of-4 table).
__device__ __forceinline__ void hif4_encode_lane(const float (&x)[8], unsigned grp_mask, int lane8,
                                                 uint32_t& codes, uint32_t& meta, float (&deq)[8], uint32_t& oct) {
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
    const uint32_t E = (uint32_t)s >> 2, Mn = (uint32_t)s & 3u;
    // (4+Mn) * 2^x as fp32 bits: exponent field x + 2 + 127, top mantissa bits Mn
    const uint32_t dbits = Mn << 21;
    const float S1 = __uint_as_float(((E + 79u) << 23) | dbits);          // (4+Mn) * 2^(E-50)
    // levels 2 and 3: raise an exponent exactly when the group would clip without it
    const uint32_t e2 = m8 > 3.5f * S1;
    const float thr3 = 1.75f * __uint_as_float(((E + 79u + e2) << 23) | dbits);
    const uint32_t e3a = m4a > thr3, e3b = m4b > thr3;
    const uint32_t mine = (e2 << (8 + lane8)) | ((e3a | (e3b << 1)) << (16 + 2 * lane8));
    meta = __reduce_or_sync(grp_mask, mine) | (uint32_t)s;
    // elements: step = (4+Mn) * 2^(E-52+e2+e3); inv = fl(1/(4+Mn)) * 2^-(E-52+e2+e3) by exponent arithmetic
    const uint32_t rcp_bits = Mn == 0 ? 0x3E800000u : (Mn == 1 ? 0x3E4CCCCDu : (Mn == 2 ? 0x3E2AAAABu : 0x3E124925u));
    const uint32_t ea = E + 77u + e2 + e3a, eb = E + 77u + e2 + e3b;        // biased exponent of 2^(j+2)
    const float step_a = __uint_as_float((ea << 23) | dbits), step_b = __uint_as_float((eb << 23) | dbits);
    const float inv_a = __uint_as_float(rcp_bits - ((ea - 129u) << 23)), inv_b = __uint_as_float(rcp_bits - ((eb - 129u) << 23));
    uint32_t c = 0, oa = 0, ob = 0;
#pragma unroll
    for (int i = 7; i >= 0; --i) {
        const float step = i < 4 ? step_a : step_b;
        const float inv = i < 4 ? inv_a : inv_b;
        const float u = rne_magic(fabsf(x[i]), inv);
        const uint32_t ub = __float_as_uint(u);
        c = c * 16u + (ub | ((__float_as_uint(x[i]) >> 28) & 8u));
        if (i < 4) oa = oa * 8u + ub; else ob = ob * 8u + ub;
        const float qf = __fadd_rn(u, -kMagicInt);
        deq[i] = copysignf(__fmul_rn(qf, step), x[i]);
    }
    codes = c - kNibbleBias;
    oct = ((oa - kOctalBias) & 0xFFFu) | (((ob - kOctalBias) & 0xFFFu) << 16);
}

// ---- streaming variant of the same encoder, arranged for instruction count -----------------------------
// Sign bits of 8 elements as a nibble mask (bit 4e+3 for element e).  sw[i] carries the sign of element 2i
// in bit 15 and of element 2i+1 in bit 31 (a pair of bf16 values, or any word with those two bits).
__device__ __forceinline__ uint32_t sign_nibbles(const uint32_t (&sw)[4]) {
    const uint32_t p01 = __byte_perm(sw[0], sw[1], 0x7351);  // high bytes: e0, e2 | e1, e3
    const uint32_t p23 = __byte_perm(sw[2], sw[3], 0x7351);  //             e4, e6 | e5, e7
    const uint32_t ev = __byte_perm(p01, p23, 0x5410);       // e0 e2 e4 e6: sign in bit 7 of bytes 0..3
    const uint32_t od = __byte_perm(p01, p23, 0x7632);       // e1 e3 e5 e7
    return ((ev >> 4) & 0x08080808u) | (od & 0x80808080u);   // element 2k -> bit 8k+3, 2k+1 -> bit 8k+7
}

// Element loop.  cm: magnitudes q as 8 nibbles; dq: decoded magnitudes q * step (exact); oct as above.
// CLAMP is only needed when the level-1 code saturated (block maximum above 7 * S1max) or the block holds
// a non-finite value: otherwise the scale rule guarantees |x| / step <= 7.
template <bool CLAMP, bool DEQ, bool OCT>
__device__ __forceinline__ void hif4_round_elements(const float (&x)[8], float inv_a, float inv_b, float step_a,
                                                    float step_b, uint32_t& cm, float (&dq)[8], uint32_t& oct) {
    const float nms_a = __fmul_rn(-kMagicInt, step_a), nms_b = __fmul_rn(-kMagicInt, step_b);  // exact
    uint32_t c = 0, oa = 0, ob = 0;
#pragma unroll
    for (int i = 7; i >= 0; --i) {
        const float inv = i < 4 ? inv_a : inv_b;
        float t = __fmaf_rn(fabsf(x[i]), inv, 768.0f);
        if (CLAMP) t = fminf(t, 775.25f);
        const float u = __fadd_rn(t, kMagicInt - 768.0f);
        const uint32_t ub = __float_as_uint(u);
        c = c * 16u + ub;
        if (OCT) {
            if (i < 4) oa = oa * 8u + ub; else ob = ob * 8u + ub;
        }
        // (magic + q) * step - magic * step: the product is exact inside the fused multiply-add
        if (DEQ) dq[i] = __fmaf_rn(u, i < 4 ? step_a : step_b, i < 4 ? nms_a : nms_b);
    }
    cm = c - kNibbleBias;
    if (OCT) oct = ((oa - kOctalBias) & 0xFFFu) | (((ob - kOctalBias) & 0xFFFu) << 16);
}

constexpr uint32_t kHif4SatBits = 0x48C40000u;  // 401408 = 7 * 1.75 * 2^15: the largest block maximum level 1 covers

// Same results as hif4_encode_lane, except that `dq` holds decoded MAGNITUDES and the signs come from sw.
template <bool DEQ, bool OCT>
__device__ __forceinline__ void hif4_encode_stream(const float (&x)[8], const uint32_t (&sw)[4], unsigned grp_mask,
                                                   int lane8, uint32_t& codes, uint32_t& meta, float (&dq)[8],
                                                   uint32_t& oct) {
    const float m4a = fmaxf(fmaxf(fabsf(x[0]), fabsf(x[1])), fmaxf(fabsf(x[2]), fabsf(x[3])));
    const float m4b = fmaxf(fmaxf(fabsf(x[4]), fabsf(x[5])), fmaxf(fabsf(x[6]), fabsf(x[7])));
    const float m8 = fmaxf(m4a, m4b);
    const uint32_t ab = __reduce_max_sync(grp_mask, __float_as_uint(m8));
    const uint32_t mant = ab & 0x7FFFFFu;
    int s = 4 * (int)(ab >> 23) - 327 + (mant > 0x0C0000u) + (mant > 0x280000u) + (mant > 0x440000u) + (mant > 0x600000u);
    s = min(max(s, 0), 255);
    const uint32_t E = (uint32_t)s >> 2;
    const uint32_t dbits = ((uint32_t)s & 3u) << 21;
    const float S1 = __uint_as_float(((E + 79u) << 23) | dbits);          // (4+Mn) * 2^(E-50)
    const uint32_t e2 = m8 > 3.5f * S1;
    const float thr3 = 1.75f * __uint_as_float(((E + 79u + e2) << 23) | dbits);
    const uint32_t e3a = m4a > thr3, e3b = m4b > thr3;
    const uint32_t mine = (e2 << (8 + lane8)) | ((e3a | (e3b << 1)) << (16 + 2 * lane8));
    meta = __reduce_or_sync(grp_mask, mine) | (uint32_t)s;
    const float step_a = __uint_as_float(((E + 77u + e2 + e3a) << 23) | dbits);
    const float step_b = __uint_as_float(((E + 77u + e2 + e3b) << 23) | dbits);
    // 1/step to within one ulp: the rounding below snaps to a 2^-14 grid, far coarser than that error
    float inv_a, inv_b;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(inv_a) : "f"(step_a));
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(inv_b) : "f"(step_b));
    uint32_t cm;
    if (ab > kHif4SatBits) hif4_round_elements<true, DEQ, OCT>(x, inv_a, inv_b, step_a, step_b, cm, dq, oct);
    else hif4_round_elements<false, DEQ, OCT>(x, inv_a, inv_b, step_a, step_b, cm, dq, oct);
    codes = cm | sign_nibbles(sw);
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
