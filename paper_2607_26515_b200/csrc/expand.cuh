// Expansion of packed 4-bit weight codes to bf16 (exact), shared by the GEMM kernels.
#pragma once
#include <stdint.h>
#include <cuda_runtime.h>

namespace resq {

// Expand one 32-bit word of 8 HiF4 codes (one level-2 group) into 8 bf16 values (one 16-byte chunk).
// bf16x2 trick: (0x4300 | q) is the bf16 number 128+q and (0x4300 | q<<4) is 128+16q, so one packed
// FMA with (scale, scale/16) and (-128 scale, -8 scale) yields q*scale exactly for both nibbles of a
// byte; the sign bits are then XOR-ed in.  Per pair of elements: one byte permute, one logic op, one
// packed FMA, one logic op.
// The scale words are linear in the metadata fields: with v = (s << 5) + (77 << 7) + ((e2 + e3) << 7) the bf16 bits of the
// scale (s << 5 already is (E << 7) | (Mn << 5)), the word (scale, scale / 16) is v * 0x10001 - 0x02000000 =
// s * 0x00200020 + (e2 + e3) * 0x00800080 + 0x24802680.  They are formed by integer multiply-adds (which run beside the
// integer-ALU pipe that the element work below saturates) from three single-bit extractions.
__device__ __forceinline__ uint32_t mad_u32(uint32_t a, uint32_t b, uint32_t c) {
    uint32_t r;
    asm("mad.lo.u32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(c));
    return r;
}
__device__ __forceinline__ uint4 expand_hif4_chunk(uint32_t c, uint32_t meta, int chunk) {
    const uint32_t e2 = (meta >> (8 + chunk)) & 1u;
    const uint32_t e3 = (meta >> (16 + 2 * chunk)) & 3u;
    const uint32_t base = mad_u32(e2, 0x00800080u, mad_u32(meta & 255u, 0x00200020u, 0x24802680u));
    const uint32_t scale_a = mad_u32(e3 & 1u, 0x00800080u, base);  // (scale, scale / 16)
    const uint32_t scale_b = mad_u32(e3 >> 1, 0x00800080u, base);
    const uint32_t add_a = mad_u32(e3 & 1u, 0x00800080u, base + 0x83808380u);  // -(128 * scale) in both halves
    const uint32_t add_b = mad_u32(e3 >> 1, 0x00800080u, base + 0x83808380u);
    const uint32_t c4 = c << 4;
    uint32_t out[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        // w: byte i of c in bytes 0, 2 and 3; byte i of (c << 4) in byte 1.  Bits 2:0 and 22:20 are the two
        // magnitudes; bit 15 is the sign of the even element, bit 31 the sign of the odd one.
        const uint32_t w = __byte_perm(c, c4, (uint32_t)(i | ((4 + i) << 4) | (i << 8) | (i << 12)));
        const uint32_t t = (w & 0x00700007u) | 0x43004300u;
        uint32_t v;
        asm("fma.rn.bf16x2 %0, %1, %2, %3;" : "=r"(v) : "r"(t), "r"(i < 2 ? scale_a : scale_b), "r"(i < 2 ? add_a : add_b));
        out[i] = v ^ (w & 0x80008000u);
    }
    return make_uint4(out[0], out[1], out[2], out[3]);
}

// MXFP4: expand 8 E2M1 codes with their E8M0 block scale `sc` (2^(sc-127)).  The eight E2M1 magnitudes
// 0, .5, 1, 1.5, 2, 3, 4, 6 are bf16 values whose high / low bytes come from two 8-entry byte tables
// indexed with a byte permute; the power-of-two scale is applied with an exact packed multiply.
__device__ __forceinline__ uint4 expand_mxfp4_chunk(uint32_t c, uint32_t sc) {
    // bf16(2^(sc-127)): exponent field sc; sc = 0 is the subnormal 2^-127 (mantissa bit 6)
    const uint32_t s16 = sc == 0 ? 0x0040u : (sc << 7);
    const uint32_t scale = s16 * 0x10001u;
    const uint32_t c4 = c << 4;
    uint32_t out[4];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const uint32_t sel = (c >> (16 * h)) & 0x7777u;                 // four magnitude indices
        const uint32_t hi4 = __byte_perm(0x3F3F3F00u, 0x40404040u, sel);  // high bytes of the four bf16 values
        const uint32_t lo4 = __byte_perm(0xC0800000u, 0xC0804000u, sel);  // low bytes
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const int i = 2 * h + j;  // byte of c holding this pair
            uint32_t v = __byte_perm(lo4, hi4, j == 0 ? 0x5140u : 0x7362u);
            asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(v) : "r"(v), "r"(scale));
            const uint32_t w = __byte_perm(c, c4, (uint32_t)(i | ((4 + i) << 4) | (i << 8) | (i << 12)));
            out[i] = v ^ (w & 0x80008000u);
        }
    }
    return make_uint4(out[0], out[1], out[2], out[3]);
}

}  // namespace resq
