// Quantizer kernels: Q(X), dX = X - deq Q(X) (Eq. (3)), Q(dX) (Eq. (4)) and the selection S
// (Eq. (5), Section 4.3) in one pass over X; plus weight packing and the decode helper.
//
// All kernels stream X once with 128-bit loads and write packed 4-bit codes (32-bit stores), the
// block metadata, the mask bits and, for the GEMM, the exact bf16 images of the decoded operands.
// They are HBM-bound by design: nothing dense and wide is written except what the GEMM consumes.
#include "quant_device.cuh"

#include <algorithm>

namespace resq {

namespace {

constexpr int kWarpsPerCta = 8;
constexpr int kThreads = kWarpsPerCta * 32;
constexpr int kColsPerWarp = 256;  // 32 lanes x 8 elements

struct alignas(16) Bf16x8 {
    uint4 v;
};

__device__ __forceinline__ void unpack_bf16x8(const uint4& r, float (&x)[8]) {
    const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        x[2 * i] = __uint_as_float(w[i] << 16);
        x[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
}

__device__ __forceinline__ uint32_t pack_bf16x2_exact(float lo, float hi) {
    // the values are bf16-representable: truncation is exact
    return __byte_perm(__float_as_uint(lo), __float_as_uint(hi), 0x7632);
}

__device__ __forceinline__ uint4 ld_nc_16(const void* p) {
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
    return r;
}

// oct: the 3-bit magnitude keys of elements 0..3 in bits 11:0 and of elements 4..7 in bits 27:16
// (indices of the top-2-of-4 table).
template <int FMT>
__device__ __forceinline__ void encode_lane(const float (&x)[8], int lane, uint32_t& codes, uint32_t& side,
                                            float (&deq)[8], uint32_t& oct) {
    if (FMT == kHiF4) {
        unsigned m = 0xFFu << (lane & 24);
        hif4_encode_lane(x, m, lane & 7, codes, side, deq, oct);
    } else {
        unsigned m = 0xFu << (lane & 28);
        mxfp4_encode_lane(x, m, codes, side, deq);
        uint32_t o = 0;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            o |= ((codes >> (4 * i)) & 7u) << (3 * i);
            o |= ((codes >> (16 + 4 * i)) & 7u) << (16 + 3 * i);
        }
        oct = o;
    }
}

// keep mask of the lane's two groups of four; nsh = 4 * (n - 1) selects the n-of-4 nibble of the table entries
__device__ __forceinline__ uint32_t topn_mask8(uint32_t oct, int nsh) {
    return (((uint32_t)kTopNTable.v[oct & 0xFFFu] >> nsh) & 15u) | ((((uint32_t)kTopNTable.v[(oct >> 16) & 0xFFFu] >> nsh) & 15u) << 4);
}

template <int FMT>
__device__ __forceinline__ void store_side(void* side_ptr, int64_t row, int64_t K, int64_t k0, int lane, uint32_t side) {
    if (FMT == kHiF4) {
        if ((lane & 7) == 0) reinterpret_cast<uint32_t*>(side_ptr)[row * (K / kHif4Block) + k0 / kHif4Block] = side;
    } else {
        if ((lane & 3) == 0) reinterpret_cast<uint8_t*>(side_ptr)[row * (K / kMxBlock) + k0 / kMxBlock] = (uint8_t)side;
    }
}

// Per-pair keep masks for the bf16 image: word i is 0xFFFF in the half of every kept element of (2i, 2i+1).
// n * 0x10204080 puts bit j of a nibble n into the top bit of byte j; the permute then replicates those bits.
__device__ __forceinline__ void keep_words(uint32_t keep, uint32_t (&km)[4]) {
    const uint32_t zl = (keep & 15u) * 0x10204080u, zh = (keep >> 4) * 0x10204080u;
    // prmt selector nibbles with bit 3 set replicate the top bit of the selected byte
    asm("prmt.b32 %0, %1, 0, 0x9988;" : "=r"(km[0]) : "r"(zl));
    asm("prmt.b32 %0, %1, 0, 0xBBAA;" : "=r"(km[1]) : "r"(zl));
    asm("prmt.b32 %0, %1, 0, 0x9988;" : "=r"(km[2]) : "r"(zh));
    asm("prmt.b32 %0, %1, 0, 0xBBAA;" : "=r"(km[3]) : "r"(zh));
}

// 2:4 compression of four consecutive bf16 values held in two words whose dropped halves are already zero:
// returns the two kept values in channel order and the 4-bit index pair (idx0 | idx1 << 2) of the sparse MMA.
// `nib` has exactly two bits set (the top-2-of-4 table guarantees it).
__device__ __forceinline__ uint32_t compress24(uint32_t w0, uint32_t w1, uint32_t nib, uint32_t& idx) {
    const uint32_t i0 = (uint32_t)__ffs((int)nib) - 1u, i1 = 31u - (uint32_t)__clz((int)nib);
    idx = i0 | (i1 << 2);
    // halves 0..3 of (w0, w1) are bytes (2h, 2h + 1)
    return __byte_perm(w0, w1, (0x10u + 0x22u * i0) | ((0x10u + 0x22u * i1) << 8));
}

// Rows M .. (whole 256-row tiles) of the index metadata get a valid index pair (0, 1): the GEMM reads them next to
// zero-filled values.  Every 16-bit piece (one row, 16 channels) is written on its own.
__device__ __forceinline__ void fill_meta_pad(const QuantArgs& a, int64_t tid, int64_t nthreads) {
    const int64_t pad_rows = a.meta_rows128 * 128 - a.M;
    const int64_t pieces_per_row = a.meta_ka * 8;
    for (int64_t i = tid; i < pad_rows * pieces_per_row; i += nthreads) {
        const int64_t m = a.M + i / pieces_per_row, k = (i % pieces_per_row) * 16;
        *reinterpret_cast<uint16_t*>(a.r_meta + sparse24_meta_offset(m, k, a.meta_ka)) = (uint16_t)0x4444u;
    }
}

// ------------------------------------------------------------------------------------------------
// Streaming kernel for the patterns whose selection is local to a row segment (NONE, DENSE, 2:4) and
// first pass of the global ones (CHAN50, BLOCK: writes the unmasked residual and accumulates scores).
// grid.y: groups of 8 warps, each warp owning 256 channels; grid.x: row chunks of `rows_per_cta`.
// IMG: the bf16 images for the GEMM are written (a_bf16, and r_bf16 when RESIDUAL).
// Fused producer of the down projection: x = bf16(SiLU(g) * u).  Its rounding decides 4-bit codes, so the evaluation
// is fixed operation by operation (fp32, round to nearest even, no contraction into fused multiply-adds):
//   t = g * (-log2 e) clamped to [-126, 126]; n = rint(t); f = t - n; p = 2^f by the degree-6 Taylor polynomial of
//   exp(f ln 2) in Horner form; e = p * 2^n (= exp(-g)); s = g / (1 + e); x = bf16(s * u).
__device__ __forceinline__ float silu32(float g) {
    float t = __fmul_rn(g, -1.4426950408889634f);
    t = fminf(fmaxf(t, -126.0f), 126.0f);
    const float n = rintf(t);
    const float f = __fsub_rn(t, n);
    float p = 0.00015403530393381608f;
    p = __fadd_rn(__fmul_rn(p, f), 0.0013333558146428443f);
    p = __fadd_rn(__fmul_rn(p, f), 0.009618129107628477f);
    p = __fadd_rn(__fmul_rn(p, f), 0.05550410866482158f);
    p = __fadd_rn(__fmul_rn(p, f), 0.2402265069591007f);
    p = __fadd_rn(__fmul_rn(p, f), 0.6931471805599453f);
    p = __fadd_rn(__fmul_rn(p, f), 1.0f);
    const float e = __fmul_rn(p, __int_as_float(((int)n + 127) << 23));
    return __fdiv_rn(g, __fadd_rn(1.0f, e));
}
__device__ __forceinline__ uint4 swiglu_bf16x8(const uint4& graw, const uint4& uraw) {
    float g[8], u[8];
    unpack_bf16x8(graw, g);
    unpack_bf16x8(uraw, u);
    uint32_t o[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const __nv_bfloat162 v = __floats2bfloat162_rn(__fmul_rn(silu32(g[2 * i]), u[2 * i]), __fmul_rn(silu32(g[2 * i + 1]), u[2 * i + 1]));
        o[i] = *reinterpret_cast<const uint32_t*>(&v);
    }
    return make_uint4(o[0], o[1], o[2], o[3]);
}

// Fused RMSNorm producer, first kernel: r[m] = 1 / sqrt(sum_k X[m,k]^2 / K + eps).  The squares of bf16 values are
// exact; a warp sums its row in fp64 in a fixed order (lane-strided partial sums, then a shuffle tree), which is
// the exact sum except beyond 2^-40 relative; everything after the one rounding to fp32 is correctly rounded fp32.
__global__ void __launch_bounds__(256) rmsnorm_row_scale_kernel(const __nv_bfloat16* __restrict__ X, int64_t M, int64_t K, int64_t ldx,
                                                                float eps, float* __restrict__ row_scale) {
    pdl_wait();
    pdl_trigger();
    const int lane = threadIdx.x & 31;
    const int64_t m = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (m >= M) return;
    const __nv_bfloat16* row = X + m * ldx;
    double acc = 0.0;
    for (int64_t k = (int64_t)lane * 8; k < K; k += 256) {  // K is a multiple of 32, rows are 16-byte aligned
        float x[8];
        unpack_bf16x8(ld_nc_16(row + k), x);
#pragma unroll
        for (int i = 0; i < 8; ++i) acc += (double)x[i] * (double)x[i];
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
    if (lane == 0) {
        const float ss = (float)acc;  // round to nearest
        const float v = __fadd_rn(__fdiv_rn(ss, (float)K), eps);
        row_scale[m] = __fdiv_rn(1.0f, __fsqrt_rn(v));
    }
}

// Randomized Hadamard pre-transform of one block of 64 channels held by an aligned octet of lanes (8 values per
// lane): x' = bf16((1/8) H64 (s * x)).  In-place fast transform in fp32, strides 1, 2, 4 inside the lane and 8, 16, 32
// across lanes, each stage (a, b) -> (a + b, a - b) with a the lower channel; every operation rounded to nearest
// (no contraction), so the result is the same on every implementation that keeps this order.
__device__ __forceinline__ uint4 rht64_bf16x8(const uint4& raw, unsigned long long signs, int lane) {
    float v[8];
    unpack_bf16x8(raw, v);
    const uint32_t sb = (uint32_t)(signs >> (8 * (lane & 7))) & 0xFFu;
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = ((sb >> i) & 1u) ? -v[i] : v[i];
#pragma unroll
    for (int h = 1; h < 8; h <<= 1) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            if ((i & h) == 0) {
                const float a = v[i], b = v[i + h];
                v[i] = __fadd_rn(a, b);
                v[i + h] = __fsub_rn(a, b);
            }
        }
    }
#pragma unroll
    for (int d = 1; d < 8; d <<= 1) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const float other = __shfl_xor_sync(0xFFFFFFFFu, v[i], d);
            v[i] = (lane & d) ? __fsub_rn(other, v[i]) : __fadd_rn(v[i], other);
        }
    }
    uint32_t o[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const __nv_bfloat162 p = __floats2bfloat162_rn(__fmul_rn(v[2 * i], 0.125f), __fmul_rn(v[2 * i + 1], 0.125f));
        o[i] = *reinterpret_cast<const uint32_t*>(&p);
    }
    return make_uint4(o[0], o[1], o[2], o[3]);
}

// COMP (2:4 only): the residual image leaves in compressed form with its index metadata (a.r_comp, a.r_meta).
// PROD = 3: the input is the randomized Hadamard transform of X (rht64_bf16x8).  PROD = 1: the input is x = bf16(SiLU(g) * u) of a.X (g) and a.X_up (u); PROD = 2: x = bf16((X * r[m]) * gamma[k])
// with the row scales of rmsnorm_row_scale_kernel; computed on the fly, never stored.
// Body of the chunk-per-lane kernel for the CTA (bx, by) of a grid of gx x gy CTAs over one problem.
template <int FMT, bool RESIDUAL, bool IMG, bool COMP = false, int PROD = 0>
__device__ __forceinline__ void quant_stream_body(const QuantArgs& a, int rows_per_cta, int bx, int by, int gx, int gy) {
    if (a.clear_words && bx == 0 && by == 0)
        for (int i = threadIdx.x; i < a.n_clear_words; i += blockDim.x) a.clear_words[i] = 0u;
    if constexpr (COMP)
        fill_meta_pad(a, ((int64_t)by * gx + bx) * blockDim.x + threadIdx.x, (int64_t)gx * gy * blockDim.x);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t k0 = ((int64_t)by * kWarpsPerCta + warp) * kColsPerWarp + lane * 8;
    const bool active = k0 < a.K;  // whole blocks are active or not (K is a multiple of the block size)
    const int64_t m_begin = (int64_t)bx * rows_per_cta;
    const int64_t m_end = min(a.M, m_begin + rows_per_cta);
    const int pattern = a.pattern;
    const unsigned grp = FMT == kHiF4 ? 0xFFu << (lane & 24) : 0xFu << (lane & 28);
    const int lane8 = lane & 7;
    const bool side_lane = FMT == kHiF4 ? (lane & 7) == 0 : (lane & 3) == 0;
    const int64_t side_cols = a.K / (FMT == kHiF4 ? kHif4Block : kMxBlock);
    const int64_t side_k = k0 / (FMT == kHiF4 ? kHif4Block : kMxBlock);

    double chan_acc[8];
    double blk_acc = 0.0;
#pragma unroll
    for (int i = 0; i < 8; ++i) chan_acc[i] = 0.0;

    uint4 raw = make_uint4(0, 0, 0, 0), raw_up = make_uint4(0, 0, 0, 0);
    float gam[8];
    if constexpr (PROD == 2) {
        if (active) unpack_bf16x8(ld_nc_16(a.gamma + k0), gam);
    }
    if (active && m_begin < m_end) {
        raw = ld_nc_16(a.X + m_begin * a.ldx + k0);
        if constexpr (PROD == 1) raw_up = ld_nc_16(a.X_up + m_begin * a.ldx + k0);
    }
    for (int64_t m = m_begin; m < m_end; ++m) {
        uint4 cur = raw;
        if constexpr (PROD == 1) cur = swiglu_bf16x8(raw, raw_up);
        if constexpr (PROD == 3) cur = rht64_bf16x8(raw, a.rht_signs, lane);  // all lanes: the octets exchange values
        if constexpr (PROD == 2) {
            if (active) {
                const float r = a.row_scale[m];
                float h[8];
                unpack_bf16x8(raw, h);
                uint32_t o[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const __nv_bfloat162 v = __floats2bfloat162_rn(__fmul_rn(__fmul_rn(h[2 * i], r), gam[2 * i]),
                                                                   __fmul_rn(__fmul_rn(h[2 * i + 1], r), gam[2 * i + 1]));
                    o[i] = *reinterpret_cast<const uint32_t*>(&v);
                }
                cur = make_uint4(o[0], o[1], o[2], o[3]);
            }
        }
        if (active && m + 1 < m_end) {  // prefetch the next row
            raw = ld_nc_16(a.X + (m + 1) * a.ldx + k0);
            if constexpr (PROD == 1) raw_up = ld_nc_16(a.X_up + (m + 1) * a.ldx + k0);
        }
        const uint32_t w[4] = {cur.x, cur.y, cur.z, cur.w};
        float x[8], deq[8];
        unpack_bf16x8(cur, x);
        uint32_t codes, side, oct;
        if constexpr (FMT == kHiF4) {
            // deq holds magnitudes here; the signs are those of x
            hif4_encode_stream<RESIDUAL || IMG, false>(x, w, grp, lane8, codes, side, deq, oct);
        } else {
            encode_lane<FMT>(x, lane, codes, side, deq, oct);
        }
        if (active) {
            if (a.x_codes) *reinterpret_cast<uint32_t*>(a.x_codes + m * (a.K / 2) + k0 / 2) = codes;
            if (a.x_side && side_lane) {
                if (FMT == kHiF4) reinterpret_cast<uint32_t*>(a.x_side)[m * side_cols + side_k] = side;
                else reinterpret_cast<uint8_t*>(a.x_side)[m * side_cols + side_k] = (uint8_t)side;
            }
        }
        if constexpr (RESIDUAL && FMT == kHiF4) {
#pragma unroll
            for (int i = 0; i < 8; ++i) deq[i] = copysignf(deq[i], x[i]);
        }
        if constexpr (IMG) {
            if (active) {
                uint4 o;
                o.x = pack_bf16x2_exact(deq[0], deq[1]);
                o.y = pack_bf16x2_exact(deq[2], deq[3]);
                o.z = pack_bf16x2_exact(deq[4], deq[5]);
                o.w = pack_bf16x2_exact(deq[6], deq[7]);
                if constexpr (!RESIDUAL && FMT == kHiF4) {
                    o.x |= w[0] & 0x80008000u;
                    o.y |= w[1] & 0x80008000u;
                    o.z |= w[2] & 0x80008000u;
                    o.w |= w[3] & 0x80008000u;
                }
                *reinterpret_cast<uint4*>(a.a_bf16 + m * a.K + k0) = o;
            }
        }
        if constexpr (RESIDUAL) {
        // Eq. (3): the difference of a bf16 value and its decoded code is exact in fp32
        float dx[8], rdeq[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) dx[i] = __fsub_rn(x[i], deq[i]);
        uint32_t rcodes, rside, roct;
        uint32_t dw[4];  // signs of dx in bits 15 / 31
        if constexpr (FMT == kHiF4) {
#pragma unroll
            for (int i = 0; i < 4; ++i) dw[i] = pack_bf16x2_exact(dx[2 * i], dx[2 * i + 1]);
            hif4_encode_stream<true, true>(dx, dw, grp, lane8, rcodes, rside, rdeq, roct);  // rdeq: magnitudes
        } else {
            encode_lane<FMT>(dx, lane, rcodes, rside, rdeq, roct);
        }
        uint32_t keep = 0xFFu;
        if (pattern == RESQ_S_2_4) keep = topn_mask8(roct, 4 * (a.keep_quarters - 1));
        uint32_t comp0 = 0, comp1 = 0, idx_byte = 0;
        if constexpr (COMP) {
            {  // compressed image: 8 bytes per lane, and one byte of index pairs
                uint32_t km[4], o[4], ia, ib;
                keep_words(keep, km);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    o[i] = pack_bf16x2_exact(rdeq[2 * i], rdeq[2 * i + 1]);
                    if constexpr (FMT == kHiF4) o[i] |= dw[i] & 0x80008000u;
                    o[i] &= km[i];
                }
                comp0 = compress24(o[0], o[1], keep & 15u, ia);
                comp1 = compress24(o[2], o[3], keep >> 4, ib);
                idx_byte = ia | (ib << 4);
                // the even lane of a pair stores the 16-bit piece of 16 channels
                idx_byte |= __shfl_down_sync(0xFFFFFFFFu, idx_byte, 1) << 8;
            }
        }
        if (pattern == RESQ_S_CHAN50) {
#pragma unroll
            for (int i = 0; i < 8; ++i) chan_acc[i] += (double)rdeq[i] * (double)rdeq[i];
        } else if (pattern == RESQ_S_BLOCK32x64_50) {
            // squares have <= 12 significant bits; they are summed in fp64
#pragma unroll
            for (int i = 0; i < 8; ++i) blk_acc += (double)rdeq[i] * (double)rdeq[i];
            if (((m + 1) % kBlkRows) == 0 || m + 1 == m_end) {
                // one score per 32 x 64 block: reduce over the 8 lanes that share the 64 channels
                double v = blk_acc;
#pragma unroll
                for (int o = 1; o < 8; o <<= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
                if (active && (lane & 7) == 0)
                    atomicAdd(&a.scores[(m / kBlkRows) * (a.K / kBlkCols) + k0 / kBlkCols], v);
                blk_acc = 0.0;
            }
        }
        if (active) {
            if (a.r_codes) {
                uint32_t rc = rcodes;
                if (a.mask_r_codes) {  // operand form for the block-scaled FP4 GEMM: dropped entries become code 0
                    uint32_t nib = 0;
#pragma unroll
                    for (int i = 0; i < 8; ++i) nib |= ((keep >> i) & 1u) * (0xFu << (4 * i));
                    rc &= nib;
                }
                *reinterpret_cast<uint32_t*>(a.r_codes + m * (a.K / 2) + k0 / 2) = rc;
            }
            if (a.r_side && side_lane) {
                if (FMT == kHiF4) reinterpret_cast<uint32_t*>(a.r_side)[m * side_cols + side_k] = rside;
                else reinterpret_cast<uint8_t*>(a.r_side)[m * side_cols + side_k] = (uint8_t)rside;
            }
            const bool local = pattern == RESQ_S_DENSE || pattern == RESQ_S_2_4;
            if (a.mask_bits && local) a.mask_bits[m * (a.K / 8) + k0 / 8] = (uint8_t)keep;
            if constexpr (IMG) {
              if constexpr (COMP) {
                *reinterpret_cast<uint2*>(a.r_comp + m * (a.K / 2) + k0 / 2) = make_uint2(comp0, comp1);
                if ((lane & 1) == 0)
                    *reinterpret_cast<uint16_t*>(a.r_meta + sparse24_meta_offset(m, k0, a.meta_ka)) = (uint16_t)idx_byte;
              } else {
                // for the global patterns this is the unmasked image; the apply kernel zeroes dropped entries
                uint32_t km[4];
                keep_words(keep, km);
                uint4 o;
                o.x = pack_bf16x2_exact(rdeq[0], rdeq[1]);
                o.y = pack_bf16x2_exact(rdeq[2], rdeq[3]);
                o.z = pack_bf16x2_exact(rdeq[4], rdeq[5]);
                o.w = pack_bf16x2_exact(rdeq[6], rdeq[7]);
                if constexpr (FMT == kHiF4) {
                    o.x |= dw[0] & 0x80008000u;
                    o.y |= dw[1] & 0x80008000u;
                    o.z |= dw[2] & 0x80008000u;
                    o.w |= dw[3] & 0x80008000u;
                }
                o.x &= km[0];
                o.y &= km[1];
                o.z &= km[2];
                o.w &= km[3];
                *reinterpret_cast<uint4*>(a.r_bf16 + m * a.K + k0) = o;
              }
            }
        }
        }  // RESIDUAL
    }
    if (RESIDUAL && pattern == RESQ_S_CHAN50 && active) {
#pragma unroll
        for (int i = 0; i < 8; ++i) atomicAdd(&a.scores[k0 + i], chan_acc[i]);
    }
}

template <int FMT, bool RESIDUAL, bool IMG, bool COMP = false, int PROD = 0>
__global__ void __launch_bounds__(kThreads) quant_stream_kernel(QuantArgs a, int rows_per_cta) {
    pdl_wait();     // nothing below may touch global memory before the previous kernel of the stream is done
    pdl_trigger();  // the next kernel (the GEMM) may be scheduled and run its set-up
    quant_stream_body<FMT, RESIDUAL, IMG, COMP, PROD>(a, rows_per_cta, (int)blockIdx.x, (int)blockIdx.y, (int)gridDim.x, (int)gridDim.y);
}

// The same pass over a group of independent activations in one launch (the quantizer side of *_resq_linear_group):
// CTA b of the grid works on problem q with block_base[q] <= b < block_base[q + 1], as CTA (local % gx, local / gx) of
// that problem's own grid.
struct QuantGroup {
    QuantArgs a[kMaxQuantGroup];
    int rows_per_cta[kMaxQuantGroup], gx[kMaxQuantGroup], gy[kMaxQuantGroup];
    int block_base[kMaxQuantGroup + 1];
    int count;
};

template <int FMT, bool RESIDUAL, bool IMG, bool COMP>
__global__ void __launch_bounds__(kThreads) quant_stream_group_kernel(const __grid_constant__ QuantGroup g) {
    pdl_wait();
    pdl_trigger();
    int q = 0;
#pragma unroll 1
    while (q + 1 < g.count && (int)blockIdx.x >= g.block_base[q + 1]) ++q;
    const int local = (int)blockIdx.x - g.block_base[q];
    quant_stream_body<FMT, RESIDUAL, IMG, COMP, 0>(g.a[q], g.rows_per_cta[q], local % g.gx[q], local / g.gx[q], g.gx[q], g.gy[q]);
}

// ------------------------------------------------------------------------------------------------
// Block-per-lane streaming kernel (HiF4; NONE, DENSE, 2:4, BLOCK32x64).  A lane owns one whole block of 64
// values, so the block maximum, the level-1 scale and the metadata word need no cross-lane traffic and the
// scale set-up is paid once per 64 values instead of once per 8.  A warp owns 32 consecutive blocks (2048
// channels) of a row and walks down `rows_per_warp` rows.  Global accesses stay coalesced: rows arrive
// through a double-buffered cp.async stage in shared memory, each block padded to 144 bytes so that the
// 128-bit accesses of 8 neighbouring lanes fall on distinct banks; the bf16 images leave the same way.
constexpr int kStagePitch = 144;                 // bytes per staged block (128 + 16 padding)
constexpr int kStageBytes = 32 * kStagePitch;    // one row segment of a warp

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void cp_async_16(uint32_t dst, const void* src, bool valid) {
    const int n = valid ? 16 : 0;  // 0: the destination is zero-filled
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" :: "r"(dst), "l"(src), "r"(n) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" :: "n"(N) : "memory"); }

__device__ __forceinline__ uint4 lds_16(uint32_t addr) {
    uint4 r;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "r"(addr));
    return r;
}
__device__ __forceinline__ void sts_16(uint32_t addr, const uint4& v) {
    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" :: "r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ uint32_t max_u16x2(uint32_t a, uint32_t b) {
    uint32_t r;
    asm("max.u16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}

// Maxima of |v| over elements 0..3 and 4..7 of a chunk of 8 bf16 values, as bf16 bit patterns
// (non-negative bf16 values order like their bit patterns).
__device__ __forceinline__ void chunk_maxima(const uint32_t* w, uint32_t& mA, uint32_t& mB) {
    const uint32_t p = max_u16x2(w[0] & 0x7FFF7FFFu, w[1] & 0x7FFF7FFFu);
    const uint32_t q = max_u16x2(w[2] & 0x7FFF7FFFu, w[3] & 0x7FFF7FFFu);
    mA = max(p & 0xFFFFu, p >> 16);
    mB = max(q & 0xFFFFu, q >> 16);
}

// Level-1 scale of a block from its maximum (bf16 bits), plus what the per-group decisions need.
struct Hif4BlockScale {
    uint32_t s;          // level-1 code
    uint32_t base_bits;  // fp32 bits of the element step (4+Mn) * 2^(E-52) with both exponents 0
    uint32_t inv_bits;   // fp32 bits of 1/step (to within one ulp)
    uint32_t thr2;       // bf16 bits of 3.5 * S1: a level-2 group above it needs e2 = 1
    uint32_t thr3;       // bf16 bits of 1.75 * S1: a level-3 group above thr3 * 2^e2 needs e3 = 1
    bool saturated;      // the block maximum exceeds what code 255 covers (or is not finite)
};

__device__ __forceinline__ Hif4BlockScale hif4_block_scale(uint32_t amax16) {
    Hif4BlockScale b;
    const uint32_t ab = amax16 << 16;
    const uint32_t mant = ab & 0x7FFFFFu;
    int s = 4 * (int)(ab >> 23) - 327 + (mant > 0x0C0000u) + (mant > 0x280000u) + (mant > 0x440000u) + (mant > 0x600000u);
    s = min(max(s, 0), 255);
    b.s = (uint32_t)s;
    const uint32_t E = (uint32_t)s >> 2, dbits = ((uint32_t)s & 3u) << 21;
    const float S1 = __uint_as_float(((E + 79u) << 23) | dbits);  // (4+Mn) * 2^(E-50)
    b.thr2 = __float_as_uint(3.5f * S1) >> 16;                    // 14, 17.5, 21, 24.5 times a power of two: exact in bf16
    b.thr3 = __float_as_uint(1.75f * S1) >> 16;
    b.base_bits = ((E + 77u) << 23) | dbits;
    float inv;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(inv) : "f"(__uint_as_float(b.base_bits)));
    b.inv_bits = __float_as_uint(inv);
    b.saturated = ab > kHif4SatBits;
    return b;
}

// One chunk of 8 values (a level-2 group) of a block whose scale is known.  w: the values as bf16 pairs.
// Returns the 8 codes; meta_bits: this chunk's e2 / e3 bits at their place in the metadata word.
template <bool CLAMP, bool DEQ, bool OCT>
__device__ __forceinline__ uint32_t hif4_encode_chunk(const uint32_t* w, const Hif4BlockScale& b, uint32_t mA, uint32_t mB,
                                                      int c, uint32_t& meta_bits, float (&x)[8], float (&dq)[8],
                                                      uint32_t& oct) {
    const uint32_t e2 = max(mA, mB) > b.thr2;
    const uint32_t t3 = b.thr3 + (e2 << 7);  // bf16 exponent + e2
    const uint32_t e3a = mA > t3, e3b = mB > t3;
    meta_bits = (e2 << (8 + c)) | ((e3a | (e3b << 1)) << (16 + 2 * c));
    const uint32_t na = (e2 + e3a) << 23, nb = (e2 + e3b) << 23;
    const float step_a = __uint_as_float(b.base_bits + na), step_b = __uint_as_float(b.base_bits + nb);
    const float inv_a = __uint_as_float(b.inv_bits - na), inv_b = __uint_as_float(b.inv_bits - nb);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        x[2 * i] = __uint_as_float(w[i] << 16);
        x[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
    uint32_t cm;
    hif4_round_elements<CLAMP, DEQ, OCT>(x, inv_a, inv_b, step_a, step_b, cm, dq, oct);
    const uint32_t sw[4] = {w[0], w[1], w[2], w[3]};
    return cm | sign_nibbles(sw);
}

// Encode the lane's block held in w[32] (bf16 pairs).  Outputs the 8 code words and the metadata word.
// Per chunk, `sink(c, x, dq, oct)` receives the unpacked values, the decoded magnitudes and the top-2-of-4
// table indices (only what DEQ / OCT ask for is defined).
template <bool DEQ, bool OCT, typename Sink>
__device__ __forceinline__ void hif4_encode_block(const uint32_t (&w)[32], uint32_t (&codes)[8], uint32_t& meta, Sink&& sink) {
    uint32_t mA[8], mB[8];
    uint32_t amax = 0;
#pragma unroll
    for (int c = 0; c < 8; ++c) {
        chunk_maxima(&w[4 * c], mA[c], mB[c]);
        amax = max(amax, max(mA[c], mB[c]));
    }
    const Hif4BlockScale b = hif4_block_scale(amax);
    uint32_t m = b.s;
    if (b.saturated) {
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            float x[8], dq[8];
            uint32_t mb, oct = 0;
            codes[c] = hif4_encode_chunk<true, DEQ, OCT>(&w[4 * c], b, mA[c], mB[c], c, mb, x, dq, oct);
            m |= mb;
            sink(c, x, dq, oct);
        }
    } else {
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            float x[8], dq[8];
            uint32_t mb, oct = 0;
            codes[c] = hif4_encode_chunk<false, DEQ, OCT>(&w[4 * c], b, mA[c], mB[c], c, mb, x, dq, oct);
            m |= mb;
            sink(c, x, dq, oct);
        }
    }
    meta = m;
}

// MXFP4 counterpart: the lane's 64 values are two blocks of 32 (chunks 0..3 and 4..7), each with its own E8M0
// scale; `scales` returns the two scale bytes.  Same element arithmetic as mxfp4_encode_lane (hardware E2M1
// conversion of the exactly scaled values); dq: decoded magnitudes.
template <bool DEQ, bool OCT, typename Sink>
__device__ __forceinline__ void mxfp4_encode_block(const uint32_t (&w)[32], uint32_t (&codes)[8], uint32_t& scales, Sink&& sink) {
    uint32_t m8[8];
#pragma unroll
    for (int c = 0; c < 8; ++c) {
        uint32_t mA, mB;
        chunk_maxima(&w[4 * c], mA, mB);
        m8[c] = max(mA, mB);
    }
    scales = 0;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const uint32_t amax16 = max(max(m8[4 * h], m8[4 * h + 1]), max(m8[4 * h + 2], m8[4 * h + 3]));
        const int sc = max((int)(amax16 >> 7) - 2, 0);  // bf16 exponent field of the block maximum, minus E2M1's top exponent
        scales |= (uint32_t)sc << (8 * h);
        const float inv = pow2_from_biased(254 - sc);
        const float sf = e8m0_to_float(sc);
#pragma unroll
        for (int cc = 0; cc < 4; ++cc) {
            const int c = 4 * h + cc;
            float x[8], dq[8];
            uint32_t packed4 = 0;
#pragma unroll
            for (int i = 3; i >= 0; --i) {
                x[2 * i] = __uint_as_float(w[4 * c + i] << 16);
                x[2 * i + 1] = __uint_as_float(w[4 * c + i] & 0xFFFF0000u);
                const float lo = __fmul_rn(x[2 * i], inv), hi = __fmul_rn(x[2 * i + 1], inv);
                uint16_t pk;
                asm("{ .reg .b8 t; cvt.rn.satfinite.e2m1x2.f32 t, %1, %2; mov.b16 %0, {t, 0}; }" : "=h"(pk) : "f"(hi), "f"(lo));
                if (DEQ) {
                    uint32_t h2;
                    asm("{ .reg .b8 t, z; mov.b16 {t, z}, %1; cvt.rn.f16x2.e2m1x2 %0, t; }" : "=r"(h2) : "h"(pk));
                    const __half2 hv = *reinterpret_cast<__half2*>(&h2);
                    dq[2 * i] = fabsf(__fmul_rn(__low2float(hv), sf));
                    dq[2 * i + 1] = fabsf(__fmul_rn(__high2float(hv), sf));
                }
                packed4 = (packed4 << 8) | (uint32_t)(pk & 0xFF);
            }
            codes[c] = packed4;
            uint32_t oct = 0;
            if (OCT) {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    oct |= ((packed4 >> (4 * i)) & 7u) << (3 * i);
                    oct |= ((packed4 >> (16 + 4 * i)) & 7u) << (16 + 3 * i);
                }
            }
            sink(c, x, dq, oct);
        }
    }
}

template <int FMT, bool DEQ, bool OCT, typename Sink>
__device__ __forceinline__ void encode_block(const uint32_t (&w)[32], uint32_t (&codes)[8], uint32_t& side, Sink&& sink) {
    if constexpr (FMT == kHiF4) hif4_encode_block<DEQ, OCT>(w, codes, side, sink);
    else mxfp4_encode_block<DEQ, OCT>(w, codes, side, sink);
}

template <int FMT, bool RESIDUAL, bool IMG, bool COMP = false>
__global__ void __launch_bounds__(kThreads, 2) quant_block_kernel(QuantArgs a, int rows_per_warp) {
    pdl_wait();     // nothing below may touch global memory before the previous kernel of the stream is done
    pdl_trigger();  // the next kernel (the GEMM) may be scheduled and run its set-up
    if (a.clear_words && blockIdx.x == 0 && blockIdx.y == 0)
        for (int i = threadIdx.x; i < a.n_clear_words; i += blockDim.x) a.clear_words[i] = 0u;
    constexpr bool comp = COMP;  // 2:4: compressed residual image + index metadata
    if constexpr (comp) fill_meta_pad(a, (int64_t)blockIdx.x * blockDim.x + threadIdx.x, (int64_t)gridDim.x * blockDim.x);
    extern __shared__ __align__(16) uint8_t smem_q[];
    constexpr int kBufs = IMG ? 3 : 2;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t G = a.K / kHif4Block;
    const int64_t ncg = (G + 31) / 32;                       // column groups of 32 blocks
    const int64_t task = (int64_t)blockIdx.x * kWarpsPerCta + warp;
    const int64_t cg = task % ncg;
    const int64_t m_begin = (task / ncg) * rows_per_warp;
    const int64_t m_end = min(a.M, m_begin + rows_per_warp);
    if (m_begin >= m_end) return;                            // warps are independent: no CTA-wide barrier below
    const uint32_t in0 = smem_u32(smem_q) + (uint32_t)(warp * kBufs * kStageBytes);
    const uint32_t stage = in0 + 2 * kStageBytes;            // only with IMG
    const int pattern = a.pattern;
    const int nsh = 4 * (a.keep_quarters - 1);               // n-of-4 selection: which nibble of the table entries

    // cooperative row copies: piece j of lane l is chunk (l & 7) of block 4j + (l >> 3)
    const int cp_blk = lane >> 3, cp_ch = lane & 7;
    const uint32_t cp_smem = (uint32_t)(cp_blk * kStagePitch + cp_ch * 16);
    const int64_t cp_col = (cg * 32 + cp_blk) * kHif4Block + cp_ch * 8;  // first channel of piece 0
    auto issue_row = [&](int64_t m, uint32_t buf) {
        const __nv_bfloat16* src = a.X + m * a.ldx + cp_col;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const bool valid = cp_col + j * 4 * kHif4Block < a.K;
            cp_async_16(buf + cp_smem + j * 4 * kStagePitch, valid ? (const void*)(src + j * 4 * kHif4Block) : (const void*)a.X, valid);
        }
    };
    // write-out of a staged bf16 image row (same piece mapping)
    auto drain_stage = [&](__nv_bfloat16* dst_row) {
        __syncwarp();
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const uint4 v = lds_16(stage + cp_smem + j * 4 * kStagePitch);
            if (cp_col + j * 4 * kHif4Block < a.K) *reinterpret_cast<uint4*>(dst_row + cp_col + j * 4 * kHif4Block) = v;
        }
        __syncwarp();
    };
    // same for a staged compressed row (64 bytes per block): piece j of lane l is chunk (l & 3) of block 8j + (l >> 2)
    auto drain_stage_comp = [&](__nv_bfloat16* dst_row) {
        __syncwarp();
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int b = 8 * j + (lane >> 2);
            const uint4 v = lds_16(stage + (uint32_t)(b * kStagePitch + (lane & 3) * 16));
            if (cg * 32 + b < G) *reinterpret_cast<uint4*>(dst_row + (cg * 32 + b) * (kHif4Block / 2) + (lane & 3) * 8) = v;
        }
        __syncwarp();
    };

    const int64_t blk = cg * 32 + lane;  // the lane's block within the row
    const bool active = blk < G;
    const uint32_t my_in = (uint32_t)(lane * kStagePitch);
    double blk_acc = 0.0;

    issue_row(m_begin, in0);
    cp_async_commit();
    if (m_begin + 1 < m_end) issue_row(m_begin + 1, in0 + kStageBytes);
    cp_async_commit();
    for (int64_t m = m_begin; m < m_end; ++m) {
        const uint32_t buf = in0 + (uint32_t)(((m - m_begin) & 1) * kStageBytes);
        cp_async_wait<1>();
        __syncwarp();
        uint32_t w[32];
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            const uint4 v = lds_16(buf + my_in + c * 16);
            w[4 * c] = v.x; w[4 * c + 1] = v.y; w[4 * c + 2] = v.z; w[4 * c + 3] = v.w;
        }
        __syncwarp();
        if (m + 2 < m_end) issue_row(m + 2, buf);
        cp_async_commit();  // one group per row keeps the wait count uniform

        uint32_t codes[8], meta;
        // main encode; with RESIDUAL, w is overwritten by dX = X - deq Q(X) (Eq. (3)), exact in bf16
        encode_block<FMT, RESIDUAL || IMG, false>(w, codes, meta, [&](int c, const float (&x)[8], const float (&dq)[8], uint32_t) {
            if constexpr (RESIDUAL) {
                float sd[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) sd[i] = copysignf(dq[i], x[i]);
                if constexpr (IMG)
                    sts_16(stage + my_in + c * 16, make_uint4(pack_bf16x2_exact(sd[0], sd[1]), pack_bf16x2_exact(sd[2], sd[3]),
                                                              pack_bf16x2_exact(sd[4], sd[5]), pack_bf16x2_exact(sd[6], sd[7])));
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    w[4 * c + i] = pack_bf16x2_exact(__fsub_rn(x[2 * i], sd[2 * i]), __fsub_rn(x[2 * i + 1], sd[2 * i + 1]));
            } else if constexpr (IMG) {
                uint32_t img[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) img[i] = pack_bf16x2_exact(dq[2 * i], dq[2 * i + 1]) | (w[4 * c + i] & 0x80008000u);
                sts_16(stage + my_in + c * 16, make_uint4(img[0], img[1], img[2], img[3]));
            }
        });
        if (active) {
            if (a.x_codes) {
                uint4* p = reinterpret_cast<uint4*>(a.x_codes + m * (a.K / 2) + blk * 32);
                p[0] = make_uint4(codes[0], codes[1], codes[2], codes[3]);
                p[1] = make_uint4(codes[4], codes[5], codes[6], codes[7]);
            }
            if (a.x_side) {
                if constexpr (FMT == kHiF4) reinterpret_cast<uint32_t*>(a.x_side)[m * G + blk] = meta;
                else *reinterpret_cast<uint16_t*>(static_cast<uint8_t*>(a.x_side) + (m * G + blk) * 2) = (uint16_t)meta;
            }
        }
        if constexpr (IMG) drain_stage(a.a_bf16 + m * a.K);
        if constexpr (RESIDUAL) {
            uint32_t rcodes[8], rmeta, keep_lo = 0xFFFFFFFFu, keep_hi = 0xFFFFFFFFu;
            uint32_t idx_lo = 0, idx_hi = 0;  // comp: index pairs of channels 0..31 and 32..63 of the block
            float sq0 = 0.0f, sq1 = 0.0f;  // per 32 values: exact in fp32 for both formats (see below)
            encode_block<FMT, true, true>(w, rcodes, rmeta, [&](int c, const float (&)[8], const float (&rdq)[8], uint32_t roct) {
                uint32_t keep = 0xFFu;
                if (pattern == RESQ_S_2_4) {
                    keep = topn_mask8(roct, nsh);
                    if (c < 4) keep_lo = (keep_lo & ~(0xFFu << (8 * c))) | (keep << (8 * c));
                    else keep_hi = (keep_hi & ~(0xFFu << (8 * (c - 4)))) | (keep << (8 * (c - 4)));
                }
                if (pattern == RESQ_S_BLOCK32x64_50) {
                    // 32 squares of at most 12 significant bits whose exponents differ by at most 4 (HiF4) or that
                    // share one power-of-two scale (MXFP4): exact in fp32; the two halves may differ more (MXFP4)
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        if (c < 4) sq0 = __fmaf_rn(rdq[i], rdq[i], sq0);
                        else sq1 = __fmaf_rn(rdq[i], rdq[i], sq1);
                    }
                }
                if constexpr (IMG) {
                    // for BLOCK this is the unmasked image; the apply kernel zeroes dropped entries
                    uint32_t km[4];
                    keep_words(keep, km);
                    uint32_t img[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i)
                        img[i] = (pack_bf16x2_exact(rdq[2 * i], rdq[2 * i + 1]) | (w[4 * c + i] & 0x80008000u)) & km[i];
                    if constexpr (comp) {
                        uint32_t ia, ib;
                        const uint32_t c0 = compress24(img[0], img[1], keep & 15u, ia);
                        const uint32_t c1 = compress24(img[2], img[3], keep >> 4, ib);
                        asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(stage + my_in + c * 8), "r"(c0), "r"(c1) : "memory");
                        if (c < 4) idx_lo |= (ia | (ib << 4)) << (8 * c);
                        else idx_hi |= (ia | (ib << 4)) << (8 * (c - 4));
                    } else {
                        sts_16(stage + my_in + c * 16, make_uint4(img[0], img[1], img[2], img[3]));
                    }
                }
            });
            if (pattern == RESQ_S_BLOCK32x64_50) {
                blk_acc += (double)sq0 + (double)sq1;
                if (((m + 1) % kBlkRows) == 0 || m + 1 == m_end) {
                    if (active) atomicAdd(&a.scores[(m / kBlkRows) * G + blk], blk_acc);
                    blk_acc = 0.0;
                }
            }
            if (active) {
                if (a.r_codes) {
                    if (a.mask_r_codes) {  // operand form for the block-scaled FP4 GEMM: dropped entries become code 0
#pragma unroll
                        for (int c = 0; c < 8; ++c) {
                            const uint32_t keep = ((c < 4 ? keep_lo : keep_hi) >> (8 * (c & 3))) & 0xFFu;
                            uint32_t nib = 0;
#pragma unroll
                            for (int i = 0; i < 8; ++i) nib |= ((keep >> i) & 1u) * (0xFu << (4 * i));
                            rcodes[c] &= nib;
                        }
                    }
                    uint4* p = reinterpret_cast<uint4*>(a.r_codes + m * (a.K / 2) + blk * 32);
                    p[0] = make_uint4(rcodes[0], rcodes[1], rcodes[2], rcodes[3]);
                    p[1] = make_uint4(rcodes[4], rcodes[5], rcodes[6], rcodes[7]);
                }
                if (a.r_side) {
                    if constexpr (FMT == kHiF4) reinterpret_cast<uint32_t*>(a.r_side)[m * G + blk] = rmeta;
                    else *reinterpret_cast<uint16_t*>(static_cast<uint8_t*>(a.r_side) + (m * G + blk) * 2) = (uint16_t)rmeta;
                }
                const bool local = pattern == RESQ_S_DENSE || pattern == RESQ_S_2_4;
                if (a.mask_bits && local) *reinterpret_cast<uint2*>(a.mask_bits + m * (a.K / 8) + blk * 8) = make_uint2(keep_lo, keep_hi);
            }
            if constexpr (IMG) {
                if constexpr (comp) {
                    if (active) {
                        // four 16-bit pieces (16 channels each); consecutive pieces alternate between the two halves
                        // of a metadata block's row group and advance one 32-bit word every second piece
                        uint8_t* e = a.r_meta + sparse24_meta_offset(m, blk * kHif4Block, a.meta_ka);
                        *reinterpret_cast<uint16_t*>(e) = (uint16_t)idx_lo;
                        *reinterpret_cast<uint16_t*>(e + 128) = (uint16_t)(idx_lo >> 16);
                        *reinterpret_cast<uint16_t*>(e + 4) = (uint16_t)idx_hi;
                        *reinterpret_cast<uint16_t*>(e + 132) = (uint16_t)(idx_hi >> 16);
                    }
                    drain_stage_comp(a.r_comp + m * (a.K / 2));
                } else {
                    drain_stage(a.r_bf16 + m * a.K);
                }
            }
        }
    }
    cp_async_wait<0>();
}

// ------------------------------------------------------------------------------------------------
// ROW50 with a warp per row (block-per-lane encoders).  The row is walked in segments of 32 blocks; the signed
// bf16 image of deq Q(dX) of the whole row stays in the warp's shared memory (same padded block layout as the
// staging buffers), so that the K/2 largest magnitudes can be selected and the image masked before it leaves.
// Selection: most significant bit first over the 15 magnitude bits, counting with warp reductions only; ties
// at the threshold are kept lowest index first.  Shared memory per warp: (3 + segments) staging tiles.
// WPR = 1: a warp per row (rows of up to two segments, MAXSEG = 2).  WPR = 8 or 16: the warps of a CTA share one row,
// one segment per warp (MAXSEG = 1: fewer registers and two shared-memory tiles per warp, so that two 8-warp CTAs
// fit on an SM); the per-bit counts and the tie counts of the segments are summed through shared memory with one
// CTA barrier each.
template <int FMT, bool IMG, int WPR, int MAXSEG>
__global__ void __launch_bounds__(WPR == 16 ? 512 : kThreads, (WPR != 16 && MAXSEG == 1) ? 2 : 1)
quant_row50_warp_kernel(QuantArgs a, int warps_per_cta) {
    pdl_wait();
    pdl_trigger();
    if (a.clear_words && blockIdx.x == 0)
        for (int i = threadIdx.x; i < a.n_clear_words; i += blockDim.x) a.clear_words[i] = 0u;
    extern __shared__ __align__(16) uint8_t smem_q[];
    __shared__ int s_cnt[2][16];   // WPR > 1: candidates with bit b set, summed over the row's warps (alternating per row)
    __shared__ int s_ties[16];     // WPR > 1: entries equal to the threshold, per segment
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int wr = WPR == 1 ? 0 : warp;  // rank of the warp in its row's team
    if (WPR == 1 && warp >= warps_per_cta) return;  // warps are independent: no CTA-wide barrier below
    // WPR > 1: the CTA walks rows blockIdx.x, blockIdx.x + gridDim.x, ... and loads the next row while it selects
    int64_t m = WPR == 1 ? (int64_t)blockIdx.x * warps_per_cta + warp : (int64_t)blockIdx.x;
    const int64_t m_step = WPR == 1 ? a.M : (int64_t)gridDim.x;
    if (WPR == 1 && m >= a.M) return;
    if (WPR > 1) {
        if (threadIdx.x < 32) s_cnt[threadIdx.x >> 4][threadIdx.x & 15] = 0;
        __syncthreads();
    }
    const int64_t G = a.K / kHif4Block;
    const int nseg_row = (int)((G + 31) / 32);                                   // segments of the row
    const int nseg = WPR == 1 ? nseg_row : max(0, (nseg_row - wr + WPR - 1) / WPR);  // segments of this warp (at most 2)
    const int seg_cap = WPR == 1 ? nseg_row : (nseg_row + WPR - 1) / WPR;           // row-image tiles per warp
    auto gseg = [&](int ls) -> int { return wr + ls * WPR; };                      // local -> row segment
    // tiles per warp: two input stages, the image stage and the row image; with one segment per warp the input
    // tile doubles as the image stage (it is in registers before the encode writes the image)
    const uint32_t base = smem_u32(smem_q) + (uint32_t)(warp * (MAXSEG == 1 ? 2 : 3 + seg_cap) * kStageBytes);
    const uint32_t in0 = base, stage = MAXSEG == 1 ? base : base + 2 * kStageBytes,
                   rrow = MAXSEG == 1 ? base + kStageBytes : base + 3 * kStageBytes;
    const int cp_blk = lane >> 3, cp_ch = lane & 7;
    const uint32_t cp_smem = (uint32_t)(cp_blk * kStagePitch + cp_ch * 16);
    const uint32_t my_in = (uint32_t)(lane * kStagePitch);
    auto seg_col = [&](int seg) -> int64_t { return ((int64_t)seg * 32 + cp_blk) * kHif4Block + cp_ch * 8; };
    auto issue_seg = [&](int seg, uint32_t buf, int64_t row) {
        const int64_t col = seg_col(seg);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const bool valid = col + j * 4 * kHif4Block < a.K;
            cp_async_16(buf + cp_smem + j * 4 * kStagePitch,
                        valid ? (const void*)(a.X + row * a.ldx + col + j * 4 * kHif4Block) : (const void*)a.X, valid);
        }
    };
    auto drain = [&](uint32_t src, __nv_bfloat16* dst_row, int seg) {
        const int64_t col = seg_col(seg);
        __syncwarp();
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const uint4 v = lds_16(src + cp_smem + j * 4 * kStagePitch);
            if (col + j * 4 * kHif4Block < a.K) *reinterpret_cast<uint4*>(dst_row + col + j * 4 * kHif4Block) = v;
        }
        __syncwarp();
    };

    bool loaded = false;  // the first two segments of row m are already on their way
    for (int row_it = 0; m < a.M; m += m_step, ++row_it) {
    int* const cnt_row = s_cnt[row_it & 1];
    if (WPR > 1 && row_it > 0 && threadIdx.x < 16) s_cnt[(row_it + 1) & 1][threadIdx.x] = 0;  // for the next row
    // ---- phase A: both encodes, segment by segment
    if (!loaded) {
        if (nseg > 0) issue_seg(gseg(0), in0, m);
        cp_async_commit();
        if (nseg > 1) issue_seg(gseg(1), in0 + kStageBytes, m);
        cp_async_commit();
    }
    for (int ls = 0; ls < nseg; ++ls) {
        const int seg = gseg(ls);
        const uint32_t buf = in0 + (uint32_t)((ls & 1) * kStageBytes);
        cp_async_wait<1>();
        __syncwarp();
        uint32_t w[32];
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            const uint4 v = lds_16(buf + my_in + c * 16);
            w[4 * c] = v.x; w[4 * c + 1] = v.y; w[4 * c + 2] = v.z; w[4 * c + 3] = v.w;
        }
        __syncwarp();
        if (ls + 2 < nseg) issue_seg(gseg(ls + 2), buf, m);
        cp_async_commit();
        const int64_t blk = (int64_t)seg * 32 + lane;
        const bool active = blk < G;
        uint32_t codes[8], side;
        encode_block<FMT, true, false>(w, codes, side, [&](int c, const float (&x)[8], const float (&dq)[8], uint32_t) {
            float sd[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) sd[i] = copysignf(dq[i], x[i]);
            if constexpr (IMG)
                sts_16(stage + my_in + c * 16, make_uint4(pack_bf16x2_exact(sd[0], sd[1]), pack_bf16x2_exact(sd[2], sd[3]),
                                                          pack_bf16x2_exact(sd[4], sd[5]), pack_bf16x2_exact(sd[6], sd[7])));
#pragma unroll
            for (int i = 0; i < 4; ++i)
                w[4 * c + i] = pack_bf16x2_exact(__fsub_rn(x[2 * i], sd[2 * i]), __fsub_rn(x[2 * i + 1], sd[2 * i + 1]));
        });
        if (active) {
            if (a.x_codes) {
                uint4* p = reinterpret_cast<uint4*>(a.x_codes + m * (a.K / 2) + blk * 32);
                p[0] = make_uint4(codes[0], codes[1], codes[2], codes[3]);
                p[1] = make_uint4(codes[4], codes[5], codes[6], codes[7]);
            }
            if (a.x_side) {
                if constexpr (FMT == kHiF4) reinterpret_cast<uint32_t*>(a.x_side)[m * G + blk] = side;
                else *reinterpret_cast<uint16_t*>(static_cast<uint8_t*>(a.x_side) + (m * G + blk) * 2) = (uint16_t)side;
            }
        }
        if constexpr (IMG) drain(stage, a.a_bf16 + m * a.K, seg);
        uint32_t rcodes[8], rside;
        const uint32_t rdst = rrow + (uint32_t)(ls * kStageBytes) + my_in;
        encode_block<FMT, true, false>(w, rcodes, rside, [&](int c, const float (&)[8], const float (&rdq)[8], uint32_t) {
            uint32_t img[4];
#pragma unroll
            for (int i = 0; i < 4; ++i)
                img[i] = active ? (pack_bf16x2_exact(rdq[2 * i], rdq[2 * i + 1]) | (w[4 * c + i] & 0x80008000u)) : 0u;
            sts_16(rdst + c * 16, make_uint4(img[0], img[1], img[2], img[3]));
        });
        if (active) {
            if (a.r_codes) {
                uint4* p = reinterpret_cast<uint4*>(a.r_codes + m * (a.K / 2) + blk * 32);
                p[0] = make_uint4(rcodes[0], rcodes[1], rcodes[2], rcodes[3]);
                p[1] = make_uint4(rcodes[4], rcodes[5], rcodes[6], rcodes[7]);
            }
            if (a.r_side) {
                if constexpr (FMT == kHiF4) reinterpret_cast<uint32_t*>(a.r_side)[m * G + blk] = rside;
                else *reinterpret_cast<uint16_t*>(static_cast<uint8_t*>(a.r_side) + (m * G + blk) * 2) = (uint16_t)rside;
            }
        }
    }
    cp_async_wait<0>();
    __syncwarp();
    loaded = false;
    if (WPR > 1 && m + m_step < a.M) {  // the input staging tiles are free: the next row loads during phases B and C
        if (nseg > 0) issue_seg(gseg(0), in0, m + m_step);
        cp_async_commit();
        if (nseg > 1) issue_seg(gseg(1), in0 + kStageBytes, m + m_step);
        cp_async_commit();
        loaded = true;
    }

    // ---- phase B: the keep-th largest 15-bit magnitude of the row, on bit planes.  The lane's 64 magnitudes of a
    // segment are 32 words of two 16-bit halves: a 32 x 32 bit-matrix transpose turns them into planes -- word b
    // holds bit b of the even elements (element 2r at bit r), word 16 + b that of the odd elements.  The most-
    // significant-bit-first select then costs two population counts and a warp sum per bit; the sets "equal to the
    // threshold" and "greater" fall out as masks.
    constexpr int kMaxSeg = MAXSEG;               // segments per warp (the launcher picks the variant)
    uint32_t plane[kMaxSeg][32];
    uint32_t c_even[kMaxSeg], c_odd[kMaxSeg], g_even[kMaxSeg], g_odd[kMaxSeg];
#pragma unroll
    for (int seg = 0; seg < kMaxSeg; ++seg) {
        c_even[seg] = c_odd[seg] = g_even[seg] = g_odd[seg] = 0u;
        if (seg < nseg) {
            const uint32_t src = rrow + (uint32_t)(seg * kStageBytes) + my_in;
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const uint4 v = lds_16(src + c * 16);
                plane[seg][4 * c] = v.x; plane[seg][4 * c + 1] = v.y; plane[seg][4 * c + 2] = v.z; plane[seg][4 * c + 3] = v.w;
            }
            // transpose: afterwards bit r of word c is bit c of the former word r
#pragma unroll
            for (int lg = 4; lg >= 0; --lg) {
                const int j = 1 << lg;
                const uint32_t msk = j == 16 ? 0x0000FFFFu : j == 8 ? 0x00FF00FFu : j == 4 ? 0x0F0F0F0Fu : j == 2 ? 0x33333333u : 0x55555555u;
#pragma unroll
                for (int k = 0; k < 32; ++k) {
                    if ((k & j) == 0) {
                        const uint32_t t = ((plane[seg][k] >> j) ^ plane[seg][k + j]) & msk;
                        plane[seg][k] ^= t << j;
                        plane[seg][k + j] ^= t;
                    }
                }
            }
            const bool seg_active = (int64_t)gseg(seg) * 32 + lane < G;
            c_even[seg] = c_odd[seg] = seg_active ? 0xFFFFFFFFu : 0u;   // candidates: every element of an existing block
        }
    }
    int remaining = (int)(a.K * a.keep_quarters / 4);
#pragma unroll
    for (int b = 14; b >= 0; --b) {
        int cnt = 0;
#pragma unroll
        for (int seg = 0; seg < kMaxSeg; ++seg)
            if (seg < nseg) cnt += __popc(c_even[seg] & plane[seg][b]) + __popc(c_odd[seg] & plane[seg][16 + b]);
        cnt = __reduce_add_sync(0xFFFFFFFFu, cnt);
        if (WPR > 1) {
            if (lane == 0 && cnt) atomicAdd(&cnt_row[b], cnt);
            __syncthreads();
            cnt = cnt_row[b];
        }
        const bool take = cnt >= remaining;       // the threshold has this bit set: candidates without it fall below
        if (!take) remaining -= cnt;
#pragma unroll
        for (int seg = 0; seg < kMaxSeg; ++seg) {
            if (seg < nseg) {
                const uint32_t one_e = c_even[seg] & plane[seg][b], one_o = c_odd[seg] & plane[seg][16 + b];
                if (take) {
                    c_even[seg] = one_e;
                    c_odd[seg] = one_o;
                } else {                          // candidates with the bit are above the threshold
                    g_even[seg] |= one_e;
                    g_odd[seg] |= one_o;
                    c_even[seg] ^= one_e;
                    c_odd[seg] ^= one_o;
                }
            }
        }
    }
    int need = remaining;        // entries equal to the threshold that are kept, lowest index first
    // masks of even / odd elements -> element order (element e at bit e of a 64-bit mask)
    auto spread16 = [](uint32_t x) -> uint32_t {
        x &= 0xFFFFu;
        x = (x | (x << 8)) & 0x00FF00FFu;
        x = (x | (x << 4)) & 0x0F0F0F0Fu;
        x = (x | (x << 2)) & 0x33333333u;
        x = (x | (x << 1)) & 0x55555555u;
        return x;
    };

    // ---- phase C: masks in index order (segment, lane, position), masked image, masked codes
    const int need_row = need;
    if (WPR > 1) {  // ties of every segment of the row, so that each warp knows how many come before its segments
#pragma unroll
        for (int ls = 0; ls < kMaxSeg; ++ls)
            if (ls < nseg) {
                const int t = __reduce_add_sync(0xFFFFFFFFu, __popc(c_even[ls]) + __popc(c_odd[ls]));
                if (lane == 0) s_ties[gseg(ls)] = t;
            }
        __syncthreads();
    }
    for (int ls = 0; ls < nseg; ++ls) {
        const int seg = gseg(ls);
        if (WPR > 1) {
            int before = 0;
            for (int q = 0; q < seg; ++q) before += s_ties[q];
            need = max(0, need_row - before);
        }
        const int64_t blk = (int64_t)seg * 32 + lane;
        const bool active = blk < G;
        const uint32_t src = rrow + (uint32_t)(ls * kStageBytes) + my_in;
        uint32_t wv[32];
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            const uint4 v = lds_16(src + c * 16);
            wv[4 * c] = v.x; wv[4 * c + 1] = v.y; wv[4 * c + 2] = v.z; wv[4 * c + 3] = v.w;
        }
        // bit per element of the lane's block (low / high 32): greater than / equal to the threshold
        const uint32_t ce = ls == 0 ? c_even[0] : c_even[kMaxSeg - 1], co = ls == 0 ? c_odd[0] : c_odd[kMaxSeg - 1];
        const uint32_t ge = ls == 0 ? g_even[0] : g_even[kMaxSeg - 1], go = ls == 0 ? g_odd[0] : g_odd[kMaxSeg - 1];
        uint32_t gt[2] = {spread16(ge) | (spread16(go) << 1), spread16(ge >> 16) | (spread16(go >> 16) << 1)};
        uint32_t eq[2] = {spread16(ce) | (spread16(co) << 1), spread16(ce >> 16) | (spread16(co >> 16) << 1)};
        const int mine = __popc(eq[0]) + __popc(eq[1]);
        int incl = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
            if (lane >= o) incl += t;
        }
        const int total = __shfl_sync(0xFFFFFFFFu, incl, 31);
        int quota = max(0, min(mine, need - (incl - mine)));  // how many of this lane's ties are kept
        need = max(0, need - total);
        uint32_t keep[2] = {gt[0], gt[1]};
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            uint32_t e = eq[h];
            while (e && quota > 0) {  // lowest set bits first
                const uint32_t low = e & (0u - e);
                keep[h] |= low;
                e ^= low;
                --quota;
            }
        }
        if (active) {
            if (a.mask_bits) *reinterpret_cast<uint2*>(a.mask_bits + m * (a.K / 8) + blk * 8) = make_uint2(keep[0], keep[1]);
            if (a.r_codes && a.mask_r_codes) {
                uint4* p = reinterpret_cast<uint4*>(a.r_codes + m * (a.K / 2) + blk * 32);
                uint4 c0 = __ldcg(p), c1 = __ldcg(p + 1);
                uint32_t cw[8] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w};
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    const uint32_t k8 = (keep[c >> 2] >> (8 * (c & 3))) & 0xFFu;
                    uint32_t nib = 0;
#pragma unroll
                    for (int i = 0; i < 8; ++i) nib |= ((k8 >> i) & 1u) * (0xFu << (4 * i));
                    cw[c] &= nib;
                }
                p[0] = make_uint4(cw[0], cw[1], cw[2], cw[3]);
                p[1] = make_uint4(cw[4], cw[5], cw[6], cw[7]);
            }
        }
        if constexpr (IMG) {
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                uint32_t km[4];
                keep_words((keep[c >> 2] >> (8 * (c & 3))) & 0xFFu, km);
                sts_16(src + c * 16, make_uint4(wv[4 * c] & km[0], wv[4 * c + 1] & km[1], wv[4 * c + 2] & km[2], wv[4 * c + 3] & km[3]));
            }
            drain(rrow + (uint32_t)(ls * kStageBytes), a.r_bf16 + m * a.K, seg);
        }
    }
    }  // rows of this CTA
}

// ------------------------------------------------------------------------------------------------
// Exact top-`keep` of n non-negative fp64 scores, ties to the lower index.  One CTA: MSB-first radix
// select over the 64-bit patterns (8 passes of 8 bits), then an index-ordered pass that admits the
// first `need` entries equal to the threshold.
constexpr int kSelThreads = 1024;

// (All kSelThreads threads of a CTA call it; `flag` may point to global or to shared memory.)
__device__ __forceinline__ void topk_select_cta(const double* __restrict__ score, int n, int keep, uint8_t* flag) {
    __shared__ unsigned hist[256];
    __shared__ unsigned long long s_prefix;
    __shared__ int s_remaining;
    __shared__ int s_warp_count[kSelThreads / 32];
    __shared__ int s_base;
    const int tid = threadIdx.x;
    if (keep <= 0 || keep >= n) {
        for (int i = tid; i < n; i += kSelThreads) flag[i] = keep >= n ? 1 : 0;
        return;
    }
    if (tid == 0) {
        s_prefix = 0ull;
        s_remaining = keep;
    }
    __syncthreads();
    for (int shift = 56; shift >= 0; shift -= 8) {
        if (tid < 256) hist[tid] = 0u;
        __syncthreads();
        const unsigned long long prefix = s_prefix;
        // scores of one tensor mostly share their leading digits: lanes that hit the same bucket add once
        for (int i0 = 0; i0 < n; i0 += kSelThreads) {
            const int i = i0 + tid;
            unsigned long long key = i < n ? (unsigned long long)__double_as_longlong(score[i]) : 0ull;
            const bool match = i < n && (shift == 56 ? true : ((key ^ prefix) >> (shift + 8)) == 0ull);
            const unsigned bucket = match ? (unsigned)(key >> shift) & 255u : 0xFFFFFFFFu;
            const unsigned same = __match_any_sync(0xFFFFFFFFu, bucket);
            if (match && (unsigned)(__ffs((int)same) - 1) == (unsigned)(tid & 31)) atomicAdd(&hist[bucket], (unsigned)__popc(same));
        }
        __syncthreads();
        // pick the bucket that holds the remaining-th largest key: suffix sums of the histogram by one warp
        if (tid < 32) {
            const int remaining = s_remaining;
            // lane l owns buckets 8l .. 8l+7; above[l] = number of keys in buckets of higher lanes
            int mine = 0;
#pragma unroll
            for (int j = 0; j < 8; ++j) mine += (int)hist[8 * tid + j];
            int incl = mine;  // inclusive suffix sum over lanes >= l
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                int t = __shfl_down_sync(0xFFFFFFFFu, incl, o);
                if (tid + o < 32) incl += t;
            }
            const int above = incl - mine;
            const bool here = above < remaining && incl >= remaining;  // exactly one lane
            if (here) {
                int rem = remaining - above;
                int b = 8 * tid + 7;
                for (; b > 8 * tid; --b) {
                    int c = (int)hist[b];
                    if (c >= rem) break;
                    rem -= c;
                }
                s_prefix = prefix | ((unsigned long long)b << shift);
                s_remaining = rem;  // how many are still to be taken among keys sharing the new prefix
            }
        }
        __syncthreads();
    }
    const unsigned long long T = s_prefix;  // the keep-th largest key
    const int need = s_remaining;           // entries equal to T that are kept (lowest indices first)
    if (tid == 0) s_base = 0;
    __syncthreads();
    for (int i0 = 0; i0 < n; i0 += kSelThreads) {
        int i = i0 + tid;
        unsigned long long key = i < n ? (unsigned long long)__double_as_longlong(score[i]) : 0ull;
        bool eq = i < n && key == T;
        unsigned bal = __ballot_sync(0xFFFFFFFFu, eq);
        int lane = tid & 31, w = tid >> 5;
        if (lane == 0) s_warp_count[w] = __popc(bal);
        __syncthreads();
        int before = s_base;
        for (int j = 0; j < w; ++j) before += s_warp_count[j];
        before += __popc(bal & ((1u << lane) - 1u));
        if (i < n) flag[i] = (key > T || (eq && before < need)) ? 1 : 0;
        __syncthreads();
        if (tid == 0) {
            int tot = 0;
            for (int j = 0; j < kSelThreads / 32; ++j) tot += s_warp_count[j];
            s_base += tot;
        }
        __syncthreads();
    }
}

__global__ void __launch_bounds__(kSelThreads) topk_select_kernel(const double* __restrict__ score, int n, int keep,
                                                                 uint8_t* __restrict__ flag) {
    pdl_wait();     // the scores come from the quantizer kernel just before
    pdl_trigger();  // the mask pass may be scheduled (it waits for this kernel's flags)
    // one independent selection of n scores per CTA (a single CTA for the tensor-wide rules)
    topk_select_cta(score + (int64_t)blockIdx.x * n, n, keep, flag + (int64_t)blockIdx.x * n);
}

// Turn the kept-channel / kept-block flags into mask bits and zero the dropped entries of the GEMM's
// residual operand.  One thread per 8 channels of one row.
// One item of the mask pass: 8 consecutive channels of one row (`flag`: global or shared memory).
__device__ __forceinline__ void apply_mask_item(int64_t idx, int pattern, int64_t M, int64_t K, const uint8_t* flag,
                                                uint8_t* __restrict__ mask_bits, __nv_bfloat16* __restrict__ r_bf16,
                                                uint8_t* __restrict__ r_codes_masked) {
    int64_t per_row = K / 8;
    if (idx >= M * per_row) return;
    int64_t m = idx / per_row, k0 = (idx % per_row) * 8;
    uint32_t keep = 0;
    if (pattern == RESQ_S_CHAN50) {
        uint2 f = *reinterpret_cast<const uint2*>(flag + k0);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            keep |= ((f.x >> (8 * i)) & 1u) << i;
            keep |= ((f.y >> (8 * i)) & 1u) << (4 + i);
        }
    } else {
        keep = flag[(m / kBlkRows) * (K / kBlkCols) + k0 / kBlkCols] ? 0xFFu : 0u;
    }
    if (mask_bits) mask_bits[idx] = (uint8_t)keep;
    if (r_codes_masked && keep != 0xFFu) {  // operand form for the block-scaled FP4 GEMM: dropped entries become code 0
        uint32_t nib = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) nib |= ((keep >> i) & 1u) * (0xFu << (4 * i));
        uint32_t* c = reinterpret_cast<uint32_t*>(r_codes_masked + m * (K / 2) + k0 / 2);
        *c &= nib;
    }
    if (r_bf16 && keep != 0xFFu) {
        uint4* p = reinterpret_cast<uint4*>(r_bf16 + m * K + k0);
        uint4 v = keep == 0 ? make_uint4(0, 0, 0, 0) : *p;
        if (keep != 0) {
            uint32_t* w = reinterpret_cast<uint32_t*>(&v);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                uint32_t lo = (keep >> (2 * i)) & 1u ? 0x0000FFFFu : 0u;
                uint32_t hi = (keep >> (2 * i + 1)) & 1u ? 0xFFFF0000u : 0u;
                w[i] &= lo | hi;
            }
        }
        *p = v;
    }
}

__global__ void apply_global_mask_kernel(int pattern, int64_t M, int64_t K, const uint8_t* __restrict__ flag,
                                         uint8_t* __restrict__ mask_bits, __nv_bfloat16* __restrict__ r_bf16,
                                         uint8_t* __restrict__ r_codes_masked) {
    pdl_wait();     // the keep flags come from the selection kernel just before
    pdl_trigger();  // the GEMM may be scheduled and run its set-up
    apply_mask_item((int64_t)blockIdx.x * blockDim.x + threadIdx.x, pattern, M, K, flag, mask_bits, r_bf16, r_codes_masked);
}

// ------------------------------------------------------------------------------------------------
// ROW50: per row, keep the K/2 largest decoded magnitudes (ties: lower index).  One CTA per row: the
// row's decoded residual (bf16-exact, so its 15 magnitude bits order like the values) is staged in
// shared memory, a 2-pass radix select finds the threshold, an index-ordered pass resolves ties.
template <int FMT>
__global__ void __launch_bounds__(kThreads) quant_row50_kernel(QuantArgs a) {
    pdl_wait();     // nothing below may touch global memory before the previous kernel of the stream is done
    pdl_trigger();  // the next kernel (the GEMM) may be scheduled and run its set-up
    if (a.clear_words && blockIdx.x == 0 && blockIdx.y == 0)
        for (int i = threadIdx.x; i < a.n_clear_words; i += blockDim.x) a.clear_words[i] = 0u;
    extern __shared__ __align__(16) uint16_t s_r[];  // [K] signed bf16 image of deq Q(dX)
    __shared__ unsigned hist[256];
    __shared__ unsigned s_prefix;
    __shared__ int s_remaining;
    __shared__ int s_warp_count[kWarpsPerCta];
    __shared__ int s_base;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, tid = threadIdx.x;
    const int64_t m = blockIdx.x;
    const int64_t K = a.K;
    for (int64_t kb = (int64_t)warp * kColsPerWarp; kb < K; kb += (int64_t)kWarpsPerCta * kColsPerWarp) {
        const int64_t k0 = kb + lane * 8;
        const bool active = k0 < K;
        uint4 raw = make_uint4(0, 0, 0, 0);
        if (active) raw = ld_nc_16(a.X + m * a.ldx + k0);
        float x[8], deq[8], dx[8], rdeq[8];
        unpack_bf16x8(raw, x);
        uint32_t codes, side, rcodes, rside, oct;
        encode_lane<FMT>(x, lane, codes, side, deq, oct);
#pragma unroll
        for (int i = 0; i < 8; ++i) dx[i] = __fsub_rn(x[i], deq[i]);
        encode_lane<FMT>(dx, lane, rcodes, rside, rdeq, oct);
        if (active) {
            if (a.x_codes) *reinterpret_cast<uint32_t*>(a.x_codes + m * (K / 2) + k0 / 2) = codes;
            if (a.x_side) store_side<FMT>(a.x_side, m, K, k0, lane, side);
            if (a.r_codes) *reinterpret_cast<uint32_t*>(a.r_codes + m * (K / 2) + k0 / 2) = rcodes;
            if (a.r_side) store_side<FMT>(a.r_side, m, K, k0, lane, rside);
            uint4 o;
            if (a.a_bf16) {
                o.x = pack_bf16x2_exact(deq[0], deq[1]);
                o.y = pack_bf16x2_exact(deq[2], deq[3]);
                o.z = pack_bf16x2_exact(deq[4], deq[5]);
                o.w = pack_bf16x2_exact(deq[6], deq[7]);
                *reinterpret_cast<uint4*>(a.a_bf16 + m * K + k0) = o;
            }
            o.x = pack_bf16x2_exact(rdeq[0], rdeq[1]);
            o.y = pack_bf16x2_exact(rdeq[2], rdeq[3]);
            o.z = pack_bf16x2_exact(rdeq[4], rdeq[5]);
            o.w = pack_bf16x2_exact(rdeq[6], rdeq[7]);
            *reinterpret_cast<uint4*>(&s_r[k0]) = o;
        }
    }
    if (tid == 0) {
        s_prefix = 0u;
        s_remaining = (int)(K * a.keep_quarters / 4);
    }
    __syncthreads();
    // radix select on the 15-bit magnitude: bits 14:8 then 7:0
    for (int pass = 0; pass < 2; ++pass) {
        if (tid < 256) hist[tid] = 0u;
        __syncthreads();
        const unsigned prefix = s_prefix;
        for (int64_t k = tid; k < K; k += kThreads) {
            unsigned key = s_r[k] & 0x7FFFu;
            if (pass == 0) atomicAdd(&hist[key >> 8], 1u);
            else if ((key >> 8) == (prefix >> 8)) atomicAdd(&hist[key & 255u], 1u);
        }
        __syncthreads();
        if (tid == 0) {
            int remaining = s_remaining;
            int b = 255;
            for (; b > 0; --b) {
                int c = (int)hist[b];
                if (c >= remaining) break;
                remaining -= c;
            }
            s_prefix = pass == 0 ? ((unsigned)b << 8) : (prefix | (unsigned)b);
            s_remaining = remaining;
        }
        __syncthreads();
    }
    const unsigned T = s_prefix;
    const int need = s_remaining;
    if (tid == 0) s_base = 0;
    __syncthreads();
    // index-ordered pass: each thread owns 8 consecutive channels so that it can emit one mask byte
    for (int64_t kb = 0; kb < K; kb += (int64_t)kThreads * 8) {
        const int64_t k0 = kb + (int64_t)tid * 8;
        const bool active = k0 < K;
        uint32_t eqm = 0, gtm = 0;
        uint16_t v[8];
        if (active) {
            uint4 r = *reinterpret_cast<const uint4*>(&s_r[k0]);
            const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                v[i] = (uint16_t)(w[i >> 1] >> ((i & 1) * 16));
                unsigned key = v[i] & 0x7FFFu;
                eqm |= (key == T ? 1u : 0u) << i;
                gtm |= (key > T ? 1u : 0u) << i;
            }
        }
        int cnt = __popc(eqm);
        // exclusive prefix of cnt over the CTA (thread order = channel order)
        int incl = cnt;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
            if (lane >= o) incl += t;
        }
        if (lane == 31) s_warp_count[warp] = incl;
        __syncthreads();
        int before = s_base + incl - cnt;
        for (int j = 0; j < warp; ++j) before += s_warp_count[j];
        if (active) {
            uint32_t keep = gtm;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                if ((eqm >> i) & 1u) {
                    if (before < need) keep |= 1u << i;
                    ++before;
                }
            }
            if (a.mask_bits) a.mask_bits[m * (K / 8) + k0 / 8] = (uint8_t)keep;
            if (a.r_codes && a.mask_r_codes) {  // written earlier by this CTA (a barrier ago): zero the dropped codes
                uint32_t nib = 0;
#pragma unroll
                for (int i = 0; i < 8; ++i) nib |= ((keep >> i) & 1u) * (0xFu << (4 * i));
                uint32_t* c = reinterpret_cast<uint32_t*>(a.r_codes + m * (K / 2) + k0 / 2);
                *c = __ldcg(c) & nib;
            }
            if (a.r_bf16) {
                uint32_t w[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    uint32_t lo = (keep >> (2 * i)) & 1u ? (uint32_t)v[2 * i] : 0u;
                    uint32_t hi = (keep >> (2 * i + 1)) & 1u ? (uint32_t)v[2 * i + 1] : 0u;
                    w[i] = lo | (hi << 16);
                }
                *reinterpret_cast<uint4*>(a.r_bf16 + m * K + k0) = make_uint4(w[0], w[1], w[2], w[3]);
            }
        }
        __syncthreads();
        if (tid == 0) {
            int tot = 0;
            for (int j = 0; j < kWarpsPerCta; ++j) tot += s_warp_count[j];
            s_base += tot;
        }
        __syncthreads();
    }
}

// ------------------------------------------------------------------------------------------------
template <int FMT>
__global__ void __launch_bounds__(kThreads) dequant_kernel(const uint8_t* __restrict__ codes, const void* __restrict__ side,
                                                           int64_t rows, int64_t K, float* __restrict__ out) {
    int64_t idx = (int64_t)blockIdx.x * kThreads + threadIdx.x;  // one thread per 8 elements
    int64_t per_row = K / 8;
    if (idx >= rows * per_row) return;
    int64_t r = idx / per_row, k0 = (idx % per_row) * 8;
    uint32_t c = *reinterpret_cast<const uint32_t*>(codes + r * (K / 2) + k0 / 2);
    float v[8];
    if (FMT == kHiF4) {
        uint32_t meta = reinterpret_cast<const uint32_t*>(side)[r * (K / kHif4Block) + k0 / kHif4Block];
        hif4_decode_lane(c, meta, (int)((k0 / 8) & 7), v);
    } else {
        uint32_t sc = reinterpret_cast<const uint8_t*>(side)[r * (K / kMxBlock) + k0 / kMxBlock];
        mxfp4_decode_lane(c, sc, v);
    }
    float4* o = reinterpret_cast<float4*>(out + r * K + k0);
    o[0] = make_float4(v[0], v[1], v[2], v[3]);
    o[1] = make_float4(v[4], v[5], v[6], v[7]);
}

// debugging overrides (honoured only under RESQ_DEBUG, see common.cuh)
bool getenv_is_zero(const char* name) { return env_is_zero(name); }
// RESQ_ROW50_TEAM=0 sends long rows to the older CTA-per-row kernel
bool env_flag_row50_team() { return !env_is_zero("RESQ_ROW50_TEAM"); }

int pick_rows_per_cta(int64_t M, int64_t K, int pattern) {
    // enough CTAs to fill 148 SMs several times over, but long enough row loops to amortize set-up
    int64_t col_ctas = (K + (int64_t)kWarpsPerCta * kColsPerWarp - 1) / ((int64_t)kWarpsPerCta * kColsPerWarp);
    int64_t want_ctas = 148 * 8;
    int64_t rows = std::max<int64_t>(1, (M * col_ctas) / want_ctas);
    int r = 1;
    while (r * 2 <= rows && r < 32) r *= 2;
    (void)pattern;
    return r;  // a power of two <= 32, so a CTA never straddles a 32-row block boundary
}

}  // namespace

size_t quant_scratch_bytes(int64_t M, int64_t K, int pattern) {
    size_t n = 0;
    if (pattern == RESQ_S_CHAN50) n = (size_t)K;
    if (pattern == RESQ_S_BLOCK32x64_50) n = (size_t)(M / kBlkRows) * (size_t)(K / kBlkCols);
    if (n == 0) return 0;
    return align_up(n * sizeof(double), 256) + align_up(n, 256) + ((int64_t)n > kSelGridMin ? kSelGridScratch : 0);
}

// 8-bit activations of the "W4A8" ablation: MXFP8 with E4M3 elements (blocks of 32 along K, E8M0 scale
// 2^(floor(log2 amax) - 8), elements rounded to nearest even and saturated at 448).  Only the decoded image is
// needed (the GEMM takes a bf16 operand; an E4M3 value times a power of two is exact in bf16).  A lane owns 8
// values, an aligned quad of lanes a block.
__global__ void __launch_bounds__(kThreads) quant_mxfp8_image_kernel(const __nv_bfloat16* __restrict__ X, int64_t M, int64_t K,
                                                                     int64_t ldx, __nv_bfloat16* __restrict__ img,
                                                                     uint32_t* clear_words, int n_clear_words) {
    pdl_wait();
    pdl_trigger();
    if (clear_words && blockIdx.x == 0)
        for (int i = threadIdx.x; i < n_clear_words; i += blockDim.x) clear_words[i] = 0u;
    const int lane = threadIdx.x & 31;
    const int64_t chunks_per_row = K / 8;
    const int64_t total = M * chunks_per_row;  // K % 32 == 0: whole quads are in range or not
    for (int64_t c0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) - lane; c0 < total; c0 += (int64_t)gridDim.x * blockDim.x) {
        const int64_t c = c0 + lane;
        const bool active = c < total;
        const int64_t m = active ? c / chunks_per_row : 0, k0 = active ? (c % chunks_per_row) * 8 : 0;
        float x[8];
        uint4 raw = make_uint4(0, 0, 0, 0);
        if (active) raw = ld_nc_16(X + m * ldx + k0);
        unpack_bf16x8(raw, x);
        float m8 = 0.0f;
#pragma unroll
        for (int i = 0; i < 8; ++i) m8 = fmaxf(m8, fabsf(x[i]));
        const uint32_t ab = __reduce_max_sync(0xFu << (lane & 28), __float_as_uint(m8));
        const int e = ab == 0u ? -127 : max((int)(ab >> 23) - 127 - 8, -127);
        const float inv = __uint_as_float((uint32_t)(127 - e) << 23);                          // 2^-e, exact
        const float scale = __uint_as_float(e == -127 ? 0x00400000u : (uint32_t)(e + 127) << 23);  // 2^e
        uint32_t o[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            uint16_t pk;
            asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(pk) : "f"(__fmul_rn(x[2 * i + 1], inv)), "f"(__fmul_rn(x[2 * i], inv)));
            uint32_t h2;
            asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"(pk));
            const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&h2));
            const __nv_bfloat162 b = __floats2bfloat162_rn(__fmul_rn(f.x, scale), __fmul_rn(f.y, scale));
            o[i] = *reinterpret_cast<const uint32_t*>(&b);
        }
        if (active) *reinterpret_cast<uint4*>(img + m * K + k0) = make_uint4(o[0], o[1], o[2], o[3]);
    }
}

int launch_quantize_mxfp8_image(const __nv_bfloat16* X, int64_t M, int64_t K, int64_t ldx, __nv_bfloat16* img, uint32_t* clear_words,
                                int n_clear_words, cudaStream_t stream) {
    const int64_t threads = M * (K / 8);
    const unsigned ctas = (unsigned)std::min<int64_t>((threads + kThreads - 1) / kThreads, 148 * 16);
    LaunchScope scope(kKindQuant, stream);
    return cuda_fail(launch_kernel(quant_mxfp8_image_kernel, dim3(ctas), dim3(kThreads), 0, stream, X, M, K, ldx, img, clear_words,
                                   n_clear_words),
                     "quant_mxfp8_image_kernel launch");
}

// ------------------------------------------------------------------------------------------------
// The same exact selection for many scores (tens of thousands of blocks at prefill sizes), where one CTA re-reading
// all keys eight times is the bottleneck: four passes over 16-bit digits, each a grid-wide histogram kernel
// (global counters) and a one-CTA kernel that finds the bucket of the keep-th largest key and clears the counters
// for the next pass; then a grid-wide flag kernel.  Ties at the threshold are kept lowest index first: when not all
// of them are kept (rare) a one-CTA pass orders them.  State block after the histogram: [0..1] prefix (u64),
// [2] remaining, [3] entries equal to the threshold.
struct SelState {
    unsigned long long prefix;
    int remaining;
    int equal;
};

__global__ void __launch_bounds__(256) sel_grid_init_kernel(uint32_t* hist, SelState* st, int keep) {
    pdl_wait();
    pdl_trigger();
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < 65536; i += gridDim.x * blockDim.x) hist[i] = 0u;
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        st->prefix = 0ull;
        st->remaining = keep;
        st->equal = 0;
    }
}

__global__ void __launch_bounds__(256) sel_grid_hist_kernel(const double* __restrict__ score, int n, int shift, uint32_t* hist,
                                                            const SelState* st) {
    pdl_wait();
    pdl_trigger();
    const unsigned long long prefix = st->prefix;
    for (int i0 = blockIdx.x * blockDim.x; i0 < n; i0 += gridDim.x * blockDim.x) {
        const int i = i0 + threadIdx.x;
        const unsigned long long key = i < n ? (unsigned long long)__double_as_longlong(score[i]) : 0ull;
        const bool match = i < n && (shift == 48 ? true : ((key ^ prefix) >> (shift + 16)) == 0ull);
        const unsigned bucket = match ? (unsigned)(key >> shift) & 0xFFFFu : 0xFFFFFFFFu;
        const unsigned same = __match_any_sync(0xFFFFFFFFu, bucket);  // neighbouring scores often share the digit
        if (match && (unsigned)(__ffs((int)same) - 1) == (threadIdx.x & 31u)) atomicAdd(&hist[bucket], (unsigned)__popc(same));
    }
}

// One CTA of 1024 threads: thread t owns buckets 64 t .. 64 t + 63.
__global__ void __launch_bounds__(1024) sel_grid_scan_kernel(uint32_t* hist, SelState* st, int shift) {
    __shared__ int s_part[1024];
    pdl_wait();
    pdl_trigger();
    const int tid = threadIdx.x;
    uint32_t h[64];
    int mine = 0;
#pragma unroll
    for (int j = 0; j < 64; j += 4) {
        const uint4 v = *reinterpret_cast<const uint4*>(hist + 64 * tid + j);
        h[j] = v.x; h[j + 1] = v.y; h[j + 2] = v.z; h[j + 3] = v.w;
        mine += (int)(v.x + v.y + v.z + v.w);
    }
#pragma unroll
    for (int j = 0; j < 64; j += 4) *reinterpret_cast<uint4*>(hist + 64 * tid + j) = make_uint4(0, 0, 0, 0);  // for the next pass
    s_part[tid] = mine;
    __syncthreads();
    // inclusive suffix sums over threads (keys in higher buckets are larger)
    for (int o = 1; o < 1024; o <<= 1) {
        const int t = tid + o < 1024 ? s_part[tid + o] : 0;
        __syncthreads();
        s_part[tid] += t;
        __syncthreads();
    }
    const int remaining = st->remaining;
    const int incl = s_part[tid], above = incl - mine;
    __syncthreads();
    if (above < remaining && incl >= remaining) {  // exactly one thread
        int rem = remaining - above;
        int b = 63;
        for (; b > 0; --b) {
            const int c = (int)h[b];
            if (c >= rem) break;
            rem -= c;
        }
        st->prefix |= (unsigned long long)(64 * tid + b) << shift;
        st->remaining = rem;
        st->equal = (int)h[b];
    }
}

__global__ void __launch_bounds__(256) sel_grid_flag_kernel(const double* __restrict__ score, int n, const SelState* st,
                                                            uint8_t* __restrict__ flag) {
    pdl_wait();
    pdl_trigger();
    const unsigned long long T = st->prefix;
    const bool all_ties = st->remaining == st->equal;  // every entry equal to the threshold is kept
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) {
        const unsigned long long key = (unsigned long long)__double_as_longlong(score[i]);
        flag[i] = (key > T || (key == T && all_ties)) ? 1 : 0;
    }
}

// Only when some but not all ties are kept: one CTA walks the scores in index order and admits the first `remaining`.
__global__ void __launch_bounds__(kSelThreads) sel_grid_ties_kernel(const double* __restrict__ score, int n, const SelState* st,
                                                                    uint8_t* __restrict__ flag) {
    __shared__ int s_warp_count[kSelThreads / 32];
    __shared__ int s_base;
    pdl_wait();
    pdl_trigger();
    if (st->remaining == st->equal) return;
    const unsigned long long T = st->prefix;
    const int need = st->remaining;
    const int tid = threadIdx.x;
    if (tid == 0) s_base = 0;
    __syncthreads();
    for (int i0 = 0; i0 < n; i0 += kSelThreads) {
        const int i = i0 + tid;
        const bool eq = i < n && (unsigned long long)__double_as_longlong(score[i]) == T;
        const unsigned bal = __ballot_sync(0xFFFFFFFFu, eq);
        const int lane = tid & 31, w = tid >> 5;
        if (lane == 0) s_warp_count[w] = __popc(bal);
        __syncthreads();
        int before = s_base;
        for (int j = 0; j < w; ++j) before += s_warp_count[j];
        before += __popc(bal & ((1u << lane) - 1u));
        if (eq && before < need) flag[i] = 1;
        __syncthreads();
        if (tid == 0) {
            int tot = 0;
            for (int j = 0; j < kSelThreads / 32; ++j) tot += s_warp_count[j];
            s_base += tot;
        }
        __syncthreads();
    }
}

// The same exact selection for at most 1024 scores (block scores of decode-sized calls, the blocks of one strip):
// one key per thread, a bitonic sort of (score, index) in descending score / ascending index order -- strides below
// 32 by shuffles, the others through shared memory -- after which the thread at position p holds the p-th entry of
// the ranking.  The CTA has as many threads as the sort network has inputs (the power of two at or above n).
__global__ void __launch_bounds__(1024) topk_sort1024_kernel(const double* __restrict__ score, int n, int keep,
                                                             uint8_t* __restrict__ flag) {
    __shared__ unsigned long long s_key[1024];
    __shared__ int s_idx[1024];
    pdl_wait();
    pdl_trigger();
    const int tid = threadIdx.x;
    score += (int64_t)blockIdx.x * n;  // one independent selection of n scores per CTA
    flag += (int64_t)blockIdx.x * n;
    unsigned long long key = tid < n ? (unsigned long long)__double_as_longlong(score[tid]) : 0ull;  // scores are >= 0
    int idx = tid;  // padding entries: key 0 and the highest indices, so they rank last
    const int np2 = blockDim.x;  // a power of two >= n (at least a warp): the sort network's size
    for (int k = 2; k <= np2; k <<= 1) {
        for (int j = k >> 1; j > 0; j >>= 1) {
            unsigned long long pk;
            int pi;
            if (j < 32) {
                pk = __shfl_xor_sync(0xFFFFFFFFu, key, j);
                pi = __shfl_xor_sync(0xFFFFFFFFu, idx, j);
            } else {
                s_key[tid] = key;
                s_idx[tid] = idx;
                __syncthreads();
                pk = s_key[tid ^ j];
                pi = s_idx[tid ^ j];
                __syncthreads();
            }
            // "mine ranks before the partner's": larger score, or equal score and lower index
            const bool mine_first = key > pk || (key == pk && idx < pi);
            const bool lower = (tid & j) == 0;          // this thread is the lower position of the pair
            const bool ranked_order = (tid & k) == 0;   // this sub-sequence is being put in ranking order
            const bool keep_mine = (lower == ranked_order) ? mine_first : !mine_first;
            if (!keep_mine) {
                key = pk;
                idx = pi;
            }
        }
    }
    if (idx < n) flag[idx] = tid < keep ? 1 : 0;
}

// Channel scores of CHAN50 from the (unmasked) bf16 residual image the block-per-lane quantizer has just written
// (still in L2 for all but the largest inputs): a thread owns 8 channels and a strip of rows; the squares of the
// decoded values are exact, the strip sums run in fp64, one atomic per channel and strip.
__global__ void __launch_bounds__(256) chan_score_kernel(const __nv_bfloat16* __restrict__ img, int64_t M, int64_t K,
                                                         double* __restrict__ scores, int strip_rows) {
    pdl_wait();
    pdl_trigger();
    const int64_t per_row = K / 8;
    const int64_t strips = (M + strip_rows - 1) / strip_rows;
    const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= per_row * strips) return;
    const int64_t k0 = (idx % per_row) * 8, m0 = (idx / per_row) * strip_rows;
    const int64_t m1 = min(M, m0 + strip_rows);
    double acc[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] = 0.0;
    for (int64_t m = m0; m < m1; ++m) {
        float v[8];
        unpack_bf16x8(__ldcg(reinterpret_cast<const uint4*>(img + m * K + k0)), v);
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[i] += (double)v[i] * (double)v[i];
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) atomicAdd(&scores[k0 + i], acc[i]);
}

// Second and third kernel of the patterns with a tensor-wide selection (CHAN50, BLOCK): top half of the scores,
// then the mask pass over the residual outputs.
static int launch_global_select(const QuantArgs& a, int64_t nscore, cudaStream_t stream) {
    int rc = RESQ_OK;
    // per-strip block rule: one selection of K/64 scores per strip of 32 rows (the scores of a strip are contiguous)
    const bool strips = a.per_strip && a.pattern == RESQ_S_BLOCK32x64_50;
    const unsigned nsel = strips ? (unsigned)(a.M / kBlkRows) : 1u;
    if (strips) nscore = a.K / kBlkCols;
    const int keep = (int)(nscore * a.keep_quarters / 4);
    // (debugging override RESQ_SEL_GRID=0 keeps the one-CTA selection)
    if (!strips && a.sel_hist && nscore > kSelGridMin && keep > 0 && keep < nscore && !env_is_zero("RESQ_SEL_GRID")) {
        SelState* st = reinterpret_cast<SelState*>(a.sel_hist + 65536);
        const unsigned grid = (unsigned)std::min<int64_t>((nscore + 255) / 256, 148 * 4);
        {
            LaunchScope scope(kKindSelect, stream);
            rc = cuda_fail(launch_kernel(sel_grid_init_kernel, dim3(64), dim3(256), 0, stream, a.sel_hist, st, keep),
                           "sel_grid_init_kernel launch");
        }
        for (int shift = 48; shift >= 0 && !rc; shift -= 16) {
            {
                LaunchScope scope(kKindSelect, stream);
                rc = cuda_fail(launch_kernel(sel_grid_hist_kernel, dim3(grid), dim3(256), 0, stream, (const double*)a.scores, (int)nscore,
                                             shift, a.sel_hist, (const SelState*)st),
                               "sel_grid_hist_kernel launch");
            }
            if (!rc) {
                LaunchScope scope(kKindSelect, stream);
                rc = cuda_fail(launch_kernel(sel_grid_scan_kernel, dim3(1), dim3(1024), 0, stream, a.sel_hist, st, shift),
                               "sel_grid_scan_kernel launch");
            }
        }
        if (!rc) {
            LaunchScope scope(kKindSelect, stream);
            rc = cuda_fail(launch_kernel(sel_grid_flag_kernel, dim3(grid), dim3(256), 0, stream, (const double*)a.scores, (int)nscore,
                                         (const SelState*)st, a.keep_flags),
                           "sel_grid_flag_kernel launch");
        }
        if (!rc) {
            LaunchScope scope(kKindSelect, stream);
            rc = cuda_fail(launch_kernel(sel_grid_ties_kernel, dim3(1), dim3(kSelThreads), 0, stream, (const double*)a.scores, (int)nscore,
                                         (const SelState*)st, a.keep_flags),
                           "sel_grid_ties_kernel launch");
        }
    } else if (nscore <= 1024 && !getenv_is_zero("RESQ_SEL_SORT")) {
        LaunchScope scope(kKindSelect, stream);
        unsigned np2 = 32;
        while ((int64_t)np2 < nscore) np2 <<= 1;
        rc = cuda_fail(launch_kernel(topk_sort1024_kernel, dim3(nsel), dim3(np2), 0, stream, (const double*)a.scores, (int)nscore, keep,
                                     a.keep_flags),
                       "topk_sort1024_kernel launch");
    } else {
        LaunchScope scope(kKindSelect, stream);
        rc = cuda_fail(launch_kernel(topk_select_kernel, dim3(nsel), dim3(kSelThreads), 0, stream, (const double*)a.scores, (int)nscore,
                                     keep, a.keep_flags),
                       "topk_select_kernel launch");
    }
    if (rc) return rc;
    // (block-wise selection feeding the CTA-pair GEMM: the image stays unmasked, the GEMM reads the keep flags)
    __nv_bfloat16* mask_img = (a.skip_image_mask && a.pattern == RESQ_S_BLOCK32x64_50) ? nullptr : a.r_bf16;
    if (a.mask_bits || mask_img || (a.r_codes && a.mask_r_codes)) {
        const int64_t n = a.M * (a.K / 8);
        LaunchScope scope(kKindSelect, stream);
        rc = cuda_fail(launch_kernel(apply_global_mask_kernel, dim3((unsigned)((n + 255) / 256)), dim3(256), 0, stream, a.pattern, a.M,
                                     a.K, (const uint8_t*)a.keep_flags, a.mask_bits, mask_img, a.mask_r_codes ? a.r_codes : (uint8_t*)nullptr),
                       "apply_global_mask_kernel launch");
    }
    return rc;
}

int launch_quantize(int fmt, const QuantArgs& a_in, cudaStream_t stream) {
    QuantArgs a = a_in;
    if (a.keep_quarters < 1 || a.keep_quarters > 3) a.keep_quarters = 2;  // the paper's 50 %
    if (a.r_comp && a.keep_quarters != 2) {
        set_last_error("internal: the compressed residual operand exists for 2:4 only");
        return RESQ_ERR_CUDA;
    }
    const int pattern = a.pattern;
    const bool residual = pattern != RESQ_S_NONE;
    if (pattern == RESQ_S_ROW50 && (a.X_up || a.gamma || a.rht)) {
        set_last_error("the fused producers do not support the row-wise selection");
        return RESQ_ERR_PATTERN;
    }
    if (a.gamma) {  // row scales first (the quantizer kernel waits for them through the programmatic dependency)
        LaunchScope scope(kKindQuant, stream);
        int rc0 = cuda_fail(launch_kernel(rmsnorm_row_scale_kernel, dim3((unsigned)((a.M + 7) / 8)), dim3(256), 0, stream, a.X, a.M, a.K,
                                          a.ldx, a.eps, a.row_scale),
                            "rmsnorm_row_scale_kernel launch");
        if (rc0) return rc0;
    }
    if (pattern == RESQ_S_ROW50) {
        // a warp per row with the block-per-lane encoders, if the row's image fits next to the staging tiles
        auto al16r = [](const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; };
        const int nseg = (int)((a.K / kHif4Block + 31) / 32);
        const int per_warp = (3 + nseg) * kStageBytes;
        const int wpc = std::min(kWarpsPerCta, (220 * 1024) / per_warp);
        const bool aligned = al16r(a.x_codes) && al16r(a.r_codes) && al16r(a.mask_bits) && al16r(a.x_side) && al16r(a.r_side) &&
                             al16r(a.a_bf16) && al16r(a.r_bf16);
        const bool img = a.a_bf16 != nullptr;
        if (a.K % kHif4Block == 0 && nseg <= 2 && wpc >= 1 && a.M >= 148 && aligned) {
            void (*kern)(QuantArgs, int);
            if (nseg == 1)  // one segment: the lean variant (128 registers, two tiles per warp: two CTAs per SM)
                kern = fmt == kHiF4 ? (img ? quant_row50_warp_kernel<kHiF4, true, 1, 1> : quant_row50_warp_kernel<kHiF4, false, 1, 1>)
                                    : (img ? quant_row50_warp_kernel<kMXFP4, true, 1, 1> : quant_row50_warp_kernel<kMXFP4, false, 1, 1>);
            else
                kern = fmt == kHiF4 ? (img ? quant_row50_warp_kernel<kHiF4, true, 1, 2> : quant_row50_warp_kernel<kHiF4, false, 1, 2>)
                                    : (img ? quant_row50_warp_kernel<kMXFP4, true, 1, 2> : quant_row50_warp_kernel<kMXFP4, false, 1, 2>);
            const int smem_w = nseg == 1 ? wpc * 2 * kStageBytes : wpc * per_warp;
            cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_w);
            if (e != cudaSuccess) return cuda_fail(e, "cudaFuncSetAttribute(row50 warp)");
            LaunchScope scope(kKindQuant, stream);
            return cuda_fail(launch_kernel(kern, dim3((unsigned)((a.M + wpc - 1) / wpc)), dim3(kThreads), (size_t)smem_w, stream, a, wpc),
                             "quant_row50_warp_kernel launch");
        }
        // longer rows (up to 16 segments): the warps of a persistent CTA share a row, one segment each
        if (a.K % kHif4Block == 0 && nseg <= 16 && aligned && env_flag_row50_team()) {
            const bool wide = nseg > kWarpsPerCta;  // 16 warps per CTA instead of 8
            void (*kern)(QuantArgs, int);
            if (wide)
                kern = fmt == kHiF4 ? (img ? quant_row50_warp_kernel<kHiF4, true, 16, 1> : quant_row50_warp_kernel<kHiF4, false, 16, 1>)
                                    : (img ? quant_row50_warp_kernel<kMXFP4, true, 16, 1> : quant_row50_warp_kernel<kMXFP4, false, 16, 1>);
            else
                kern = fmt == kHiF4 ? (img ? quant_row50_warp_kernel<kHiF4, true, 8, 1> : quant_row50_warp_kernel<kHiF4, false, 8, 1>)
                                    : (img ? quant_row50_warp_kernel<kMXFP4, true, 8, 1> : quant_row50_warp_kernel<kMXFP4, false, 8, 1>);
            const int warps = wide ? 16 : 8;
            const int smem_t = warps * 2 * kStageBytes;
            cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_t);
            if (e != cudaSuccess) return cuda_fail(e, "cudaFuncSetAttribute(row50 team)");
            LaunchScope scope(kKindQuant, stream);
            const unsigned ctas = (unsigned)std::min<int64_t>(a.M, wide ? 148 : 296);  // resident CTAs, rows strided
            return cuda_fail(launch_kernel(kern, dim3(ctas), dim3(32 * warps), (size_t)smem_t, stream, a, warps),
                             "quant_row50_warp_kernel (team) launch");
        }
        size_t smem = (size_t)a.K * sizeof(uint16_t);
        if (smem > 200 * 1024) {
            set_last_error("ROW50 supports K <= %d", 200 * 1024 / 2);
            return RESQ_ERR_SHAPE;
        }
        auto kern = fmt == kHiF4 ? quant_row50_kernel<kHiF4> : quant_row50_kernel<kMXFP4>;
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return cuda_fail(e, "cudaFuncSetAttribute(row50)");
        LaunchScope scope(kKindQuant, stream);
        return cuda_fail(launch_kernel(kern, dim3((unsigned)a.M), dim3(kThreads), smem, stream, a), "quant_row50_kernel launch");
    }
    const bool global_sel = pattern == RESQ_S_CHAN50 || pattern == RESQ_S_BLOCK32x64_50;
    int64_t nscore = 0;
    if (global_sel) {
        nscore = pattern == RESQ_S_CHAN50 ? a.K : (a.M / kBlkRows) * (a.K / kBlkCols);
        cudaError_t e = cudaMemsetAsync(a.scores, 0, (size_t)nscore * sizeof(double), stream);
        if (e != cudaSuccess) return cuda_fail(e, "cudaMemsetAsync(scores)");
    }
    // row-local or block-wise selection on a large enough input: block-per-lane kernel (needs 16-byte aligned
    // outputs and, for MXFP4, whole pairs of 32-value blocks)
    auto al16 = [](const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; };
    // Worth it once there is a warp task (32 blocks of one row) for every warp slot of the machine; below
    // that the finer-grained kernel (a lane per 8 values) finishes sooner.
    const int64_t block_tasks = a.M * ((a.K / kHif4Block + 31) / 32);
    // (CHAN50 only when the residual image is written: its channel scores are then summed from the image)
    const bool chan_from_image = pattern == RESQ_S_CHAN50 && a.r_bf16 != nullptr && !getenv_is_zero("RESQ_CHAN_FROM_IMAGE");
    // (the chunk-per-lane kernel pays for CHAN50 with fp64 atomics per row and channel: the block kernel takes over earlier)
    const int64_t min_block_tasks = chan_from_image ? 148 : 148 * 16;
    if (!a.X_up && !a.gamma && !a.rht && (pattern != RESQ_S_CHAN50 || chan_from_image) && a.K % kHif4Block == 0 && block_tasks >= min_block_tasks && al16(a.x_codes) && al16(a.r_codes) && al16(a.mask_bits) &&
        al16(a.x_side) && al16(a.r_side) && al16(a.a_bf16) && al16(a.r_bf16) && al16(a.r_comp)) {
        const bool img = a.a_bf16 != nullptr;
        const int64_t ncg = (a.K / kHif4Block + 31) / 32;
        int rows_per_warp = 1;
        while (rows_per_warp < 32 && (a.M / (rows_per_warp * 2)) * ncg >= 148 * 16 * 4) rows_per_warp *= 2;
        const int64_t tasks = ((a.M + rows_per_warp - 1) / rows_per_warp) * ncg;
        const unsigned ctas = (unsigned)((tasks + kWarpsPerCta - 1) / kWarpsPerCta);
        const int smem = kWarpsPerCta * (img ? 3 : 2) * kStageBytes;
        auto launch = [&](void (*kern)(QuantArgs, int)) -> int {
            cudaError_t attr_err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
            if (attr_err != cudaSuccess) return cuda_fail(attr_err, "cudaFuncSetAttribute(quant_block_kernel)");
            LaunchScope scope(kKindQuant, stream);
            return cuda_fail(launch_kernel(kern, dim3(ctas), dim3(kThreads), (size_t)smem, stream, a, rows_per_warp),
                             "quant_block_kernel launch");
        };
        int rc;
        if (fmt == kHiF4)
            rc = residual ? (a.r_comp ? launch(quant_block_kernel<kHiF4, true, true, true>)
                                      : img ? launch(quant_block_kernel<kHiF4, true, true>) : launch(quant_block_kernel<kHiF4, true, false>))
                          : (img ? launch(quant_block_kernel<kHiF4, false, true>) : launch(quant_block_kernel<kHiF4, false, false>));
        else
            rc = residual ? (a.r_comp ? launch(quant_block_kernel<kMXFP4, true, true, true>)
                                      : img ? launch(quant_block_kernel<kMXFP4, true, true>) : launch(quant_block_kernel<kMXFP4, true, false>))
                          : (img ? launch(quant_block_kernel<kMXFP4, false, true>) : launch(quant_block_kernel<kMXFP4, false, false>));
        if (rc) return rc;
        if (chan_from_image) {
            // strips of rows per thread: long enough to amortise the atomics, short enough for a few threads per lane slot
            int strip = 64;
            while (strip > 4 && (a.K / 8) * ((a.M + strip - 1) / strip) < 148 * 512) strip /= 2;
            const int64_t nthreads = (a.K / 8) * ((a.M + strip - 1) / strip);
            LaunchScope scope(kKindSelect, stream);
            rc = cuda_fail(launch_kernel(chan_score_kernel, dim3((unsigned)((nthreads + 255) / 256)), dim3(256), 0, stream,
                                         (const __nv_bfloat16*)a.r_bf16, a.M, a.K, a.scores, strip),
                           "chan_score_kernel launch");
            if (rc) return rc;
        }
        if (global_sel) rc = launch_global_select(a, nscore, stream);
        return rc;
    }
    const int rows_per_cta = pick_rows_per_cta(a.M, a.K, pattern);
    dim3 grid((unsigned)((a.M + rows_per_cta - 1) / rows_per_cta),
              (unsigned)((a.K + (int64_t)kWarpsPerCta * kColsPerWarp - 1) / ((int64_t)kWarpsPerCta * kColsPerWarp)));
    cudaError_t launch_err = cudaSuccess;
    {
    LaunchScope scope(kKindQuant, stream);
    const bool img = a.a_bf16 != nullptr;  // the GEMM path asks for both images (r_bf16 whenever there is a residual)
    auto launch = [&](void (*kern)(QuantArgs, int)) { launch_err = launch_kernel(kern, grid, dim3(kThreads), 0, stream, a, rows_per_cta); };
    if (a.rht) {  // rotation baseline: weight packing (plain outputs) or the GEMM-feeding variants
        if (a.r_comp || (!img && residual)) {
            set_last_error("internal: the Hadamard pre-transform feeds weight packing or the dense GEMM operand images");
            return RESQ_ERR_CUDA;
        }
        if (fmt == kHiF4) {
            if (!img) launch(quant_stream_kernel<kHiF4, false, false, false, 3>);
            else residual ? launch(quant_stream_kernel<kHiF4, true, true, false, 3>) : launch(quant_stream_kernel<kHiF4, false, true, false, 3>);
        } else {
            if (!img) launch(quant_stream_kernel<kMXFP4, false, false, false, 3>);
            else residual ? launch(quant_stream_kernel<kMXFP4, true, true, false, 3>) : launch(quant_stream_kernel<kMXFP4, false, true, false, 3>);
        }
    } else if (a.X_up || a.gamma) {  // fused producer: GEMM-feeding variants only
        if (!img || a.r_comp) {
            set_last_error("internal: the fused producer feeds the dense GEMM operand images only");
            return RESQ_ERR_CUDA;
        }
        if (a.X_up) {
            if (fmt == kHiF4) residual ? launch(quant_stream_kernel<kHiF4, true, true, false, 1>) : launch(quant_stream_kernel<kHiF4, false, true, false, 1>);
            else residual ? launch(quant_stream_kernel<kMXFP4, true, true, false, 1>) : launch(quant_stream_kernel<kMXFP4, false, true, false, 1>);
        } else {
            if (fmt == kHiF4) residual ? launch(quant_stream_kernel<kHiF4, true, true, false, 2>) : launch(quant_stream_kernel<kHiF4, false, true, false, 2>);
            else residual ? launch(quant_stream_kernel<kMXFP4, true, true, false, 2>) : launch(quant_stream_kernel<kMXFP4, false, true, false, 2>);
        }
    } else if (fmt == kHiF4) {
        if (residual && a.r_comp) launch(quant_stream_kernel<kHiF4, true, true, true>);
        else if (residual) img ? launch(quant_stream_kernel<kHiF4, true, true>) : launch(quant_stream_kernel<kHiF4, true, false>);
        else img ? launch(quant_stream_kernel<kHiF4, false, true>) : launch(quant_stream_kernel<kHiF4, false, false>);
    } else {
        if (residual && a.r_comp) launch(quant_stream_kernel<kMXFP4, true, true, true>);
        else if (residual) img ? launch(quant_stream_kernel<kMXFP4, true, true>) : launch(quant_stream_kernel<kMXFP4, true, false>);
        else img ? launch(quant_stream_kernel<kMXFP4, false, true>) : launch(quant_stream_kernel<kMXFP4, false, false>);
    }
    }
    int rc = cuda_fail(launch_err, "quant_stream_kernel launch");
    if (rc) return rc;
    if (global_sel) rc = launch_global_select(a, nscore, stream);
    return rc;
}

// bf16 matrix transpose (the backward products quantize along their own contraction axes): 64 x 64 tiles through
// shared memory, coalesced on both sides.
__global__ void __launch_bounds__(256) transpose_bf16_kernel(const uint16_t* __restrict__ src, int64_t rows, int64_t cols, int64_t ld_src,
                                                             uint16_t* __restrict__ dst, int64_t ld_dst) {
    pdl_wait();
    pdl_trigger();
    __shared__ uint16_t tile[64][66];
    const int64_t r0 = (int64_t)blockIdx.y * 64, c0 = (int64_t)blockIdx.x * 64;
    const int tx = threadIdx.x & 63, ty = threadIdx.x >> 6;  // 64 x 4
    for (int i = ty; i < 64; i += 4) {
        const int64_t r = r0 + i, c = c0 + tx;
        tile[i][tx] = (r < rows && c < cols) ? src[r * ld_src + c] : (uint16_t)0;
    }
    __syncthreads();
    for (int i = ty; i < 64; i += 4) {
        const int64_t c = c0 + i, r = r0 + tx;  // dst row = source column
        if (c < cols && r < rows) dst[c * ld_dst + r] = tile[tx][i];
    }
}

int launch_transpose_bf16(const __nv_bfloat16* src, int64_t rows, int64_t cols, int64_t ld_src, __nv_bfloat16* dst, int64_t ld_dst,
                          cudaStream_t stream) {
    LaunchScope scope(kKindQuant, stream);
    dim3 grid((unsigned)((cols + 63) / 64), (unsigned)((rows + 63) / 64));
    return cuda_fail(launch_kernel(transpose_bf16_kernel, grid, dim3(256), 0, stream, reinterpret_cast<const uint16_t*>(src), rows, cols,
                                   ld_src, reinterpret_cast<uint16_t*>(dst), ld_dst),
                     "transpose_bf16_kernel launch");
}

// One launch for a group of activations with a row-local selection (NONE, DENSE, n:4) that feed the GEMM (images).
int launch_quantize_group(int fmt, const QuantArgs* a_in, int count, cudaStream_t stream) {
    if (count < 1 || count > kMaxQuantGroup) {
        set_last_error("a group holds 1 to %d problems (got %d)", kMaxQuantGroup, count);
        return RESQ_ERR_SHAPE;
    }
    QuantGroup g;
    memset(&g, 0, sizeof(g));
    g.count = count;
    const int pattern = a_in[0].pattern;
    const bool residual = pattern != RESQ_S_NONE;
    int blocks = 0;
    for (int i = 0; i < count; ++i) {
        QuantArgs a = a_in[i];
        if (a.keep_quarters < 1 || a.keep_quarters > 3) a.keep_quarters = 2;
        if (a.pattern != pattern || (pattern != RESQ_S_NONE && pattern != RESQ_S_DENSE && pattern != RESQ_S_2_4) || !a.a_bf16 ||
            a.r_comp || a.X_up || a.gamma || a.rht) {
            set_last_error("internal: a quantizer group takes one row-local pattern and the GEMM operand images");
            return RESQ_ERR_CUDA;
        }
        g.a[i] = a;
        g.rows_per_cta[i] = pick_rows_per_cta(a.M, a.K, pattern);
        g.gx[i] = (int)((a.M + g.rows_per_cta[i] - 1) / g.rows_per_cta[i]);
        g.gy[i] = (int)((a.K + (int64_t)kWarpsPerCta * kColsPerWarp - 1) / ((int64_t)kWarpsPerCta * kColsPerWarp));
        g.block_base[i] = blocks;
        blocks += g.gx[i] * g.gy[i];
    }
    for (int i = count; i <= kMaxQuantGroup; ++i) g.block_base[i] = blocks;
    void (*kern)(QuantGroup);
    if (fmt == kHiF4) kern = residual ? quant_stream_group_kernel<kHiF4, true, true, false> : quant_stream_group_kernel<kHiF4, false, true, false>;
    else kern = residual ? quant_stream_group_kernel<kMXFP4, true, true, false> : quant_stream_group_kernel<kMXFP4, false, true, false>;
    LaunchScope scope(kKindQuant, stream);
    return cuda_fail(launch_kernel(kern, dim3((unsigned)blocks), dim3(kThreads), 0, stream, g), "quant_stream_group_kernel launch");
}

int launch_dequantize(int fmt, const uint8_t* codes, const void* side, int64_t rows, int64_t K, float* out,
                      cudaStream_t stream) {
    int64_t n = rows * (K / 8);
    unsigned grid = (unsigned)((n + kThreads - 1) / kThreads);
    LaunchScope scope(kKindQuant, stream);
    if (fmt == kHiF4) dequant_kernel<kHiF4><<<grid, kThreads, 0, stream>>>(codes, side, rows, K, out);
    else dequant_kernel<kMXFP4><<<grid, kThreads, 0, stream>>>(codes, side, rows, K, out);
    return cuda_fail(cudaGetLastError(), "dequant_kernel launch");
}

}  // namespace resq
