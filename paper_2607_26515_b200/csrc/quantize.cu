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

__device__ __forceinline__ uint32_t top2_mask8(uint32_t oct) {
    return (uint32_t)kTop2Table.v[oct & 0xFFFu] | ((uint32_t)kTop2Table.v[(oct >> 16) & 0xFFFu] << 4);
}

template <int FMT>
__device__ __forceinline__ void store_side(void* side_ptr, int64_t row, int64_t K, int64_t k0, int lane, uint32_t side) {
    if (FMT == kHiF4) {
        if ((lane & 7) == 0) reinterpret_cast<uint32_t*>(side_ptr)[row * (K / kHif4Block) + k0 / kHif4Block] = side;
    } else {
        if ((lane & 3) == 0) reinterpret_cast<uint8_t*>(side_ptr)[row * (K / kMxBlock) + k0 / kMxBlock] = (uint8_t)side;
    }
}

// ------------------------------------------------------------------------------------------------
// Streaming kernel for the patterns whose selection is local to a row segment (NONE, DENSE, 2:4) and
// first pass of the global ones (CHAN50, BLOCK: writes the unmasked residual and accumulates scores).
// grid.y: groups of 8 warps, each warp owning 256 channels; grid.x: row chunks of `rows_per_cta`.
template <int FMT, bool RESIDUAL>
__global__ void __launch_bounds__(kThreads) quant_stream_kernel(QuantArgs a, int rows_per_cta) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t k0 = ((int64_t)blockIdx.y * kWarpsPerCta + warp) * kColsPerWarp + lane * 8;
    const bool active = k0 < a.K;  // whole blocks are active or not (K is a multiple of the block size)
    const int64_t m_begin = (int64_t)blockIdx.x * rows_per_cta;
    const int64_t m_end = min(a.M, m_begin + rows_per_cta);
    const int pattern = a.pattern;

    double chan_acc[8];
    double blk_acc = 0.0;
#pragma unroll
    for (int i = 0; i < 8; ++i) chan_acc[i] = 0.0;

    uint4 raw = make_uint4(0, 0, 0, 0);
    if (active && m_begin < m_end) raw = ld_nc_16(a.X + m_begin * a.ldx + k0);
    for (int64_t m = m_begin; m < m_end; ++m) {
        uint4 cur = raw;
        if (active && m + 1 < m_end) raw = ld_nc_16(a.X + (m + 1) * a.ldx + k0);  // prefetch the next row
        float x[8], deq[8];
        unpack_bf16x8(cur, x);
        uint32_t codes, side, oct;
        encode_lane<FMT>(x, lane, codes, side, deq, oct);
        if (active) {
            if (a.x_codes) *reinterpret_cast<uint32_t*>(a.x_codes + m * (a.K / 2) + k0 / 2) = codes;
            if (a.x_side) store_side<FMT>(a.x_side, m, a.K, k0, lane, side);
            if (a.a_bf16) {
                uint4 o;
                o.x = pack_bf16x2_exact(deq[0], deq[1]);
                o.y = pack_bf16x2_exact(deq[2], deq[3]);
                o.z = pack_bf16x2_exact(deq[4], deq[5]);
                o.w = pack_bf16x2_exact(deq[6], deq[7]);
                *reinterpret_cast<uint4*>(a.a_bf16 + m * a.K + k0) = o;
            }
        }
        if constexpr (RESIDUAL) {
        // Eq. (3): the difference of a bf16 value and its decoded code is exact in fp32
        float dx[8], rdeq[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) dx[i] = __fsub_rn(x[i], deq[i]);
        uint32_t rcodes, rside, roct;
        encode_lane<FMT>(dx, lane, rcodes, rside, rdeq, roct);
        uint32_t keep = 0xFFu;
        if (pattern == RESQ_S_2_4) keep = top2_mask8(roct);
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
            if (a.r_codes) *reinterpret_cast<uint32_t*>(a.r_codes + m * (a.K / 2) + k0 / 2) = rcodes;
            if (a.r_side) store_side<FMT>(a.r_side, m, a.K, k0, lane, rside);
            const bool local = pattern == RESQ_S_DENSE || pattern == RESQ_S_2_4;
            if (a.mask_bits && local) a.mask_bits[m * (a.K / 8) + k0 / 8] = (uint8_t)keep;
            if (a.r_bf16) {
                // for the global patterns this is the unmasked image; the apply kernel zeroes dropped entries
                float r[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) r[i] = ((keep >> i) & 1u) ? rdeq[i] : 0.0f;
                uint4 o;
                o.x = pack_bf16x2_exact(r[0], r[1]);
                o.y = pack_bf16x2_exact(r[2], r[3]);
                o.z = pack_bf16x2_exact(r[4], r[5]);
                o.w = pack_bf16x2_exact(r[6], r[7]);
                *reinterpret_cast<uint4*>(a.r_bf16 + m * a.K + k0) = o;
            }
        }
        }  // RESIDUAL
    }
    if (RESIDUAL && pattern == RESQ_S_CHAN50 && active) {
#pragma unroll
        for (int i = 0; i < 8; ++i) atomicAdd(&a.scores[k0 + i], chan_acc[i]);
    }
}

// ------------------------------------------------------------------------------------------------
// Exact top-`keep` of n non-negative fp64 scores, ties to the lower index.  One CTA: MSB-first radix
// select over the 64-bit patterns (8 passes of 8 bits), then an index-ordered pass that admits the
// first `need` entries equal to the threshold.
constexpr int kSelThreads = 1024;

__global__ void __launch_bounds__(kSelThreads) topk_select_kernel(const double* __restrict__ score, int n, int keep,
                                                                 uint8_t* __restrict__ flag) {
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
        for (int i = tid; i < n; i += kSelThreads) {
            unsigned long long key = (unsigned long long)__double_as_longlong(score[i]);
            bool match = shift == 56 ? true : ((key ^ prefix) >> (shift + 8)) == 0ull;
            if (match) atomicAdd(&hist[(unsigned)(key >> shift) & 255u], 1u);
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

// Turn the kept-channel / kept-block flags into mask bits and zero the dropped entries of the GEMM's
// residual operand.  One thread per 8 channels of one row.
__global__ void apply_global_mask_kernel(int pattern, int64_t M, int64_t K, const uint8_t* __restrict__ flag,
                                         uint8_t* __restrict__ mask_bits, __nv_bfloat16* __restrict__ r_bf16) {
    int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
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

// ------------------------------------------------------------------------------------------------
// ROW50: per row, keep the K/2 largest decoded magnitudes (ties: lower index).  One CTA per row: the
// row's decoded residual (bf16-exact, so its 15 magnitude bits order like the values) is staged in
// shared memory, a 2-pass radix select finds the threshold, an index-ordered pass resolves ties.
template <int FMT>
__global__ void __launch_bounds__(kThreads) quant_row50_kernel(QuantArgs a) {
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
        s_remaining = (int)(K / 2);
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
    return align_up(n * sizeof(double), 256) + align_up(n, 256);
}

int launch_quantize(int fmt, const QuantArgs& a, cudaStream_t stream) {
    const int pattern = a.pattern;
    const bool residual = pattern != RESQ_S_NONE;
    if (pattern == RESQ_S_ROW50) {
        size_t smem = (size_t)a.K * sizeof(uint16_t);
        if (smem > 200 * 1024) {
            set_last_error("ROW50 supports K <= %d", 200 * 1024 / 2);
            return RESQ_ERR_SHAPE;
        }
        auto kern = fmt == kHiF4 ? quant_row50_kernel<kHiF4> : quant_row50_kernel<kMXFP4>;
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return cuda_fail(e, "cudaFuncSetAttribute(row50)");
        LaunchScope scope(kKindQuant, stream);
        kern<<<(unsigned)a.M, kThreads, smem, stream>>>(a);
        return cuda_fail(cudaGetLastError(), "quant_row50_kernel launch");
    }
    const bool global_sel = pattern == RESQ_S_CHAN50 || pattern == RESQ_S_BLOCK32x64_50;
    int64_t nscore = 0;
    if (global_sel) {
        nscore = pattern == RESQ_S_CHAN50 ? a.K : (a.M / kBlkRows) * (a.K / kBlkCols);
        cudaError_t e = cudaMemsetAsync(a.scores, 0, (size_t)nscore * sizeof(double), stream);
        if (e != cudaSuccess) return cuda_fail(e, "cudaMemsetAsync(scores)");
    }
    const int rows_per_cta = pick_rows_per_cta(a.M, a.K, pattern);
    dim3 grid((unsigned)((a.M + rows_per_cta - 1) / rows_per_cta),
              (unsigned)((a.K + (int64_t)kWarpsPerCta * kColsPerWarp - 1) / ((int64_t)kWarpsPerCta * kColsPerWarp)));
    {
    LaunchScope scope(kKindQuant, stream);
    if (fmt == kHiF4) {
        if (residual) quant_stream_kernel<kHiF4, true><<<grid, kThreads, 0, stream>>>(a, rows_per_cta);
        else quant_stream_kernel<kHiF4, false><<<grid, kThreads, 0, stream>>>(a, rows_per_cta);
    } else {
        if (residual) quant_stream_kernel<kMXFP4, true><<<grid, kThreads, 0, stream>>>(a, rows_per_cta);
        else quant_stream_kernel<kMXFP4, false><<<grid, kThreads, 0, stream>>>(a, rows_per_cta);
    }
    }
    int rc = cuda_fail(cudaGetLastError(), "quant_stream_kernel launch");
    if (rc) return rc;
    if (global_sel) {
        { LaunchScope scope(kKindSelect, stream);
        topk_select_kernel<<<1, kSelThreads, 0, stream>>>(a.scores, (int)nscore, (int)(nscore / 2), a.keep_flags); }
        rc = cuda_fail(cudaGetLastError(), "topk_select_kernel launch");
        if (rc) return rc;
        if (a.mask_bits || a.r_bf16) {
            int64_t n = a.M * (a.K / 8);
            LaunchScope scope(kKindSelect, stream);
            apply_global_mask_kernel<<<(unsigned)((n + 255) / 256), 256, 0, stream>>>(pattern, a.M, a.K, a.keep_flags,
                                                                                      a.mask_bits, a.r_bf16);
            rc = cuda_fail(cudaGetLastError(), "apply_global_mask_kernel launch");
        }
    }
    return rc;
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
