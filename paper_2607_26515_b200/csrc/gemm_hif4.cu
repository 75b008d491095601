// HiF4 GEMM of the rollout projection, Eq. (5):
//     Y[m, n] = sum_k a[m, k] w[n, k]  +  sum_k r[m, k] w[n, k]
// a = deq Q(X) and r = S(deq Q(dX)) arrive as exact bf16 images written by the quantizer pass;
// w = deq Q(W) stays packed (4.5 bit/value) in HBM and is expanded to bf16 inside the kernel.
// HiF4 values are q*(4+Mn)*2^e with q*(4+Mn) <= 49, i.e. exact in bf16, and bf16 x bf16 products
// are exact in fp32, so the tensor-core result differs from the fp64 definition only by the fp32
// accumulation order.  (HiF4's 2-bit level-1 mantissa and uniform S1P2 grid do not map onto the
// block-scaled FP4/FP8 MMA kinds, whose scales are powers of two.)
//
// One CTA computes a (128*MT) x BN tile of Y.  Warp roles:
//   warp 0      TMA producer: activation tiles (128x64 bf16, 128-byte swizzle) and the raw weight
//               codes (BN rows x 32 bytes) of each 64-wide k-block into a ring of stages
//   warp 1      MMA issuer: tcgen05.mma kind::f16, 128 x BN x 16, accumulators in tensor memory;
//               main and residual terms accumulate into the same TMEM tile against the same B tile
//   warps 2..9  expanders: 4-bit codes + block metadata -> bf16, written in the canonical K-major
//               128-byte-swizzled layout; afterwards the same warps run the epilogue
// Stage hand-off uses mbarriers; every wait is bounded and a timeout ends the kernel cleanly.
#include "common.cuh"
#include "ptx.cuh"

#include <algorithm>
#include <mutex>

namespace resq {

namespace {

constexpr int kBM = 128;          // rows per MMA (UMMA M)
constexpr int kBK = 64;           // one HiF4 block per row per stage
constexpr int kMaxBN = 256;
constexpr int kExpWarps = 8;
constexpr int kGemmThreads = 32 * (2 + kExpWarps);
constexpr int kATileBytes = kBM * kBK * 2;       // 16 KiB
constexpr int kBExpBytes = kMaxBN * kBK * 2;     // 32 KiB
constexpr int kBRawBytes = kMaxBN * (kBK / 2);   // 8 KiB
constexpr int kMaxStages = 4;

struct GemmParams {
    const uint32_t* w_meta;   // [N, K/64]
    int64_t M, N, K;
    int bn;                   // tile width (multiple of 16, <= 256)
    int kblocks_per_split;
    int splits;
    void* Y;
    int out_f32;
    int64_t ldy;
    float* partials;          // [splits, M, N] when splits > 1
    DeviceStatus* status;
};

template <int MT, bool RES>
struct SmemLayout {
    static constexpr int kStageBytes = MT * kATileBytes * (RES ? 2 : 1) + kBExpBytes + kBRawBytes;
    static constexpr int kStages = (224 * 1024 / kStageBytes) < kMaxStages ? (224 * 1024 / kStageBytes) : kMaxStages;
    static constexpr int kAMainOff = 0;
    static constexpr int kAResOff = MT * kATileBytes;
    static constexpr int kBExpOff = MT * kATileBytes * (RES ? 2 : 1);
    static constexpr int kBRawOff = kBExpOff + kBExpBytes;
    static constexpr int kBarOff = kStages * kStageBytes;
    static constexpr int kTotal = kBarOff + 256 + 1024;  // barriers + alignment slack
};

__device__ __forceinline__ void report_timeout(DeviceStatus* st, int where) {
    if (atomicCAS(&st->code, 0, (int)RESQ_ERR_TIMEOUT) == 0) {
        st->where = where;
        st->block = (int)blockIdx.x;
    }
}

// Expand one 32-bit word of 8 HiF4 codes (one level-2 group) into 8 bf16 values (one 16-byte chunk).
// bf16x2 trick: (0x4300 | q) is the bf16 number 128+q and (0x4300 | q<<4) is 128+16q, so one packed
// FMA with (scale, scale/16) and (-128 scale, -8 scale) yields q*scale exactly for both nibbles of a
// byte; the sign bits are then XOR-ed in.
__device__ __forceinline__ uint4 expand_hif4_chunk(uint32_t c, uint32_t meta, int chunk) {
    const uint32_t s = meta & 255u;
    const uint32_t Mn = s & 3u, E = s >> 2;
    const uint32_t e2 = (meta >> (8 + chunk)) & 1u;
    const uint32_t e3a = (meta >> (16 + 2 * chunk)) & 1u, e3b = (meta >> (17 + 2 * chunk)) & 1u;
    // bf16 bits of (4+Mn) * 2^x: exponent field x + 2 + 127, top mantissa bits Mn
    const uint32_t base = ((E + 77u + e2) << 7) | (Mn << 5);   // x = E - 52 + e2
    const uint32_t sa = base + (e3a << 7), sb = base + (e3b << 7);
    const uint32_t scale_a = sa | ((sa - 0x200u) << 16), scale_b = sb | ((sb - 0x200u) << 16);
    const uint32_t add_a = scale_a + 0x03800380u + 0x80008000u;  // -(128 * scale) in both halves
    const uint32_t add_b = scale_b + 0x03800380u + 0x80008000u;
    const uint32_t c4 = c << 4;
    uint32_t out[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        // y = byte i replicated into bytes 0 and 2
        uint32_t y = __byte_perm(c, 0u, (uint32_t)(i | (4 << 4) | (i << 8) | (4 << 12)));
        uint32_t t = (y & 0x00700007u) | 0x43004300u;
        uint32_t v;
        const uint32_t sc = i < 2 ? scale_a : scale_b, ad = i < 2 ? add_a : add_b;
        asm("fma.rn.bf16x2 %0, %1, %2, %3;" : "=r"(v) : "r"(t), "r"(sc), "r"(ad));
        // signs: bit 7 of byte i (odd element) -> bit 31; bit 3 of byte i (even element) -> bit 15
        uint32_t sg = __byte_perm(c, c4, (uint32_t)(0 | ((4 + i) << 4) | (0 << 8) | (i << 12)));
        out[i] = v ^ (sg & 0x80008000u);
    }
    return make_uint4(out[0], out[1], out[2], out[3]);
}

template <int MT, bool RES>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_hif4_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_r,
                 const __grid_constant__ CUtensorMap tmap_w, const GemmParams p) {
    using L = SmemLayout<MT, RES>;
    constexpr int S = L::kStages;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::kBarOff);
    uint64_t* raw_full = bars;            // [S] TMA bytes landed
    uint64_t* exp_full = bars + S;        // [S] expanded B tile written
    uint64_t* empty = bars + 2 * S;       // [S] MMAs that read the stage have completed
    uint64_t* acc_full = bars + 3 * S;    // [1] all MMAs of the tile have completed
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 3 * S + 1);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int bn = p.bn;
    const int64_t n0 = (int64_t)blockIdx.x * bn;
    const int64_t m0 = (int64_t)blockIdx.y * (kBM * MT);
    const int split = blockIdx.z;
    const int G = (int)(p.K / kBK);
    const int kb_begin = split * p.kblocks_per_split;
    const int kb_end = min(G, kb_begin + p.kblocks_per_split);
    const int nkb = kb_end - kb_begin;
    uint32_t tmem_cols = 32;
    while ((int)tmem_cols < MT * bn) tmem_cols <<= 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            ptx::mbar_init(&raw_full[s], 1);
            ptx::mbar_init(&exp_full[s], kExpWarps);
            ptx::mbar_init(&empty[s], 1);
        }
        ptx::mbar_init(acc_full, 1);
        *abort_flag = 0;
        ptx::mbar_fence_init();
    }
    if (warp == 1) ptx::tmem_alloc(tmem_slot, tmem_cols);
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            ptx::tma_prefetch_desc(&tmap_a);
            if (RES) ptx::tma_prefetch_desc(&tmap_r);
            ptx::tma_prefetch_desc(&tmap_w);
            const uint32_t tx = (uint32_t)(MT * kATileBytes * (RES ? 2 : 1) + bn * (kBK / 2));
            for (int i = 0; i < nkb; ++i) {
                const int s = i % S;
                if (i >= S && !ptx::mbar_wait(&empty[s], ((i / S) - 1) & 1, abort_flag)) {
                    report_timeout(p.status, 1);
                    break;
                }
                uint8_t* st = smem + (size_t)s * L::kStageBytes;
                ptx::mbar_arrive_expect_tx(&raw_full[s], tx);
                const int kb = kb_begin + i;
#pragma unroll
                for (int t = 0; t < MT; ++t) {
                    ptx::tma_load_2d(st + L::kAMainOff + t * kATileBytes, &tmap_a, &raw_full[s], kb * kBK,
                                     (int)(m0 + t * kBM));
                    if (RES)
                        ptx::tma_load_2d(st + L::kAResOff + t * kATileBytes, &tmap_r, &raw_full[s], kb * kBK,
                                         (int)(m0 + t * kBM));
                }
                ptx::tma_load_2d(st + L::kBRawOff, &tmap_w, &raw_full[s], kb * (kBK / 2), (int)n0);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t idesc = ptx::idesc_bf16_f32(kBM, bn);
            bool ok = true;
            for (int i = 0; i < nkb && ok; ++i) {
                const int s = i % S;
                const uint32_t par = (i / S) & 1;
                ok = ptx::mbar_wait(&raw_full[s], par, abort_flag) && ptx::mbar_wait(&exp_full[s], par, abort_flag);
                if (!ok) {
                    report_timeout(p.status, 2);
                    break;
                }
                ptx::tc_fence_after();
                uint8_t* st = smem + (size_t)s * L::kStageBytes;
                const uint32_t b_addr = ptx::smem_u32(st + L::kBExpOff);
#pragma unroll
                for (int k = 0; k < kBK / 16; ++k) {
                    const uint64_t bdesc = ptx::smem_desc_sw128_kmajor(b_addr + k * 32);
#pragma unroll
                    for (int t = 0; t < MT; ++t) {
                        const uint32_t d = tmem_base + (uint32_t)(t * bn);
                        const uint64_t adesc =
                            ptx::smem_desc_sw128_kmajor(ptx::smem_u32(st + L::kAMainOff + t * kATileBytes) + k * 32);
                        ptx::umma_bf16(d, adesc, bdesc, idesc, (i > 0 || k > 0) ? 1u : 0u);
                        if (RES) {
                            const uint64_t rdesc =
                                ptx::smem_desc_sw128_kmajor(ptx::smem_u32(st + L::kAResOff + t * kATileBytes) + k * 32);
                            ptx::umma_bf16(d, rdesc, bdesc, idesc, 1u);
                        }
                    }
                }
                ptx::umma_commit(&empty[s]);  // frees the stage when these MMAs have read it
            }
            ptx::umma_commit(acc_full);
        }
    } else {
        // ------------------------------------------------------------------ expanders
        const int ew = warp - 2;                      // 0..7
        const int rows_per_warp = bn / kExpWarps;     // bn is a multiple of 16: 2..32 rows
        const int r_begin = ew * rows_per_warp;
        // lane -> (row within a group of 4, chunk): a quarter-warp writes one full 128-byte row
        const int sub_row = lane >> 3, chunk = lane & 7;
        uint32_t meta_next = 0;
        {
            const int64_t n = n0 + r_begin + lane;
            if (lane < rows_per_warp && n < p.N && nkb > 0) meta_next = __ldg(p.w_meta + n * G + kb_begin);
        }
        bool ok = true;
        for (int i = 0; i < nkb && ok; ++i) {
            const int s = i % S;
            const uint32_t par = (i / S) & 1;
            const uint32_t meta_cur = meta_next;
            {
                const int64_t n = n0 + r_begin + lane;
                if (lane < rows_per_warp && n < p.N && i + 1 < nkb) meta_next = __ldg(p.w_meta + n * G + kb_begin + i + 1);
            }
            if (i >= S) ok = ptx::mbar_wait(&empty[s], ((i / S) - 1) & 1, abort_flag);
            ok = ok && ptx::mbar_wait(&raw_full[s], par, abort_flag);
            if (!ok) {
                report_timeout(p.status, 3);
                break;
            }
            uint8_t* st = smem + (size_t)s * L::kStageBytes;
            const uint32_t* raw = reinterpret_cast<const uint32_t*>(st + L::kBRawOff);
            uint8_t* bexp = st + L::kBExpOff;
            for (int rr = 0; rr < rows_per_warp; rr += 4) {
                const int rl = rr + sub_row;                       // row inside this warp's slice
                const uint32_t meta = __shfl_sync(0xFFFFFFFFu, meta_cur, rl & 31);
                if (rl < rows_per_warp) {
                    const int r = r_begin + rl;
                    const uint32_t c = raw[r * 8 + chunk];
                    const uint4 v = expand_hif4_chunk(c, meta, chunk);
                    *reinterpret_cast<uint4*>(bexp + r * 128 + ((chunk ^ (r & 7)) << 4)) = v;
                }
            }
            ptx::fence_proxy_async_smem();  // make the generic-proxy stores visible to the tensor core
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&exp_full[s]);
        }
        // ------------------------------------------------------------------ epilogue (same warps)
        if (nkb > 0 && ptx::mbar_wait(acc_full, 0, abort_flag)) {
            ptx::tc_fence_after();
            const int quad = warp & 3;            // TMEM lanes 32*quad .. 32*quad+31 belong to this warp
            const int half = ew >> 2;             // two warps share a quadrant: split the column chunks
            const int nchunks = (bn + 31) / 32;
#pragma unroll 1
            for (int t = 0; t < MT; ++t) {
                const int64_t m = m0 + t * kBM + quad * 32 + lane;
                for (int cchunk = half; cchunk < nchunks; cchunk += 2) {
                    uint32_t v[32];
                    const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(t * bn + cchunk * 32);
                    if (cchunk * 32 + 32 <= bn) {
                        ptx::tmem_ld_32x32(taddr, v);
                    } else {  // bn % 32 == 16: last chunk has 16 columns
                        uint32_t h[16];
                        ptx::tmem_ld_32x16(taddr, h);
#pragma unroll
                        for (int j = 0; j < 16; ++j) { v[j] = h[j]; v[16 + j] = 0; }
                    }
                    ptx::tmem_ld_wait();
                    if (m >= p.M) continue;
                    const int64_t nb = n0 + cchunk * 32;
                    int64_t valid64 = p.N - nb;
                    if (valid64 > bn - cchunk * 32) valid64 = bn - cchunk * 32;
                    const int valid = valid64 > 32 ? 32 : (int)valid64;
                    if (valid <= 0) continue;
                    if (p.splits > 1) {
                        float* dst = p.partials + ((int64_t)split * p.M + m) * p.N + nb;
                        for (int j = 0; j < valid; ++j) dst[j] = __uint_as_float(v[j]);
                    } else if (p.out_f32) {
                        float* dst = reinterpret_cast<float*>(p.Y) + m * p.ldy + nb;
                        if (valid == 32) {
#pragma unroll
                            for (int j = 0; j < 32; j += 4)
                                *reinterpret_cast<uint4*>(dst + j) = make_uint4(v[j], v[j + 1], v[j + 2], v[j + 3]);
                        } else {
                            for (int j = 0; j < valid; ++j) dst[j] = __uint_as_float(v[j]);
                        }
                    } else {
                        __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(p.Y) + m * p.ldy + nb;
                        if (valid == 32) {
                            uint32_t o[16];
#pragma unroll
                            for (int j = 0; j < 16; ++j) {
                                __nv_bfloat162 b = __floats2bfloat162_rn(__uint_as_float(v[2 * j]), __uint_as_float(v[2 * j + 1]));
                                o[j] = *reinterpret_cast<uint32_t*>(&b);
                            }
#pragma unroll
                            for (int j = 0; j < 16; j += 4)
                                *reinterpret_cast<uint4*>(dst + 2 * j) = make_uint4(o[j], o[j + 1], o[j + 2], o[j + 3]);
                        } else {
                            for (int j = 0; j < valid; ++j) dst[j] = __float2bfloat16_rn(__uint_as_float(v[j]));
                        }
                    }
                }
            }
        } else if (nkb > 0) {
            report_timeout(p.status, 4);
        }
    }
    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, tmem_cols);
    }
}

// Sum the split-K partial tiles in a fixed order (split 0, 1, ...) and write Y.
__global__ void splitk_reduce_kernel(const float* __restrict__ partials, int splits, int64_t M, int64_t N, void* Y,
                                     int out_f32, int64_t ldy) {
    int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= M * N) return;
    int64_t m = idx / N, n = idx % N;
    float acc = partials[idx];
    for (int s = 1; s < splits; ++s) acc += partials[(int64_t)s * M * N + idx];
    if (out_f32) reinterpret_cast<float*>(Y)[m * ldy + n] = acc;
    else reinterpret_cast<__nv_bfloat16*>(Y)[m * ldy + n] = __float2bfloat16_rn(acc);
}

// ---- host side -----------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
    });
    return fn;
}

int make_tmap_2d(CUtensorMap* m, CUtensorMapDataType dt, int elem_bytes, const void* base, uint64_t inner, uint64_t rows,
                 uint64_t row_stride_bytes, uint32_t box_inner, uint32_t box_rows, CUtensorMapSwizzle sw) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) {
        set_last_error("cuTensorMapEncodeTiled is not available from the driver");
        return RESQ_ERR_CUDA;
    }
    cuuint64_t dims[2] = {inner, rows};
    cuuint64_t strides[1] = {row_stride_bytes};
    cuuint32_t box[2] = {box_inner, box_rows};
    cuuint32_t estr[2] = {1, 1};
    (void)elem_bytes;
    CUresult r = fn(m, dt, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        set_last_error("cuTensorMapEncodeTiled failed with CUresult %d", (int)r);
        return RESQ_ERR_CUDA;
    }
    return RESQ_OK;
}

struct TileChoice {
    int mt, bn, splits;
};

// Pick the tile width and K split so that the grid covers the 148 SMs in as few, as full waves as possible.
TileChoice choose_tile(int64_t M, int64_t N, int64_t K, bool res) {
    const int sms = 148;
    const int G = (int)(K / kBK);
    TileChoice best{1, 256, 1};
    double best_cost = 1e300;
    for (int mt = 1; mt <= (res ? 1 : 2); ++mt) {
        if (mt == 2 && M <= kBM) continue;
        const int64_t mtiles = (M + kBM * mt - 1) / (kBM * mt);
        for (int bn = 256; bn >= 64; bn -= 32) {
            if (mt * bn > 512) continue;
            const int64_t ntiles = (N + bn - 1) / bn;
            for (int splits = 1; splits <= 8; splits *= 2) {
                if (G / splits < 4 && splits > 1) break;
                const int64_t ctas = mtiles * ntiles * splits;
                const int64_t waves = (ctas + sms - 1) / sms;
                const int kb = (G + splits - 1) / splits;
                // per-CTA time model (arbitrary units): MMA time scales with bn*mt*(1+res) per k-block, floored by
                // the expander time (scales with bn); fixed prologue/epilogue cost; split-K adds a reduce pass
                const double mma = (double)mt * bn * (res ? 2.0 : 1.0) / 256.0;
                const double expand = bn / 256.0 * 1.0;
                const double per_kb = std::max(mma, expand) + 0.08;
                double cost = waves * (kb * per_kb + 6.0 + 0.02 * mt * bn);
                if (splits > 1) cost += 8.0 + (double)M * N * splits / 3.0e5;
                if (cost < best_cost) {
                    best_cost = cost;
                    best = TileChoice{mt, bn, splits};
                }
            }
        }
    }
    return best;
}

template <int MT, bool RES>
int launch_variant(const GemmArgs& g, const TileChoice& tc, cudaStream_t stream) {
    using L = SmemLayout<MT, RES>;
    CUtensorMap ta, tr, tw;
    int rc = make_tmap_2d(&ta, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, g.a_bf16, (uint64_t)g.K, (uint64_t)g.M,
                          (uint64_t)g.K * 2, kBK, kBM, CU_TENSOR_MAP_SWIZZLE_128B);
    if (rc) return rc;
    rc = make_tmap_2d(&tr, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, RES ? g.r_bf16 : g.a_bf16, (uint64_t)g.K, (uint64_t)g.M,
                      (uint64_t)g.K * 2, kBK, kBM, CU_TENSOR_MAP_SWIZZLE_128B);
    if (rc) return rc;
    rc = make_tmap_2d(&tw, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, g.w_codes, (uint64_t)g.K / 2, (uint64_t)g.N,
                      (uint64_t)g.K / 2, kBK / 2, (uint32_t)tc.bn, CU_TENSOR_MAP_SWIZZLE_NONE);
    if (rc) return rc;
    GemmParams p;
    p.w_meta = static_cast<const uint32_t*>(g.w_side);
    p.M = g.M;
    p.N = g.N;
    p.K = g.K;
    p.bn = tc.bn;
    const int G = (int)(g.K / kBK);
    p.splits = tc.splits;
    p.kblocks_per_split = (G + tc.splits - 1) / tc.splits;
    p.Y = g.Y;
    p.out_f32 = g.out_dtype == RESQ_OUT_F32;
    p.ldy = g.ldy;
    p.partials = g.splitk_partials;
    p.status = g.status;
    auto kern = gemm_hif4_kernel<MT, RES>;
    static std::once_flag once;
    static cudaError_t attr_err = cudaSuccess;
    std::call_once(once, [&] {
        attr_err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kTotal);
    });
    if (attr_err != cudaSuccess) return cuda_fail(attr_err, "cudaFuncSetAttribute(gemm)");
    dim3 grid((unsigned)((g.N + tc.bn - 1) / tc.bn), (unsigned)((g.M + kBM * MT - 1) / (kBM * MT)), (unsigned)tc.splits);
    {
        LaunchScope scope(kKindGemm, stream);
        kern<<<grid, kGemmThreads, L::kTotal, stream>>>(ta, tr, tw, p);
    }
    rc = cuda_fail(cudaGetLastError(), "gemm_hif4_kernel launch");
    if (rc) return rc;
    if (tc.splits > 1) {
        int64_t n = g.M * g.N;
        LaunchScope scope(kKindReduce, stream);
        splitk_reduce_kernel<<<(unsigned)((n + 255) / 256), 256, 0, stream>>>(g.splitk_partials, tc.splits, g.M, g.N, g.Y,
                                                                             p.out_f32, g.ldy);
        rc = cuda_fail(cudaGetLastError(), "splitk_reduce_kernel launch");
    }
    return rc;
}

}  // namespace

int gemm_hif4_pick_splits(int64_t M, int64_t N, int64_t K) {
    // the workspace must cover the larger of the two possible choices (with / without residual)
    return std::max(choose_tile(M, N, K, false).splits, choose_tile(M, N, K, true).splits);
}

int launch_gemm_hif4(const GemmArgs& g, cudaStream_t stream) {
    const bool res = g.r_bf16 != nullptr;
    TileChoice tc = choose_tile(g.M, g.N, g.K, res);
    if (tc.splits > 1 && (!g.splitk_partials || tc.splits > g.splits)) tc.splits = 1;
    if (res) return launch_variant<1, true>(g, tc, stream);
    if (tc.mt == 2) return launch_variant<2, false>(g, tc, stream);
    return launch_variant<1, false>(g, tc, stream);
}

}  // namespace resq
