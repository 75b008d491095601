// HiF4 GEMM of the rollout projection, Eq. (5):
//     Y[m, n] = sum_k a[m, k] w[n, k]  +  sum_k r[m, k] w[n, k]
// a = deq Q(X) and r = S(deq Q(dX)) arrive as exact bf16 images written by the quantizer pass;
// w = deq Q(W) stays packed (4.5 bit/value) in HBM and is expanded to bf16 inside the kernel.
// HiF4 values are q*(4+Mn)*2^e with q*(4+Mn) <= 49, i.e. exact in bf16, and bf16 x bf16 products
// are exact in fp32, so the tensor-core result differs from the fp64 definition only by the fp32
// accumulation order.  (HiF4's 2-bit level-1 mantissa and uniform S1P2 grid do not map onto the
// block-scaled FP4/FP8 MMA kinds, whose scales are powers of two.)
//
// Persistent kernel: one CTA per SM walks a static list of (128*MT) x BN output tiles (x K splits).
// Warp roles (16 warps):
//   warp 0       TMA producer of the activation tiles (128x64 bf16, 128-byte swizzle), main + residual
//   warp 1       MMA issuer: tcgen05.mma kind::f16, 128 x BN x 16, fp32 accumulators in tensor memory,
//                double-buffered across tiles; main and residual terms accumulate into the same tile
//                against the same expanded weight tile
//   warp 2       TMA producer of the raw weight codes (BN rows x 32 bytes per 64-wide k-block)
//   warps 4..7   epilogue: TMEM -> registers -> global (bf16 / fp32 / split-K partial), overlapped with
//                the next tile's main loop
//   warps 8..15  expanders: 4-bit codes + block metadata -> bf16 in the canonical K-major
//                128-byte-swizzled layout
// Three independent shared-memory rings (activation tiles, raw codes, expanded weights) decouple the
// TMA latency from the expansion latency.  Every wait is bounded; a timeout ends the kernel cleanly.
#include "common.cuh"
#include "ptx.cuh"
#include "expand.cuh"

#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <mutex>

namespace resq {

namespace {

constexpr int kBM = 128;          // rows per MMA (UMMA M)
constexpr int kBK = 64;           // one HiF4 block per row per stage
constexpr int kMaxBN = 256;
constexpr int kExpWarps = 8;
constexpr int kFirstEpiWarp = 4;
constexpr int kFirstExpWarp = 8;
constexpr int kGemmThreads = 32 * (kFirstExpWarp + kExpWarps);
constexpr int kATileBytes = kBM * kBK * 2;       // 16 KiB
constexpr int kMaxRing = 8;
constexpr int kSmemBudget = 232448;              // opt-in limit per block on sm_100
constexpr int kTmemCols = 512;

struct GemmParams {
    const void* w_side;       // HiF4: u32 [N, K/64]; MXFP4: u8 [N, K/32]
    int64_t M, N, K;
    int bn;                   // MMA N (multiple of 32, <= 256)
    int nt;                   // N sub-tiles per CTA tile (1 or 2): the tile is 128*MT x nt*bn
    int kblocks_per_split;
    int splits;
    int ntiles_m, ntiles_n, num_tiles;
    int sa, sr, se;           // ring depths: activation tiles, raw codes, expanded weights
    int acc_bufs;             // 2 if two accumulators fit in tensor memory, else 1
    void* Y;
    int out_f32;
    int64_t ldy;
    float* partials;          // [splits, M, N] when splits > 1
    DeviceStatus* status;
#ifdef RESQ_TIMELINE
    int debug;                // bit 4 (16): accumulate per-role cycle counters after the status word
#endif
};

__device__ __forceinline__ void report_timeout(DeviceStatus* st, int where) {
    if (atomicCAS(&st->code, 0, (int)RESQ_ERR_TIMEOUT) == 0) {
        st->where = where;
        st->block = (int)blockIdx.x;
    }
}

// Profiling builds (-DRESQ_TIMELINE) only: cycles spent per role, summed over CTAs into the 64-bit counters that
// follow the status word.  The shipped kernels carry no instrumentation.
#ifdef RESQ_TIMELINE
struct Trace {
    unsigned long long* out;
    long long t0;
    __device__ __forceinline__ void begin() { if (out) t0 = clock64(); }
    __device__ __forceinline__ void end(int slot) { if (out) atomicAdd(out + slot, (unsigned long long)(clock64() - t0)); }
};
#else
struct Trace {
    __device__ __forceinline__ void begin() {}
    __device__ __forceinline__ void end(int) {}
};
#endif

struct TileCoord {
    int64_t m0, n0;
    int split, kb_begin, nkb;
};

__device__ __forceinline__ TileCoord decode_tile(const GemmParams& p, int tile, int mt_rows) {
    TileCoord t;
    t.split = tile % p.splits;
    const int rest = tile / p.splits;
    t.n0 = (int64_t)(rest % p.ntiles_n) * (p.bn * p.nt);
    t.m0 = (int64_t)(rest / p.ntiles_n) * mt_rows;
    const int G = (int)(p.K / kBK);
    t.kb_begin = t.split * p.kblocks_per_split;
    t.nkb = min(G, t.kb_begin + p.kblocks_per_split) - t.kb_begin;
    if (t.nkb < 0) t.nkb = 0;
    return t;
}

template <int MT, bool RES, int TN, int FMT>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_hif4_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_r,
                 const __grid_constant__ CUtensorMap tmap_w, const GemmParams p) {
    constexpr int kAStage = MT * kATileBytes * (RES ? 2 : 1);
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    constexpr int tile_n = TN;                       // CTA tile width
    constexpr int bn = TN > kMaxBN ? kMaxBN : TN;    // MMA N
    constexpr int nt = TN / bn;                      // MMAs side by side in N
    const int SA = p.sa, SR = p.sr, SE = p.se;
    constexpr int exp_stage = tile_n * 128, raw_stage = tile_n * 32;
    uint8_t* ring_a = smem;
    uint8_t* ring_e = ring_a + (size_t)SA * kAStage;
    uint8_t* ring_r = ring_e + (size_t)SE * exp_stage;
    uint64_t* bars = reinterpret_cast<uint64_t*>(ring_r + (size_t)SR * raw_stage);
    uint64_t* a_full = bars;                   // [kMaxRing] TMA bytes of an activation stage landed
    uint64_t* a_empty = bars + kMaxRing;       // [kMaxRing] MMAs that read the stage have completed
    uint64_t* r_full = bars + 2 * kMaxRing;    // raw codes landed
    uint64_t* r_empty = bars + 3 * kMaxRing;   // expanders have consumed the raw codes
    uint64_t* e_full = bars + 4 * kMaxRing;    // expanded weight tile written
    uint64_t* e_empty = bars + 5 * kMaxRing;   // MMAs that read the expanded tile have completed
    uint64_t* acc_full = bars + 6 * kMaxRing;  // [2] accumulator complete
    uint64_t* acc_empty = acc_full + 2;        // [2] accumulator drained by the epilogue
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = (int)(p.K / kBK);

    if (threadIdx.x == 0) {
        for (int s = 0; s < kMaxRing; ++s) {
            ptx::mbar_init(&a_full[s], 1);
            ptx::mbar_init(&a_empty[s], 1);
            ptx::mbar_init(&r_full[s], 1);
            ptx::mbar_init(&r_empty[s], kExpWarps);
            ptx::mbar_init(&e_full[s], kExpWarps);
            ptx::mbar_init(&e_empty[s], 1);
        }
        for (int b = 0; b < 2; ++b) {
            ptx::mbar_init(&acc_full[b], 1);
            ptx::mbar_init(&acc_empty[b], 4);
        }
        *abort_flag = 0;
        ptx::mbar_fence_init();
    }
    if (warp == 1) ptx::tmem_alloc(tmem_slot, kTmemCols);
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
#ifdef RESQ_TIMELINE
    Trace tr{(p.debug & 16) ? reinterpret_cast<unsigned long long*>(p.status) + 8 : nullptr, 0};
    const long long t_kernel0 = clock64();
#else
    Trace tr;
#endif
    // programmatic dependent launch: see gemm_pair.cu (the weight side does not depend on the quantizer)
    pdl_trigger();
    if (!(warp == 2 || warp >= kFirstExpWarp)) pdl_wait();

    if (warp == 0) {
        // ------------------------------------------------------------------ activation producer
        if (lane == 0) {
            ptx::tma_prefetch_desc(&tmap_a);
            if (RES) ptx::tma_prefetch_desc(&tmap_r);
            uint32_t it = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < p.num_tiles && ok; tile += gridDim.x) {
                const TileCoord tc = decode_tile(p, tile, kBM * MT);
                for (int i = 0; i < tc.nkb; ++i, ++it) {
                    const int s = it % SA;
                    tr.begin();
                    const bool got = ptx::mbar_wait(&a_empty[s], ((it / SA) & 1) ^ 1, abort_flag);
                    tr.end(0);
                    if (!got) {
                        report_timeout(p.status, 1);
                        ok = false;
                        break;
                    }
                    uint8_t* st = ring_a + (size_t)s * kAStage;
                    ptx::mbar_arrive_expect_tx(&a_full[s], (uint32_t)kAStage);
                    const int kx = (tc.kb_begin + i) * kBK;
#pragma unroll
                    for (int t = 0; t < MT; ++t) {
                        ptx::tma_load_2d(st + t * kATileBytes, &tmap_a, &a_full[s], kx, (int)(tc.m0 + t * kBM));
                        if (RES)
                            ptx::tma_load_2d(st + (MT + t) * kATileBytes, &tmap_r, &a_full[s], kx, (int)(tc.m0 + t * kBM));
                    }
                }
            }
        }
    } else if (warp == 2) {
        // ------------------------------------------------------------------ raw weight-code producer
        if (lane == 0) {
            ptx::tma_prefetch_desc(&tmap_w);
            uint32_t it = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < p.num_tiles && ok; tile += gridDim.x) {
                const TileCoord tc = decode_tile(p, tile, kBM * MT);
                for (int i = 0; i < tc.nkb; ++i, ++it) {
                    const int s = it % SR;
                    tr.begin();
                    const bool got = ptx::mbar_wait(&r_empty[s], ((it / SR) & 1) ^ 1, abort_flag);
                    tr.end(1);
                    if (!got) {
                        report_timeout(p.status, 5);
                        ok = false;
                        break;
                    }
                    ptx::mbar_arrive_expect_tx(&r_full[s], (uint32_t)raw_stage);
#pragma unroll
                    for (int j = 0; j < nt; ++j)
                        ptx::tma_load_2d(ring_r + (size_t)s * raw_stage + (size_t)j * bn * 32, &tmap_w, &r_full[s],
                                         (tc.kb_begin + i) * (kBK / 2), (int)(tc.n0 + j * bn));
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t idesc = ptx::idesc_bf16_f32(kBM, bn);
            uint32_t it = 0;
            int local_tile = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < p.num_tiles && ok; tile += gridDim.x, ++local_tile) {
                const TileCoord tc = decode_tile(p, tile, kBM * MT);
                if (tc.nkb == 0) continue;
                const int buf = p.acc_bufs == 2 ? (local_tile & 1) : 0;
                const uint32_t use = p.acc_bufs == 2 ? (uint32_t)(local_tile >> 1) : (uint32_t)local_tile;
                tr.begin();
                const bool got_acc = ptx::mbar_wait(&acc_empty[buf], (use & 1) ^ 1, abort_flag);
                tr.end(4);
                if (!got_acc) {
                    report_timeout(p.status, 6);
                    break;
                }
                ptx::tc_fence_after();
                const uint32_t d0 = tmem_base + (uint32_t)(buf * MT * tile_n);
                for (int i = 0; i < tc.nkb; ++i, ++it) {
                    const int sa = it % SA, se = it % SE;
                    tr.begin();
                    ok = ptx::mbar_wait(&a_full[sa], (it / SA) & 1, abort_flag);
                    tr.end(2);
                    tr.begin();
                    ok = ok && ptx::mbar_wait(&e_full[se], (it / SE) & 1, abort_flag);
                    tr.end(3);
                    if (!ok) {
                        report_timeout(p.status, 2);
                        break;
                    }
                    tr.begin();
                    ptx::tc_fence_after();
                    const uint32_t a_addr = ptx::smem_u32(ring_a + (size_t)sa * kAStage);
                    const uint32_t b_addr = ptx::smem_u32(ring_e + (size_t)se * exp_stage);
#pragma unroll
                    for (int k = 0; k < kBK / 16; ++k) {
#pragma unroll
                        for (int j = 0; j < nt; ++j) {
                            const uint64_t bdesc = ptx::smem_desc_sw128_kmajor(b_addr + j * bn * 128 + k * 32);
#pragma unroll
                            for (int t = 0; t < MT; ++t) {
                                const uint32_t d = d0 + (uint32_t)((t * nt + j) * bn);
                                ptx::umma_bf16(d, ptx::smem_desc_sw128_kmajor(a_addr + t * kATileBytes + k * 32), bdesc,
                                               idesc, (i > 0 || k > 0) ? 1u : 0u);
                                if (RES)
                                    ptx::umma_bf16(d, ptx::smem_desc_sw128_kmajor(a_addr + (MT + t) * kATileBytes + k * 32),
                                                   bdesc, idesc, 1u);
                            }
                        }
                    }
                    ptx::umma_commit(&a_empty[sa]);  // frees both stages when these MMAs have read them
                    ptx::umma_commit(&e_empty[se]);
                    tr.end(5);
                }
                if (ok) ptx::umma_commit(&acc_full[buf]);
            }
        }
    } else if (warp >= kFirstExpWarp) {
        // ------------------------------------------------------------------ expanders
        const int ew = warp - kFirstExpWarp;          // 0..7
        constexpr int rows_per_warp = tile_n / kExpWarps;  // 8, 16, 32 or 64 rows
        const int r_begin = ew * rows_per_warp;
        // lane -> (row within a group of 4, chunk): a quarter-warp writes one full 128-byte row
        const int sub_row = lane >> 3, chunk = lane & 7;
        uint32_t it = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < p.num_tiles && ok; tile += gridDim.x) {
            const TileCoord tc = decode_tile(p, tile, kBM * MT);
            // lane l owns the metadata of rows l and 32 + l of this warp's slice
            const int64_t n = tc.n0 + r_begin + lane;
            const bool row_ok0 = lane < rows_per_warp && n < p.N;
            const bool row_ok1 = lane + 32 < rows_per_warp && n + 32 < p.N;
            // per row and k-block: one u32 of HiF4 metadata, or two E8M0 bytes (one u16) for MXFP4
            auto load_side = [&](int64_t row, int kb) -> uint32_t {
                if (FMT == kHiF4) return ptx::ld_nc_u32(reinterpret_cast<const uint32_t*>(p.w_side) + row * G + kb);
                return ptx::ld_nc_u16(reinterpret_cast<const uint16_t*>(p.w_side) + row * G + kb);
            };
            uint32_t meta_next0 = (row_ok0 && tc.nkb > 0) ? load_side(n, tc.kb_begin) : 0u;
            uint32_t meta_next1 = (row_ok1 && tc.nkb > 0) ? load_side(n + 32, tc.kb_begin) : 0u;
            for (int i = 0; i < tc.nkb; ++i, ++it) {
                const uint32_t meta_cur0 = meta_next0, meta_cur1 = meta_next1;
                if (i + 1 < tc.nkb) {  // prefetch the next k-block
                    meta_next0 = row_ok0 ? load_side(n, tc.kb_begin + i + 1) : 0u;
                    meta_next1 = row_ok1 ? load_side(n + 32, tc.kb_begin + i + 1) : 0u;
                }
                const int sr = it % SR, se = it % SE;
                if (ew == 0 && lane == 0) tr.begin();
                ok = ptx::mbar_wait(&e_empty[se], ((it / SE) & 1) ^ 1, abort_flag);
                if (ew == 0 && lane == 0) { tr.end(6); tr.begin(); }
                ok = ok && ptx::mbar_wait(&r_full[sr], (it / SR) & 1, abort_flag);
                if (ew == 0 && lane == 0) { tr.end(7); tr.begin(); }
                if (!ok) {
                    report_timeout(p.status, 3);
                    break;
                }
                const uint32_t* raw = reinterpret_cast<const uint32_t*>(ring_r + (size_t)sr * raw_stage);
                uint8_t* bexp = ring_e + (size_t)se * exp_stage;
                // all loads and shuffles first, then the arithmetic: independent chains interleave
                constexpr int kIters = rows_per_warp / 4;
                uint32_t cw[kIters], mw[kIters];
#pragma unroll
                for (int q = 0; q < kIters; ++q) {
                    const int rl = q * 4 + sub_row;
                    mw[q] = __shfl_sync(0xFFFFFFFFu, q < 8 ? meta_cur0 : meta_cur1, rl & 31);
                    cw[q] = raw[(r_begin + rl) * 8 + chunk];
                }
                // the reads above (generic proxy) are ordered before the TMA producer's next load into this slot (async
                // proxy) by a proxy fence; see gemm_pair.cu
                ptx::fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&r_empty[sr]);  // the raw codes are in registers now
#pragma unroll
                for (int q = 0; q < kIters; ++q) {
                    const int r = r_begin + q * 4 + sub_row;
                    const uint4 v = FMT == kHiF4 ? expand_hif4_chunk(cw[q], mw[q], chunk)
                                                 : expand_mxfp4_chunk(cw[q], (mw[q] >> (8 * (chunk >> 2))) & 255u);
                    *reinterpret_cast<uint4*>(bexp + r * 128 + ((chunk ^ (r & 7)) << 4)) = v;
                }
                ptx::fence_proxy_async_smem();  // make the generic-proxy stores visible to the tensor core
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&e_full[se]);
                if (ew == 0 && lane == 0) tr.end(8);
            }
        }
    } else if (warp >= kFirstEpiWarp) {
        // ------------------------------------------------------------------ epilogue
        const int quad = warp & 3;  // TMEM lanes 32*quad .. 32*quad+31 belong to this warp
        constexpr int nchunks = tile_n / 32;
        int local_tile = 0;
        for (int tile = blockIdx.x; tile < p.num_tiles; tile += gridDim.x, ++local_tile) {
            const TileCoord tc = decode_tile(p, tile, kBM * MT);
            if (tc.nkb == 0) continue;
            const int buf = p.acc_bufs == 2 ? (local_tile & 1) : 0;
            const uint32_t use = p.acc_bufs == 2 ? (uint32_t)(local_tile >> 1) : (uint32_t)local_tile;
            if (quad == 0 && lane == 0) tr.begin();
            const bool got_full = ptx::mbar_wait(&acc_full[buf], use & 1, abort_flag);
            if (quad == 0 && lane == 0) { tr.end(9); tr.begin(); }
            if (!got_full) {
                report_timeout(p.status, 4);
                break;
            }
            ptx::tc_fence_after();
#pragma unroll 1
            for (int t = 0; t < MT; ++t) {
                const int64_t m = tc.m0 + t * kBM + quad * 32 + lane;
#pragma unroll 1
                for (int cc = 0; cc < nchunks; ++cc) {
                    uint32_t v[32];
                    ptx::tmem_ld_32x32(tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)((buf * MT + t) * tile_n + cc * 32), v);
                    ptx::tmem_ld_wait();
                    if (t == MT - 1 && cc == nchunks - 1) {
                        // everything of this accumulator is in registers: hand it back to the MMA warp
                        ptx::tc_fence_before();
                        __syncwarp();
                        if (lane == 0) ptx::mbar_arrive(&acc_empty[buf]);
                    }
                    if (m >= p.M) continue;
                    const int64_t nb = tc.n0 + cc * 32;
                    const int64_t left = p.N - nb;
                    if (left <= 0) continue;
                    if (p.splits > 1) {
                        float* dst = p.partials + ((int64_t)tc.split * p.M + m) * p.N + nb;
                        if (left >= 32 && (p.N & 3) == 0) {
#pragma unroll
                            for (int j = 0; j < 32; j += 4)
                                *reinterpret_cast<uint4*>(dst + j) = make_uint4(v[j], v[j + 1], v[j + 2], v[j + 3]);
                        } else {
#pragma unroll
                            for (int j = 0; j < 32; ++j)
                                if (j < left) dst[j] = __uint_as_float(v[j]);
                        }
                    } else if (p.out_f32) {
                        float* dst = reinterpret_cast<float*>(p.Y) + m * p.ldy + nb;
                        if (left >= 32) {
#pragma unroll
                            for (int j = 0; j < 32; j += 4)
                                *reinterpret_cast<uint4*>(dst + j) = make_uint4(v[j], v[j + 1], v[j + 2], v[j + 3]);
                        } else {
#pragma unroll
                            for (int j = 0; j < 32; ++j)
                                if (j < left) dst[j] = __uint_as_float(v[j]);
                        }
                    } else {
                        __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(p.Y) + m * p.ldy + nb;
                        if (left >= 32) {
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
#pragma unroll
                            for (int j = 0; j < 32; ++j)
                                if (j < left) dst[j] = __float2bfloat16_rn(__uint_as_float(v[j]));
                        }
                    }
                }
            }
            if (quad == 0 && lane == 0) tr.end(10);
        }
    }
    ptx::tc_fence_before();
    __syncthreads();
#ifdef RESQ_TIMELINE
    if (tr.out && threadIdx.x == 0) {
        atomicAdd(tr.out + 11, (unsigned long long)(clock64() - t_kernel0));
        atomicAdd(tr.out + 12, 1ull);
    }
#endif
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, kTmemCols);
    }
}

// Sum the split-K partial tiles in a fixed order (split 0, 1, ...) and write Y.  Four outputs per thread
// (128-bit loads) when N is a multiple of 4.
__global__ void splitk_reduce_kernel(const float* __restrict__ partials, int splits, int64_t M, int64_t N, void* Y,
                                     int out_f32, int64_t ldy) {
    pdl_wait();     // the partial tiles come from the GEMM kernel just before
    pdl_trigger();
    const int64_t total = M * N;
    if ((N & 3) == 0) {
        const int64_t idx = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * 4;
        if (idx >= total) return;
        const int64_t m = idx / N, n = idx % N;
        float4 acc = *reinterpret_cast<const float4*>(partials + idx);
        for (int s = 1; s < splits; ++s) {
            const float4 t = *reinterpret_cast<const float4*>(partials + (int64_t)s * total + idx);
            acc.x += t.x; acc.y += t.y; acc.z += t.z; acc.w += t.w;
        }
        if (out_f32) {
            float* o = reinterpret_cast<float*>(Y) + m * ldy + n;
            o[0] = acc.x; o[1] = acc.y; o[2] = acc.z; o[3] = acc.w;
        } else {
            __nv_bfloat16* o = reinterpret_cast<__nv_bfloat16*>(Y) + m * ldy + n;
            __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y), hi = __floats2bfloat162_rn(acc.z, acc.w);
            if ((reinterpret_cast<uintptr_t>(o) & 7u) == 0) {
                *reinterpret_cast<uint2*>(o) = make_uint2(*reinterpret_cast<uint32_t*>(&lo), *reinterpret_cast<uint32_t*>(&hi));
            } else {
                o[0] = lo.x; o[1] = lo.y; o[2] = hi.x; o[3] = hi.y;
            }
        }
        return;
    }
    const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= total) return;
    const int64_t m = idx / N, n = idx % N;
    float acc = partials[idx];
    for (int s = 1; s < splits; ++s) acc += partials[(int64_t)s * total + idx];
    if (out_f32) reinterpret_cast<float*>(Y)[m * ldy + n] = acc;
    else reinterpret_cast<__nv_bfloat16*>(Y)[m * ldy + n] = __float2bfloat16_rn(acc);
}

}  // namespace

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

int make_tmap_2d(CUtensorMap* m, CUtensorMapDataType dt, const void* base, uint64_t inner, uint64_t rows,
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
    CUresult r = fn(m, dt, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        set_last_error("cuTensorMapEncodeTiled failed with CUresult %d", (int)r);
        return RESQ_ERR_CUDA;
    }
    return RESQ_OK;
}

int launch_splitk_reduce(const GemmArgs& g, int splits, cudaStream_t stream) {
    if (splits <= 1) return RESQ_OK;
    const int64_t n = (g.N & 3) == 0 ? g.M * g.N / 4 : g.M * g.N;
    LaunchScope scope(kKindReduce, stream);
    return cuda_fail(launch_kernel(splitk_reduce_kernel, dim3((unsigned)((n + 255) / 256)), dim3(256), 0, stream,
                                   (const float*)g.splitk_partials, splits, g.M, g.N, g.Y, (int)(g.out_dtype == RESQ_OUT_F32), g.ldy),
                     "splitk_reduce_kernel launch");
}

int launch_gemm_pair(const GemmArgs& g, int tn, int splits, cudaStream_t stream);
int launch_gemm_pair_streamk(const GemmArgs& g, cudaStream_t stream);
int launch_gemm_pair_plainw(const GemmArgs& g, int tn, int splits, bool streamk, cudaStream_t stream);
size_t gemm_pair_streamk_scratch_bytes();

namespace {

struct TileChoice {
    int mt, bn, splits, nt;
    int pair_tn;  // > 0: use the CTA-pair kernel with a 256 x pair_tn tile
};

// Pick the tile width and K split so that the persistent grid covers the 148 SMs evenly.
// Calls with at most this many rows take the single-CTA kernel (one 128-row MMA tile); the CTA-pair kernel computes
// 256-row tiles whatever M is (rows past M are zero-filled and never stored).
int pair_min_m() { return env_int("RESQ_GEMM_PAIR_MIN_M", kBM); }

TileChoice choose_tile(int64_t M, int64_t N, int64_t K, bool res, bool sparse = false) {
    const int sms = 148;
    const int G = (int)(K / kBK);
    TileChoice best{1, 256, 1, 1, 0};
    double best_cost = 1e300;
    for (int mt = 1; mt <= (res ? 1 : 2); ++mt) {
        if (mt == 2 && M <= kBM) continue;
        const int64_t mtiles = (M + kBM * mt - 1) / (kBM * mt);
        for (int nt = 1; nt <= 2; ++nt)
        for (int bn = 256; bn >= 64; bn /= 2) {
            if (mt * nt * bn > 512) continue;
            if (nt == 2 && bn < 256) continue;
            const int64_t ntiles = (N + nt * bn - 1) / (nt * bn);
            for (int splits = 1; splits <= 8; splits *= 2) {
                if (G / splits < 4 && splits > 1) break;
                const int64_t tiles = mtiles * ntiles * splits;
                const int64_t per_cta = (tiles + sms - 1) / sms;  // tiles walked by the busiest CTA
                const int kb = (G + splits - 1) / splits;
                // per-k-block time (arbitrary units): tensor time scales with mt*bn*(1+res), floored by the
                // expander time (scales with bn); small tiles pay a fixed hand-off cost per k-block
                const double mma = (double)mt * nt * bn * (res ? 2.0 : 1.0) / 256.0;
                const double expand = nt * bn / 256.0 * 0.8;
                // bytes pulled from L2 per k-block (activation tiles dominate), in units that make a
                // 128x256 tile with a residual operand cost about 1.3 tensor-time units
                const double l2 = (mt * (res ? 2.0 : 1.0) * 16.0 + nt * bn * 36.0 / 1024.0) / 31.0;
                const double per_kb = std::max(std::max(mma, expand), l2) + 0.15;
                double cost = per_cta * kb * per_kb + 8.0;  // pipeline fill + last epilogue
                if (mt * nt * bn > 256) cost += per_cta * 4.0;   // single accumulator: the epilogue is not overlapped
                if (splits > 1) cost += 8.0 + (double)M * N * splits / 2.0e5;
                if (cost < best_cost) {
                    best_cost = cost;
                    best = TileChoice{mt, bn, splits, nt, 0};
                }
            }
        }
    }
    // CTA pairs (256 x tn tiles, 74 pairs) for everything taller than one MMA.  Cycle model fitted to in-kernel
    // timelines: a k-block costs the tensor time of the tile, but not less than the ~1500 cycles the slot hand-off
    // (commit -> producers -> data landed -> MMA thread) takes, plus ~350 cycles of MMA-thread work between
    // k-blocks; a tile costs ~8000 cycles of fill and epilogue; a K split costs a second launch plus the
    // partial-tile traffic.
    if (M > pair_min_m() && env_int("RESQ_GEMM_PAIR", 1)) {
        const int64_t mtiles = (M + 2 * kBM - 1) / (2 * kBM);
        double best_pair = 1e300;
        for (int tn : {512, 480, 384, 320, 256, 128}) {
            // the sparse metadata needs a few tensor-memory columns: 480 instead of 512
            if (sparse ? tn == 512 : tn == 480) continue;
            const int64_t ntiles = (N + tn - 1) / tn;
            for (int splits = 1; splits <= 8; splits *= 2) {
                if (G / splits < 4 && splits > 1) break;
                const int64_t tiles = mtiles * ntiles * splits;
                const int64_t rounds = (tiles + sms / 2 - 1) / (sms / 2);
                const int kb = (G + splits - 1) / splits;
                const double mma = tn / 256.0 * (sparse ? 768.0 : res ? 1024.0 : 512.0);
                const double per_kb = std::max(mma, 1500.0) + 350.0;
                double cost = rounds * (kb * per_kb + 8000.0);
                if (splits > 1) cost += 15000.0 + (double)splits * M * N * 4.0 / 1200.0;  // partial tiles: ~1.6 KB/clk
                if (cost < best_pair) {
                    best_pair = cost;
                    best = TileChoice{1, std::min(tn, 256), splits, tn > 256 ? 2 : 1, tn};
                }
            }
        }
    }
    // debugging overrides (tile exploration); not part of the interface
    best.mt = env_int("RESQ_GEMM_MT", best.mt);
    best.bn = env_int("RESQ_GEMM_BN", best.bn);
    best.splits = env_int("RESQ_GEMM_SPLITS", best.splits);
    best.nt = env_int("RESQ_GEMM_NT", best.nt);
    best.pair_tn = env_int("RESQ_GEMM_PAIR_TN", best.pair_tn);
    if (M <= pair_min_m()) best.pair_tn = 0;
    if (res) best.mt = 1;
    return best;
}

template <int MT, bool RES, int TN, int FMT>
int launch_variant(const GemmArgs& g, const TileChoice& tc, cudaStream_t stream) {
    constexpr int kAStage = MT * kATileBytes * (RES ? 2 : 1);
    CUtensorMap ta, tr, tw;
    int rc = make_tmap_2d(&ta, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, g.a_bf16, (uint64_t)g.K, (uint64_t)g.M, (uint64_t)(g.lda ? g.lda : g.K) * 2,
                          kBK, kBM, CU_TENSOR_MAP_SWIZZLE_128B);
    if (rc) return rc;
    rc = make_tmap_2d(&tr, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, RES ? g.r_bf16 : g.a_bf16, (uint64_t)g.K, (uint64_t)g.M,
                      (uint64_t)(g.lda ? g.lda : g.K) * 2, kBK, kBM, CU_TENSOR_MAP_SWIZZLE_128B);
    if (rc) return rc;
    rc = make_tmap_2d(&tw, CU_TENSOR_MAP_DATA_TYPE_UINT8, g.w_codes, (uint64_t)g.K / 2, (uint64_t)g.N, (uint64_t)g.K / 2,
                      kBK / 2, (uint32_t)tc.bn, CU_TENSOR_MAP_SWIZZLE_NONE);
    if (rc) return rc;
    GemmParams p;
    p.w_side = g.w_side;
    p.M = g.M;
    p.N = g.N;
    p.K = g.K;
    p.bn = tc.bn;
    p.nt = tc.nt;
    const int G = (int)(g.K / kBK);
    p.splits = tc.splits;
    p.kblocks_per_split = (G + tc.splits - 1) / tc.splits;
    p.ntiles_m = (int)((g.M + kBM * MT - 1) / (kBM * MT));
    p.ntiles_n = (int)((g.N + tc.nt * tc.bn - 1) / (tc.nt * tc.bn));
    p.num_tiles = p.ntiles_m * p.ntiles_n * tc.splits;
    if (MT * tc.nt * tc.bn > kTmemCols) {
        set_last_error("internal: tile does not fit tensor memory");
        return RESQ_ERR_CUDA;
    }
    p.acc_bufs = MT * tc.nt * tc.bn * 2 <= kTmemCols ? 2 : 1;
    // ring depths from the shared-memory budget
    const int exp_stage = tc.nt * tc.bn * 128, raw_stage = tc.nt * tc.bn * 32;
    const int fixed = 1024 /*alignment slack*/ + 1024 /*barriers*/;
    p.se = env_int("RESQ_GEMM_SE", 3);
    p.sr = env_int("RESQ_GEMM_SR", 4);
    p.sa = (kSmemBudget - fixed - p.se * exp_stage - p.sr * raw_stage) / kAStage;
    if (p.sa < 3 && p.se > 2) {
        p.se = 2;
        p.sa = (kSmemBudget - fixed - p.se * exp_stage - p.sr * raw_stage) / kAStage;
    }
    if (p.sa < 2 && p.sr > 2) {
        p.sr = 2;
        p.sa = (kSmemBudget - fixed - p.se * exp_stage - p.sr * raw_stage) / kAStage;
    }
    p.sa = std::min(p.sa, kMaxRing);
    if (p.sa < 2 || p.se > kMaxRing || p.sr > kMaxRing) {
        set_last_error("internal: shared-memory rings do not fit (bn=%d)", tc.bn);
        return RESQ_ERR_CUDA;
    }
    const int smem_bytes = fixed + p.sa * kAStage + p.se * exp_stage + p.sr * raw_stage;
    p.Y = g.Y;
    p.out_f32 = g.out_dtype == RESQ_OUT_F32;
    p.ldy = g.ldy;
    p.partials = g.splitk_partials;
    p.status = g.status;
#ifdef RESQ_TIMELINE
    p.debug = env_int("RESQ_GEMM_DEBUG", 0);
#endif
    auto kern = gemm_hif4_kernel<MT, RES, TN, FMT>;
    rc = ensure_dynamic_smem(reinterpret_cast<const void*>(kern), kSmemBudget, "cudaFuncSetAttribute(gemm)");
    if (rc) return rc;
    const int num_sms = device_sm_count();
    const unsigned grid = (unsigned)std::min(p.num_tiles, num_sms);
    {
        LaunchScope scope(kKindGemm, stream);
        rc = cuda_fail(launch_kernel(kern, dim3(grid), dim3(kGemmThreads), (size_t)smem_bytes, stream, ta, tr, tw, p),
                       "gemm_hif4_kernel launch");
    }
    if (rc) return rc;
    return launch_splitk_reduce(g, tc.splits, stream);
}

}  // namespace

// K-streamed schedule of the pair kernel: used when there are too few 256 x 256 output tiles to give every CTA
// pair whole tiles (decode-sized M): the (tile, k-block) units are dealt out evenly instead.
bool gemm_use_streamk(int64_t M, int64_t N, int64_t K) {
    if (M <= pair_min_m() || !env_int("RESQ_GEMM_PAIR", 1)) return false;
    const int force = env_int("RESQ_GEMM_STREAMK", -1);
    if (force >= 0) return force != 0;
    if (env_int("RESQ_GEMM_PAIR_TN", 0) || env_int("RESQ_GEMM_SPLITS", 0)) return false;  // explicit tile exploration
    const int64_t tiles = ((M + 2 * kBM - 1) / (2 * kBM)) * ((N + 255) / 256);
    if (tiles <= 74 / 2 && tiles * (K / kBK) >= 2) return true;  // at least two pairs per tile: otherwise whole tiles per pair
    // Opt-in (RESQ_GEMM_HYBRID=1): one whole 256-wide tile per pair and a last round of at most half the pairs whose
    // k-blocks are dealt out over all pairs in the same kernel.  Measured slower than one round of wider tiles
    // (M = 256, 2048 -> 22016: 67.6 us against 55.0 us per call): the fp32 partial tiles of the last round cost more
    // than the narrower MMA instructions of the 320-wide tile.
    return tiles > 74 && tiles <= 74 + 74 / 2 && K / kBK >= 16 && env_int("RESQ_GEMM_HYBRID", 0);
}

// The 2:4 residual on the structured-sparse MMA (compressed operand + index metadata, half the tensor work of the
// residual term) is used where it is the faster form.  Its widest tile is 480 columns (the metadata takes eight
// tensor-memory columns), so it runs ceil(N / 480) instead of ceil(N / 512) columns of tiles; a k-block of a 480-wide
// sparse tile takes about 0.78 of the time of a 512-wide dense one (measured on the 7B and 3B prefill shapes under the
// power cap: 1.26 against 1.67 us).  It wins when that outweighs the extra tiles: every layer at M = 16384, the wide
// layers at M = 8192 (gate_up 856 against 989 us, qkv 165 against 184), not the N = 2048 layers there (five columns of
// tiles instead of four: 162 against 138 us), and not below a few thousand rows, where the calls are bound by fixed
// costs (M = 256: 150 against 146 us per step).  RESQ_SPARSE24 = 0 / 1 forces the choice (debugging override).
bool gemm_sparse24_supported(int64_t M, int64_t N, int64_t K) {
    if (M <= kBM || K % kBK != 0 || !env_int("RESQ_GEMM_PAIR", 1)) return false;
    const int forced = env_int("RESQ_SPARSE24", -1);
    if (forced >= 0) return forced != 0;
    if (M < 4096) return false;
    const int64_t mt = (M + 2 * kBM - 1) / (2 * kBM);
    const int64_t nt512 = (N + 511) / 512, nt480 = (N + 479) / 480;
    const int64_t tiles512 = mt * nt512, tail = tiles512 % 74;
    // (a small last round of the dense form is cut off into a decode-sized call: count it as a fraction of a round)
    const double rounds512 = (tiles512 > 74 && tail > 0 && tail <= nt512 && tail * 3 <= 74) ? (double)tiles512 / 74.0
                                                                                          : (double)((tiles512 + 73) / 74);
    const double rounds480 = (double)((mt * nt480 + 73) / 74);
    return rounds480 * 0.78 < rounds512;
}

// Block-wise selection: the CTA-pair kernel can take the keep flags and an unmasked residual image, which saves the
// read-modify-write pass over the image and the loads of the dropped blocks.  Used from 2048 token rows on: there the
// pass is what costs (7B prefill shapes at M = 16384: quantizer + selection + GEMM 11.27 against 11.86 ms per step; the
// wide layer's GEMM itself gains 4 %, the narrow ones lose up to 5 % to the four small boxes per tile), at M = 512 the
// saved pass (7 us per layer) and the slower K-streamed GEMM (4-15 us) cancel.  RESQ_BLOCK_LISTS = 0 / 1 forces the
// choice (debugging override).
bool gemm_block_lists_supported(int64_t M, int64_t N, int64_t K) {
    (void)N;
    if (M <= pair_min_m() || M % 32 != 0 || K % kBK != 0 || !env_int("RESQ_GEMM_PAIR", 1)) return false;
    const int forced = env_int("RESQ_BLOCK_LISTS", -1);
    if (forced >= 0) return forced != 0;
    return M >= 2048;
}

size_t gemm_hif4_scratch_bytes(int64_t M, int64_t N, int64_t K) {
    size_t classic = 0;
    const int splits = gemm_hif4_pick_splits(M, N, K);
    if (splits > 1) classic = (size_t)splits * (size_t)M * (size_t)N * 4;
    // the K-streamed schedule may be switched on or off by the debugging overrides: size for both
    const size_t sk = gemm_pair_streamk_scratch_bytes();
    return std::max(classic, sk);
}

int gemm_hif4_pick_splits(int64_t M, int64_t N, int64_t K) {
    // the workspace must cover the larger of the two possible choices (with / without residual)
    return std::max(std::max(choose_tile(M, N, K, false).splits, choose_tile(M, N, K, true).splits),
                    choose_tile(M, N, K, true, true).splits);
}

template <int MT, bool RES, int FMT>
int dispatch_tn(const GemmArgs& g, const TileChoice& tc, cudaStream_t stream) {
    const int tn = tc.bn * tc.nt;
    if (tn == 64) return launch_variant<MT, RES, 64, FMT>(g, tc, stream);
    if (tn == 128) return launch_variant<MT, RES, 128, FMT>(g, tc, stream);
    if (tn == 256) return launch_variant<MT, RES, 256, FMT>(g, tc, stream);
    if constexpr (MT == 1) {
        if (tn == 512) return launch_variant<MT, RES, 512, FMT>(g, tc, stream);
    }
    set_last_error("internal: unsupported tile width %d", tn);
    return RESQ_ERR_CUDA;
}

int launch_gemm_hif4(const GemmArgs& g, cudaStream_t stream) {
    const bool res = g.r_bf16 != nullptr || g.r_comp != nullptr;
    if (g.r_comp && !gemm_sparse24_supported(g.M, g.N, g.K)) {
        set_last_error("internal: compressed residual given for a shape the pair kernel does not run");
        return RESQ_ERR_CUDA;
    }
    const bool streamk = gemm_use_streamk(g.M, g.N, g.K) && g.splitk_partials && g.sk_flags &&
                         g.partial_bytes >= gemm_pair_streamk_scratch_bytes();
    if (g.w_bf16) {  // the CTA-pair kernel for every M (rows past M are zero-filled and never stored)
        if (streamk) return launch_gemm_pair_plainw(g, 256, 1, true, stream);
        const TileChoice c = g.M > kBM ? choose_tile(g.M, g.N, g.K, res) : TileChoice{1, 256, 1, 1, 256};
        const int splits = (c.splits > 1 && g.splitk_partials && c.splits <= g.splits) ? c.splits : 1;
        return launch_gemm_pair_plainw(g, c.pair_tn >= 384 ? 512 : 256, splits, false, stream);
    }
    if (g.blk_flags && (g.M <= pair_min_m() || !env_int("RESQ_GEMM_PAIR", 1))) {  // (any call the pair kernel runs takes them)
        set_last_error("internal: keep flags given for a shape the pair kernel does not run");
        return RESQ_ERR_CUDA;
    }
    if (streamk) return launch_gemm_pair_streamk(g, stream);
    TileChoice tc = choose_tile(g.M, g.N, g.K, res, g.r_comp != nullptr);
    if (tc.splits > 1 && (!g.splitk_partials || tc.splits > g.splits)) tc.splits = 1;
    if (env_int("RESQ_GEMM_DEBUG", 0) & 1)
        fprintf(stderr, "resq gemm M=%lld N=%lld K=%lld res=%d: pair_tn=%d mt=%d bn=%d nt=%d splits=%d\n", (long long)g.M,
                (long long)g.N, (long long)g.K, (int)res, tc.pair_tn, tc.mt, tc.bn, tc.nt, tc.splits);
    if (g.r_comp && tc.pair_tn == 512) tc.pair_tn = 480;  // (a forced width) no tensor-memory columns left for the metadata
    if (!g.r_comp && tc.pair_tn == 480) tc.pair_tn = 512;
    if (tc.pair_tn > 0) {
        // Whole tiles in rounds of 74: a last round with a handful of tiles keeps most pairs idle for a whole tile
        // time.  When those tiles are the end of the last row of tiles, they are a rectangle of the output: it is
        // cut off and computed by a second call (decode-sized: the K-streamed schedule spreads it over all pairs).
        const int64_t mtiles = (g.M + 2 * kBM - 1) / (2 * kBM), ntiles = (g.N + tc.pair_tn - 1) / tc.pair_tn;
        const int64_t tiles = mtiles * ntiles, tail = tiles % 74;
        if (tc.splits == 1 && !g.r_comp && tiles > 74 && tail > 0 && tail <= ntiles && tail * 3 <= 74 && g.tile_limit == 0 &&
            env_int("RESQ_GEMM_TAIL_SPLIT", 1)) {
            GemmArgs main_part = g, tail_part = g;
            main_part.tile_limit = (int)(tiles - tail);
            int rc = launch_gemm_pair(main_part, tc.pair_tn, 1, stream);
            if (rc) return rc;
            const int64_t m0 = (mtiles - 1) * 2 * kBM, n0 = (ntiles - tail) * tc.pair_tn;
            const int64_t lda = g.lda ? g.lda : g.K;
            tail_part.a_bf16 = g.a_bf16 + m0 * lda;
            if (g.r_bf16) tail_part.r_bf16 = g.r_bf16 + m0 * lda;
            if (g.blk_flags) tail_part.blk_flags = g.blk_flags + (m0 / 32) * (g.K / kBK);
            tail_part.lda = lda;
            if (g.w_bf16) {
                tail_part.w_bf16 = g.w_bf16 + n0 * g.ldw;
            } else {
                tail_part.w_codes = g.w_codes + n0 * (g.K / 2);
                tail_part.w_side = static_cast<const uint8_t*>(g.w_side) + n0 * (g.fmt == kHiF4 ? (g.K / kBK) * 4 : g.K / 32);
            }
            tail_part.M = g.M - m0;
            tail_part.N = g.N - n0;
            tail_part.Y = static_cast<uint8_t*>(g.Y) + (m0 * g.ldy + n0) * (g.out_dtype == RESQ_OUT_F32 ? 4 : 2);
            tail_part.tile_limit = -1;  // (no further cutting)
            return launch_gemm_hif4(tail_part, stream);
        }
        return launch_gemm_pair(g, tc.pair_tn, tc.splits, stream);
    }
    if (g.fmt == kMXFP4) {
        if (res) return dispatch_tn<1, true, kMXFP4>(g, tc, stream);
        if (tc.mt == 2) return dispatch_tn<2, false, kMXFP4>(g, tc, stream);
        return dispatch_tn<1, false, kMXFP4>(g, tc, stream);
    }
    if (res) return dispatch_tn<1, true, kHiF4>(g, tc, stream);
    if (tc.mt == 2) return dispatch_tn<2, false, kHiF4>(g, tc, stream);
    return dispatch_tn<1, false, kHiF4>(g, tc, stream);
}

}  // namespace resq
