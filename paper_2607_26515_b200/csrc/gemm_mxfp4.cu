// MXFP4 GEMM of Eq. (5) on the block-scaled FP4 tensor pipe:
//     Y[m, n] = sum_k a[m, k] w[n, k]  +  sum_k r[m, k] w[n, k]
// with a = Q(X), r = S(Q(dX)) and w = Q(W) all kept as packed E2M1 codes (two per byte, element 2j in the low
// nibble) with one E8M0 scale per 32 values along K.  tcgen05.mma kind::mxf4.block_scale multiplies the 4-bit
// operands straight from shared memory and applies the scales, which it reads from tensor memory: nothing is
// expanded.  Selected entries of the residual are kept by zeroing the dropped codes (the quantizer does that).
//
// One CTA per SM walks 128 x 256 output tiles, or (PAIR, for more than 128 token rows) a cluster of two CTAs walks
// 256 x 256 tiles with tcgen05.mma.cta_group::2: each CTA loads the codes of its own 128 token rows and of HALF of the
// tile's 256 weight rows (the tensor cores read the other half from the peer's shared memory), which cuts the bytes an
// SM pulls from L2 per unit of tensor work by a quarter to a third -- the bound of this kernel.  Every CTA still stages
// the scales of all 256 weight rows (each SM scales its own partial products).  No TMA multicast.
// A stage is 256 values of K: 128 x 128 B of activation codes
// (and as much for the residual), 256 x 128 B of weight codes, and their scales re-arranged into the 512-byte
// atoms tcgen05.cp copies to tensor memory (32 rows x 16 B: byte r1 * 4 + g of row r0 is the scale of row
// r0 + 32 * r1 for the g-th group of 32 values).
// Warp roles (8 warps): 0 TMA producer, 1 MMA issue + TMEM allocation, 2..3 scale gather, 4..7 epilogue.
// Every wait is bounded; a timeout ends the kernel cleanly (status word, abort flag).
#include "common.cuh"
#include "ptx.cuh"

#include <algorithm>
#include <cstdlib>
#include <cstring>
#include <mutex>

namespace resq {

namespace {

constexpr int kBM = 128;            // rows per tile (UMMA M)
constexpr int kBN = 256;            // columns per tile (UMMA N)
constexpr int kBKe = 256;           // K values per stage
constexpr int kRowBytes = kBKe / 2; // 128 B of codes per row per stage: one 128-byte-swizzled row
constexpr int kThreadsNative = 256;
constexpr int kATile = kBM * kRowBytes;       // 16 KiB
constexpr int kBTile = kBN * kRowBytes;       // 32 KiB
constexpr int kSfAtom = 512;                  // scales of 128 rows x 128 values of K
constexpr int kSfA = 2 * kSfAtom;             // two atoms along K per stage
constexpr int kSfB = 4 * kSfAtom;             // two along K x two along N
constexpr int kAccCols = kBN;                 // fp32 accumulator columns
constexpr int kSfSetCols = 32;                // tensor-memory columns of one stage's scales: A 8, residual 8, W 16
constexpr int kTmemColsNative = 512;
constexpr int kSmemBudgetNative = 232448;

struct NativeParams {
    const uint8_t* a_scale;   // [M, K/32]
    const uint8_t* r_scale;   // [M, K/32] or null
    const uint8_t* w_scale;   // [N, K/32]
    int64_t M, N, K;
    int ntiles_n, num_tiles;
    // K split: work item = (tile, split), split sp covers the stages [sp * kb_per_split, ...); with more than one split
    // the items write fp32 partial tiles into slabs [split][M][N] that the reduce kernel sums in a fixed order
    int splits, kb_per_split;
    float* partials;
    void* Y;
    int out_f32;
    int64_t ldy;
    DeviceStatus* status;
};

__device__ __forceinline__ void report_timeout_native(DeviceStatus* st, int where) {
    if (atomicCAS(&st->code, 0, (int)RESQ_ERR_TIMEOUT) == 0) {
        st->where = where;
        st->block = (int)blockIdx.x;
    }
}

// Instruction descriptor of kind::mxf4 (E2M1 x E2M1, E8M0 scales, K-major operands, M x N tile); the scale-factor
// ids select which byte of a 32-bit tensor-memory column holds the first scale of this K step.
__host__ __device__ constexpr uint32_t idesc_mxf4(int m, int n, uint32_t a_sf_id, uint32_t b_sf_id) {
    return (b_sf_id << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | (1u << 23) | ((uint32_t)(m >> 4) << 24) |
           (a_sf_id << 29);
}
// Shared-memory descriptor of a 32 x 16 B scale atom (no swizzle: 8-row groups of 128 contiguous bytes).
__device__ __forceinline__ uint64_t smem_desc_sf(uint32_t addr) {
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)(128 >> 4) << 16;  // leading byte offset (one 16-byte column only)
    d |= (uint64_t)(128 >> 4) << 32;  // stride between 8-row groups
    d |= (uint64_t)1 << 46;
    return d;
}
template <bool PAIR>
__device__ __forceinline__ void tmem_cp_sf(uint32_t taddr, uint64_t desc) {
    if constexpr (PAIR) asm volatile("tcgen05.cp.cta_group::2.32x128b.warpx4 [%0], %1;" ::"r"(taddr), "l"(desc) : "memory");
    else asm volatile("tcgen05.cp.cta_group::1.32x128b.warpx4 [%0], %1;" ::"r"(taddr), "l"(desc) : "memory");
}
template <bool PAIR>
__device__ __forceinline__ void umma_mxf4(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t sfa,
                                          uint32_t sfb, uint32_t accumulate) {
    if constexpr (PAIR)
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "setp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::2.kind::mxf4.block_scale.block32 [%0], %1, %2, %3, [%5], [%6], p;\n\t}"
            :
            : "r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(sfa), "r"(sfb)
            : "memory");
    else
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "setp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.block32 [%0], %1, %2, %3, [%5], [%6], p;\n\t}"
            :
            : "r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(sfa), "r"(sfb)
            : "memory");
}

constexpr int kMaxStagesNative = 6;

template <bool RES, bool PAIR>
struct StageLayout {
    static constexpr int kBBytes = PAIR ? kBTile / 2 : kBTile;          // weight codes this CTA loads per stage
    static constexpr int kStagesN = PAIR ? (RES ? 4 : 6) : (RES ? 3 : 4);
    static constexpr int kA = 0;
    static constexpr int kAr = kATile;                                  // only with RES
    static constexpr int kB = kATile * (RES ? 2 : 1);
    static constexpr int kSfAOff = kB + kBBytes;
    static constexpr int kSfArOff = kSfAOff + kSfA;                      // only with RES
    static constexpr int kSfBOff = kSfAOff + kSfA * (RES ? 2 : 1);
    static constexpr int kBytes = kSfBOff + kSfB;
    static constexpr uint32_t kTxBytes = (uint32_t)(kATile * (RES ? 2 : 1) + kBBytes);
};

template <bool RES, bool PAIR>
__global__ void __launch_bounds__(kThreadsNative, 1)
gemm_mxfp4_native_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_r,
                         const __grid_constant__ CUtensorMap tmap_w, const NativeParams p) {
    using L = StageLayout<RES, PAIR>;
    constexpr int S = L::kStagesN;
    constexpr int kTileM = PAIR ? 2 * kBM : kBM;  // token rows of a tile (of the pair's tile)
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (size_t)S * L::kBytes);
    // PAIR: the leader's "full" barriers collect both CTAs' bytes and gather warps; "empty" and "acc_full" are released in
    // both CTAs by one multicast commit; the leader's "acc_empty" collects both CTAs' epilogue warps.
    uint64_t* full = bars;                                // [S] codes landed (TMA bytes) and scale atoms written
    uint64_t* empty = bars + kMaxStagesNative;            // [S] the MMAs that read the stage completed
    uint64_t* acc_full = bars + 2 * kMaxStagesNative;     // accumulator complete
    uint64_t* acc_empty = acc_full + 1;                   // accumulator drained by the epilogue warps
    // PAIR, second CTA: its gather warps arrive here, and its otherwise idle warp 1 forwards each completed phase to the
    // leader's "full" barrier (a remote arrive with cluster-scope release stalls its thread for hundreds of cycles:
    // kept off the gather warps, which handle every stage)
    uint64_t* sf_ready = acc_empty + 1;                   // [S]
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(sf_ready + kMaxStagesNative);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nkb = (int)(p.K / kBKe);
    const int nitems = p.num_tiles * p.splits;
    auto item_of = [&](int item, int& tile, int& sp, int& kb0, int& kb1) {
        tile = item / p.splits;
        sp = item - tile * p.splits;
        kb0 = sp * p.kb_per_split;
        kb1 = min(nkb, kb0 + p.kb_per_split);
    };
    const uint32_t rank = PAIR ? ptx::cluster_ctarank() : 0u;  // 0 = leader
    const int worker = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x, nworkers = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            // leader: an arrive.expect_tx per CTA, its own two gather warps, and (PAIR) the peer's forwarding thread
            ptx::mbar_init(&full[s], PAIR ? 5 : 3);
            ptx::mbar_init(&empty[s], 1);
            ptx::mbar_init(&sf_ready[s], 2);
        }
        ptx::mbar_init(acc_full, 1);
        ptx::mbar_init(acc_empty, PAIR ? 8 : 4);
        *abort_flag = 0;
        ptx::mbar_fence_init();
    }
    if (warp == 1) {
        if constexpr (PAIR) ptx::tmem_alloc_pair(tmem_slot, kTmemColsNative);
        else ptx::tmem_alloc(tmem_slot, kTmemColsNative);
    }
    ptx::tc_fence_before();
    __syncthreads();
    if constexpr (PAIR) ptx::cluster_sync();  // the peer's barriers exist before anything arrives on them
    ptx::tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    pdl_trigger();
    pdl_wait();  // codes and scales of the activations come from the quantizer kernel just before
    // arrive on full[s] of the leader
    auto arrive_full = [&](uint64_t* bar) {
        if constexpr (PAIR) ptx::mbar_arrive_cluster(ptx::map_to_cta(bar, 0));
        else ptx::mbar_arrive(bar);
    };

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            ptx::tma_prefetch_desc(&tmap_a);
            if (RES) ptx::tma_prefetch_desc(&tmap_r);
            ptx::tma_prefetch_desc(&tmap_w);
            uint32_t s = 0, ph = 0;
            bool ok = true;
            for (int item = worker; item < nitems && ok; item += nworkers) {
                int tile, sp, kb0, kb1;
                item_of(item, tile, sp, kb0, kb1);
                const int m0 = (tile / p.ntiles_n) * kTileM + (int)rank * kBM, n0 = (tile % p.ntiles_n) * kBN;
                for (int kb = kb0; kb < kb1; ++kb) {
                    if (!ptx::mbar_wait_spin(&empty[s], ph ^ 1u, abort_flag)) {
                        report_timeout_native(p.status, 1);
                        ok = false;
                        break;
                    }
                    uint8_t* st = smem + (size_t)s * L::kBytes;
                    if constexpr (PAIR) {
                        const uint32_t fb = ptx::map_to_cta(&full[s], 0);
                        ptx::mbar_arrive_expect_tx_cluster_relaxed(fb, L::kTxBytes);  // publishes nothing itself
                        ptx::tma_load_2d_pair(st + L::kA, &tmap_a, fb, kb * kRowBytes, m0);
                        if (RES) ptx::tma_load_2d_pair(st + L::kAr, &tmap_r, fb, kb * kRowBytes, m0);
                        ptx::tma_load_2d_pair(st + L::kB, &tmap_w, fb, kb * kRowBytes, n0 + (int)rank * (kBN / 2));
                    } else {
                        ptx::mbar_arrive_expect_tx(&full[s], L::kTxBytes);
                        ptx::tma_load_2d(st + L::kA, &tmap_a, &full[s], kb * kRowBytes, m0);
                        if (RES) ptx::tma_load_2d(st + L::kAr, &tmap_r, &full[s], kb * kRowBytes, m0);
                        ptx::tma_load_2d(st + L::kB, &tmap_w, &full[s], kb * kRowBytes, n0);
                    }
                    if (++s == (uint32_t)S) { s = 0; ph ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (PAIR && lane == 0 && rank == 1) {
            // forward the peer's "scale atoms written" to the leader, stage by stage
            uint32_t s = 0, ph = 0;
            bool ok = true;
            for (int item = worker; item < nitems && ok; item += nworkers) {
                int tile, sp, kb0, kb1;
                item_of(item, tile, sp, kb0, kb1);
                for (int kb = kb0; kb < kb1; ++kb) {
                    if (!ptx::mbar_wait_spin(&sf_ready[s], ph, abort_flag)) {
                        report_timeout_native(p.status, 7);
                        ok = false;
                        break;
                    }
                    ptx::mbar_arrive_cluster(ptx::map_to_cta(&full[s], 0));
                    if (++s == (uint32_t)S) { s = 0; ph ^= 1u; }
                }
            }
        }
        if (lane == 0 && rank == 0) {
            const uint64_t desc0 = ptx::smem_desc_sw128_kmajor(0);
            const uint32_t smem_base16 = (ptx::smem_u32(smem) & 0x3FFFFu) >> 4;
            const uint64_t sf_desc0 = smem_desc_sf(0);  // everything but the start address
            uint32_t s = 0, ph = 0, it = 0;
            int local_tile = 0;
            bool ok = true;
            for (int item = worker; item < nitems && ok; item += nworkers, ++local_tile) {
                int tile, sp, kb0, kb1;
                item_of(item, tile, sp, kb0, kb1);
                if (!ptx::mbar_wait_spin(acc_empty, (uint32_t)(local_tile & 1) ^ 1u, abort_flag)) {
                    report_timeout_native(p.status, 6);
                    break;
                }
                ptx::tc_fence_after();
                for (int kb = kb0; kb < kb1; ++kb, ++it) {
                    if (!ptx::mbar_wait_spin(&full[s], ph, abort_flag)) {
                        report_timeout_native(p.status, 2);
                        ok = false;
                        break;
                    }
                    ptx::tc_fence_after();
                    // (this thread's instruction stream sits between the MMAs of consecutive stages: descriptors by additions)
                    const uint64_t sfd = sf_desc0 + (uint64_t)(smem_base16 + s * (uint32_t)(L::kBytes >> 4));
                    // scales of this stage -> tensor memory (two column sets alternate between stages)
                    const uint32_t sf = tmem_base + (uint32_t)(kAccCols + (it & 1u) * kSfSetCols);
#pragma unroll
                    for (int ka = 0; ka < 2; ++ka) {
                        tmem_cp_sf<PAIR>(sf + ka * 4, sfd + (uint64_t)((L::kSfAOff + ka * kSfAtom) >> 4));
                        if (RES) tmem_cp_sf<PAIR>(sf + 8 + ka * 4, sfd + (uint64_t)((L::kSfArOff + ka * kSfAtom) >> 4));
#pragma unroll
                        for (int nb = 0; nb < 2; ++nb)
                            tmem_cp_sf<PAIR>(sf + 16 + ka * 8 + nb * 4, sfd + (uint64_t)((L::kSfBOff + (ka * 2 + nb) * kSfAtom) >> 4));
                    }
                    const uint32_t st16 = smem_base16 + s * (uint32_t)(L::kBytes >> 4);
                    const uint64_t adesc = desc0 + (uint64_t)(st16 + (L::kA >> 4));
                    const uint64_t rdesc = desc0 + (uint64_t)(st16 + (L::kAr >> 4));
                    const uint64_t bdesc = desc0 + (uint64_t)(st16 + (L::kB >> 4));
#pragma unroll
                    for (int k4 = 0; k4 < 4; ++k4) {  // 64 values (32 B) of K per MMA: two scale groups
                        const int ka = k4 >> 1;
                        const uint32_t sfid = (uint32_t)(k4 & 1) * 2u;
                        const uint32_t idesc = idesc_mxf4(kTileM, kBN, sfid, sfid);
                        const uint32_t sfa = sf + ka * 4 + (sfid << 30), sfb = sf + 16 + ka * 8 + (sfid << 30);
                        umma_mxf4<PAIR>(tmem_base, adesc + (uint64_t)(2 * k4), bdesc + (uint64_t)(2 * k4), idesc, sfa, sfb,
                                        (kb > kb0 || k4 > 0) ? 1u : 0u);
                        if (RES)
                            umma_mxf4<PAIR>(tmem_base, rdesc + (uint64_t)(2 * k4), bdesc + (uint64_t)(2 * k4), idesc,
                                            sf + 8 + ka * 4 + (sfid << 30), sfb, 1u);
                    }
                    if constexpr (PAIR) ptx::umma_commit_pair(&empty[s], 3);  // frees the stage in both CTAs
                    else ptx::umma_commit(&empty[s]);
                    if (++s == (uint32_t)S) { s = 0; ph ^= 1u; }
                }
                if (ok) {
                    if constexpr (PAIR) ptx::umma_commit_pair(acc_full, 3);
                    else ptx::umma_commit(acc_full);
                }
            }
        }
    } else if (warp < 4) {
        // ------------------------------------------------------------------ scale gather (64 threads)
        // Each thread owns 2 activation rows (+ 2 residual rows) and 4 weight rows of the tile: 8 scale bytes per
        // row and stage.  The loads of the next stage are issued before this stage's slot is waited for, so
        // their latency (uncoalesced 8-byte reads) stays off the slot's critical path.
        const int t = (warp - 2) * 32 + lane;
        const int64_t spr = p.K / 32;  // scale bytes per row
        uint32_t s = 0, ph = 0;
        bool ok = true;
        uint2 va[2], vr[2], vw[4];
        auto load_scales = [&](int tile, int kb) {
            const int64_t m0 = (int64_t)(tile / p.ntiles_n) * kTileM + rank * kBM, n0 = (int64_t)(tile % p.ntiles_n) * kBN;
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                const int64_t m = m0 + t + 64 * j;
                va[j] = vr[j] = make_uint2(0u, 0u);
                if (m < p.M) {
                    va[j] = *reinterpret_cast<const uint2*>(p.a_scale + m * spr + kb * 8);
                    if (RES) vr[j] = *reinterpret_cast<const uint2*>(p.r_scale + m * spr + kb * 8);
                }
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int64_t n = n0 + t + 64 * j;
                vw[j] = make_uint2(0u, 0u);
                if (n < p.N) vw[j] = *reinterpret_cast<const uint2*>(p.w_scale + n * spr + kb * 8);
            }
        };
        int item = worker, tile = 0, sp = 0, kb = 0, kb1 = 0;
        if (item < nitems) {
            item_of(item, tile, sp, kb, kb1);
            load_scales(tile, kb);
        }
        while (item < nitems && ok) {
            if (!ptx::mbar_wait(&empty[s], ph ^ 1u, abort_flag)) {
                report_timeout_native(p.status, 3);
                ok = false;
                break;
            }
            uint8_t* st = smem + (size_t)s * L::kBytes;
            // row rr of a 128-row atom: 4 bytes at (rr % 32) * 16 + (rr / 32) * 4; the two K atoms are 512 B apart
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                const int rr = t + 64 * j;
                const int off = (rr & 31) * 16 + (rr >> 5) * 4;
                *reinterpret_cast<uint32_t*>(st + L::kSfAOff + off) = va[j].x;
                *reinterpret_cast<uint32_t*>(st + L::kSfAOff + kSfAtom + off) = va[j].y;
                if (RES) {
                    *reinterpret_cast<uint32_t*>(st + L::kSfArOff + off) = vr[j].x;
                    *reinterpret_cast<uint32_t*>(st + L::kSfArOff + kSfAtom + off) = vr[j].y;
                }
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int rn = t + 64 * j;  // row of the 256-row weight tile; atoms of W: (ka, nb) at (ka * 2 + nb) * 512
                const int nb = rn >> 7, rr = rn & 127;
                const int off = (rr & 31) * 16 + (rr >> 5) * 4;
                *reinterpret_cast<uint32_t*>(st + L::kSfBOff + (0 * 2 + nb) * kSfAtom + off) = vw[j].x;
                *reinterpret_cast<uint32_t*>(st + L::kSfBOff + (1 * 2 + nb) * kSfAtom + off) = vw[j].y;
            }
            ptx::fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) {
                if (PAIR && rank == 1) ptx::mbar_arrive(&sf_ready[s]);
                else ptx::mbar_arrive(&full[s]);
            }
            if (++s == (uint32_t)S) { s = 0; ph ^= 1u; }
            if (++kb == kb1) {
                item += nworkers;
                if (item < nitems) item_of(item, tile, sp, kb, kb1);
            }
            if (item < nitems) load_scales(tile, kb);  // in flight while the next slot is awaited
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 4..7)
        const int quad = warp & 3;
        int local_tile = 0;
        for (int item = worker; item < nitems; item += nworkers, ++local_tile) {
            int tile, sp, kb0, kb1;
            item_of(item, tile, sp, kb0, kb1);
            const int64_t m0 = (int64_t)(tile / p.ntiles_n) * kTileM + rank * kBM, n0 = (int64_t)(tile % p.ntiles_n) * kBN;
            // (a K split writes fp32 partial tiles into the slab of its split)
            const bool part = p.splits > 1;
            void* const out = part ? static_cast<void*>(p.partials + (size_t)sp * (size_t)p.M * (size_t)p.N) : p.Y;
            const int64_t ldo = part ? p.N : p.ldy;
            const bool f32 = part || p.out_f32;
            if (!ptx::mbar_wait(acc_full, (uint32_t)(local_tile & 1), abort_flag)) {
                report_timeout_native(p.status, 4);
                break;
            }
            ptx::tc_fence_after();
            const int64_t m = m0 + quad * 32 + lane;
#pragma unroll 1
            for (int cc = 0; cc < kBN / 32; ++cc) {
                uint32_t v[32];
                ptx::tmem_ld_32x32(tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(cc * 32), v);
                ptx::tmem_ld_wait();
                if (cc == kBN / 32 - 1) {
                    ptx::tc_fence_before();
                    __syncwarp();
                    if (lane == 0) arrive_full(acc_empty);
                }
                if (m >= p.M) continue;
                const int64_t nb = n0 + cc * 32;
                const int64_t left = p.N - nb;
                if (left <= 0) continue;
                if (f32) {
                    float* dst = reinterpret_cast<float*>(out) + m * ldo + nb;
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
                    __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(out) + m * ldo + nb;
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
    }
    ptx::tc_fence_before();
    __syncthreads();
    if constexpr (PAIR) ptx::cluster_sync();  // no CTA leaves while the peer may still signal its barriers or read its shared memory
    if (warp == 1) {
        ptx::tc_fence_after();
        if constexpr (PAIR) ptx::tmem_dealloc_pair(tmem_base, kTmemColsNative);
        else ptx::tmem_dealloc(tmem_base, kTmemColsNative);
    }
}

// K split of a decode-sized call with a long K range: enough (tile, split) items to give every SM one, at least two stages
// of 256 values per split, as many slabs as fit into the scratch (down projections at M = 256 / 512: 39.6 -> 29.0 us and
// 88.8 -> 66.2 us with the reduce launch).  RESQ_MXFP4_SPLITS is the debugging override.
int native_splits(int64_t M, int64_t N, int64_t K, size_t partial_bytes) {
    const int nkb = (int)(K / kBKe);
    const int64_t tiles = ((M + kBM - 1) / kBM) * ((N + kBN - 1) / kBN);
    int64_t want = std::min<int64_t>(148 / std::max<int64_t>(1, tiles), nkb / 2);
    want = std::min<int64_t>(want, (int64_t)(partial_bytes / ((size_t)M * (size_t)N * 4)));
    want = std::min<int64_t>(want, 16);
    if (nkb < 16) want = 1;  // short K ranges: the second launch costs what the split saves (qkv at M = 256: 18.9 -> 28.8 us)
    want = env_int("RESQ_MXFP4_SPLITS", (int)want);
    if (want < 2 || (N & 3) != 0 || (size_t)want * (size_t)M * (size_t)N * 4 > partial_bytes) return 1;
    const int per = (nkb + (int)want - 1) / (int)want;
    return (nkb + per - 1) / per;  // (no empty split)
}

template <bool RES, bool PAIR>
int launch_native_variant(const Mxfp4NativeArgs& g, cudaStream_t stream) {
    using L = StageLayout<RES, PAIR>;
    constexpr int kTileM = PAIR ? 2 * kBM : kBM;
    CUtensorMap ta, tr, tw;
    int rc = make_tmap_2d(&ta, CU_TENSOR_MAP_DATA_TYPE_UINT8, g.a_codes, (uint64_t)g.K / 2, (uint64_t)g.M, (uint64_t)g.K / 2,
                          kRowBytes, kBM, CU_TENSOR_MAP_SWIZZLE_128B);
    if (rc) return rc;
    rc = make_tmap_2d(&tr, CU_TENSOR_MAP_DATA_TYPE_UINT8, RES ? g.r_codes : g.a_codes, (uint64_t)g.K / 2, (uint64_t)g.M,
                      (uint64_t)g.K / 2, kRowBytes, kBM, CU_TENSOR_MAP_SWIZZLE_128B);
    if (rc) return rc;
    rc = make_tmap_2d(&tw, CU_TENSOR_MAP_DATA_TYPE_UINT8, g.w_codes, (uint64_t)g.K / 2, (uint64_t)g.N, (uint64_t)g.K / 2,
                      kRowBytes, PAIR ? kBN / 2 : kBN, CU_TENSOR_MAP_SWIZZLE_128B);
    if (rc) return rc;
    NativeParams p;
    p.a_scale = g.a_scale;
    p.r_scale = g.r_scale;
    p.w_scale = g.w_scale;
    p.M = g.M;
    p.N = g.N;
    p.K = g.K;
    p.ntiles_n = (int)((g.N + kBN - 1) / kBN);
    p.num_tiles = (int)((g.M + kTileM - 1) / kTileM) * p.ntiles_n;
    p.splits = (!PAIR && g.partials) ? native_splits(g.M, g.N, g.K, g.partial_bytes) : 1;
    p.kb_per_split = ((int)(g.K / kBKe) + p.splits - 1) / p.splits;
    p.partials = g.partials;
    p.Y = g.Y;
    p.out_f32 = g.out_dtype == RESQ_OUT_F32;
    p.ldy = g.ldy;
    p.status = g.status;
    const int smem_bytes = 1024 + L::kStagesN * L::kBytes + 256;
    static_assert(1024 + L::kStagesN * L::kBytes + 256 <= kSmemBudgetNative, "stages do not fit");
    auto kern = gemm_mxfp4_native_kernel<RES, PAIR>;
    rc = ensure_dynamic_smem(reinterpret_cast<const void*>(kern), smem_bytes, "cudaFuncSetAttribute(gemm mxfp4)");
    if (rc) return rc;
    const int num_sms = device_sm_count();
    if constexpr (!PAIR) {
        const unsigned grid = (unsigned)std::min(p.num_tiles * p.splits, num_sms);
        {
            LaunchScope scope(kKindGemm, stream);
            rc = cuda_fail(launch_kernel(kern, dim3(grid), dim3(kThreadsNative), (size_t)smem_bytes, stream, ta, tr, tw, p),
                           "gemm_mxfp4_native_kernel launch");
        }
        if (rc || p.splits == 1) return rc;
        GemmArgs red;  // the fixed-order sum of the slabs (the reduce kernel of the bf16 route)
        memset(&red, 0, sizeof(red));
        red.splitk_partials = g.partials;
        red.M = g.M;
        red.N = g.N;
        red.Y = g.Y;
        red.out_dtype = g.out_dtype;
        red.ldy = g.ldy;
        return launch_splitk_reduce(red, p.splits, stream);
    } else {
        LaunchScope scope(kKindGemm, stream);
        cudaLaunchConfig_t cfg;
        memset(&cfg, 0, sizeof(cfg));
        cfg.gridDim = dim3((unsigned)(2 * std::min(p.num_tiles, num_sms / 2)), 1, 1);
        cfg.blockDim = dim3(kThreadsNative, 1, 1);
        cfg.dynamicSmemBytes = (size_t)smem_bytes;
        cfg.stream = stream;
        cudaLaunchAttribute attr[2];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[1].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = pdl_enabled() ? 2 : 1;
        return cuda_fail(cudaLaunchKernelEx(&cfg, kern, ta, tr, tw, p), "gemm_mxfp4_native_kernel (pair) launch");
    }
}

}  // namespace

bool gemm_mxfp4_native_supported(int64_t M, int64_t N, int64_t K, bool res) {
    // RESQ_MXFP4_NATIVE: debugging override (0: never, 1: whenever the shape allows, unset: when it pays)
    const int mode = env_int("RESQ_MXFP4_NATIVE", -1);
    if (mode == 0 || K % kBKe != 0) return false;
    if (mode == 1) return true;
    // No K split here: a CTA walks the whole K range of its tiles, about 1.1 us per 256 values of K.  The bf16
    // route splits K for decode-sized calls; its time is about 15 us plus the executed flops at 1 PFLOP/s.
    // (Both fitted to the layer shapes of the 3B / 7B configurations at M = 256 ... 16384.)
    const int64_t tiles = ((M + kBM - 1) / kBM) * ((N + kBN - 1) / kBN);
    const int splits = native_splits(M, N, K, gemm_hif4_scratch_bytes(M, N, K));
    const int per = ((int)(K / kBKe) + splits - 1) / splits;
    // (a K split adds the reduce launch and the traffic of its slabs)
    const double t_native = 8.0 + (double)((tiles * splits + 147) / 148) * (double)per * 1.1 +
                            (splits > 1 ? 4.0 + (double)splits * (double)M * (double)N * 4.0 / 3.0e6 : 0.0);
    const double t_bf16 = 15.0 + 2.0 * (double)M * (double)N * (double)K * (res ? 2.0 : 1.0) / 1.0e9;
    return t_native < t_bf16;
}

int launch_gemm_mxfp4_native(const Mxfp4NativeArgs& g, cudaStream_t stream) {
    auto al8 = [](const void* p) { return (reinterpret_cast<uintptr_t>(p) & 7u) == 0; };
    if (!al8(g.a_scale) || !al8(g.w_scale) || (g.r_scale && !al8(g.r_scale))) {
        set_last_error("native MXFP4 GEMM: scale arrays must be 8-byte aligned");
        return RESQ_ERR_ALIGN;
    }
    // CTA pairs (256 x 256 tiles, a third less L2 -> SM traffic per unit of tensor work) are built and parity-tested but
    // measured slower than one CTA per tile (7B prefill shapes, whole step: NONE 3.34 against 2.98 ms, DENSE 4.30 against
    // 4.19 ms; decode shapes lose more, having half as many tiles to spread): opt-in by RESQ_MXFP4_PAIR=1 (debugging
    // override).  What the pair costs -- the scale copies and MMAs of both SMs issued by one thread, the cross-CTA
    // arrivals on the critical path of every 256-value stage -- outweighs the saved traffic.
    const bool pair = env_int("RESQ_MXFP4_PAIR", 0) != 0 && g.M > kBM;
    if (pair) return g.r_codes ? launch_native_variant<true, true>(g, stream) : launch_native_variant<false, true>(g, stream);
    return g.r_codes ? launch_native_variant<true, false>(g, stream) : launch_native_variant<false, false>(g, stream);
}

}  // namespace resq
