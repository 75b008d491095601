// Decode-sized calls of the layer (Eq. (5) at M <= 32 token rows), a group of projections in one launch.
//
// At these sizes the weights are the work: every packed 4-bit weight has to be expanded to bf16 once, and the tokens are a
// sliver.  So the operands change places against the CTA-pair kernel: a tile is 128 weight rows, which are the M dimension
// of the MMA (tcgen05.mma.cta_group::1.kind::f16, M = 128), and the token rows (rounded up to 16) are its N dimension; the
// rows of the residual operand follow those of the main image in shared memory, so one MMA over N = 2 x tokens accumulates
// both terms side by side and the epilogue adds them.  The accumulator is 128 lanes x (2) M columns and a partial tile is
// M x 128 floats.  What bounds it is the integer pipe (two cycles per warp instruction): about 30 instructions per 8 weights
// of expansion, and whatever else the loops execute next to them.
//
// Pipeline: a stage is a "quad" of four consecutive k-blocks -- one wait, one proxy fence and one arrive per quad and warp,
// one commit per quad.  (With one k-block per stage the loop runs at the latency of a warp's wait -> expand -> fence ->
// arrive chain, about 2000 cycles per k-block: every warp takes part in every stage.)  The packed codes of a quad arrive as
// one TMA box of 128 rows x 128 bytes (128-byte swizzle: the expanders' reads are conflict-free), a thread owns two
// 16-byte chunks of one weight row in each of the four k-blocks.
//
// Schedule: the (tile, k-block) units of all problems form one sequence that is cut into equal contiguous ranges, one
// per CTA.  A range that covers part of a tile's K range writes an fp32 partial tile into one of the CTA's two slots and
// counts itself in on the tile's arrival counter; whoever arrives last adds the tile's segments in k order (a fixed
// order: results do not depend on timing) and writes Y.  Nobody waits for another CTA.
//
// Roles per CTA (24 warps): warps 0-15 expanders, 16 raw-code TMA producer, 17 token-tile TMA producer, 18 MMA issuer,
// 20-23 epilogue (tensor-memory lanes 32 * (warp % 4) ...).  Every wait is bounded (ptx.cuh); on expiry the kernel records
// RESQ_ERR_TIMEOUT and leaves through its normal exit.  No TMA multicast.
#include "common.cuh"
#include "ptx.cuh"
#include "expand.cuh"

#include <algorithm>
#include <cstring>

namespace resq {
namespace {

constexpr int kBK = 64;            // one 64-wide k-block (a HiF4 block, two MXFP4 blocks) per pipeline stage
constexpr int kDecRows = 128;      // weight rows of a tile: the MMA's M
constexpr int kDecExpWarps = 16;
constexpr int kDecRawWarp = 16, kDecTokWarp = 17, kDecMmaWarp = 18, kDecFirstEpiWarp = 20;
constexpr int kDecThreads = 32 * 24;
constexpr int kDecMaxRing = 8;
constexpr int kDecMaxTok = 32;     // token rows (the MMA's N)
constexpr int kDecQuad = 4;        // k-blocks per pipeline stage
constexpr int kDecStages = 2;      // stages of the token ring and of the expanded-weight ring
constexpr int kDecSmem = 232448;
constexpr int kDecTmemCols = 128;  // two accumulators of 64 columns (main and residual partial sums side by side)
constexpr int kDecExpStage = kDecRows * 128, kDecExpQuad = kDecQuad * kDecExpStage, kDecRawQuad = kDecRows * 128;
constexpr int kDecMaxTiles = (int)(kWsFlags / sizeof(unsigned int));

struct DecProblem {
    const void* w_side;
    void* Y;
    int64_t ldy;
    int M, N, G;        // token rows, output columns, k-blocks (K / 64)
    int tile_base;      // the problem's first tile in the launch's tile list
    int64_t unit_base;  // (tile, k-block) units of the problems before it
};

struct DecMaps {
    CUtensorMap a[kMaxQuantGroup], r[kMaxQuantGroup], w[kMaxQuantGroup];
};

struct DecParams {
    DecProblem pr[kMaxQuantGroup];
    int nprob;
    int ntok;             // MMA N: the largest M of the group rounded up to 16
    int64_t units;        // (tile, k-block) units of the launch
    int sr;               // depth of the raw-code ring (quads)
    int a_stage;          // bytes of the token tiles of one k-block (main image, then the residual operand)
    int out_f32;
    float* slots;         // [2 * CTAs][ntok][128] fp32 partial tiles
    unsigned int* flags;  // [tiles] arrival counters (zeroed before the launch)
    DeviceStatus* status;
};

struct DecSeg {
    int prob, tile, n0, kb0, nkb, slot;
    bool partial;
};

// First unit of CTA c (c may be one past the last CTA) and the CTA that owns unit u.
__device__ __forceinline__ int64_t dec_begin(const DecParams& p, int c, int nctas) { return (int64_t)c * p.units / nctas; }
__device__ __forceinline__ int dec_cta_of(const DecParams& p, int64_t u, int nctas) { return (int)(((u + 1) * nctas - 1) / p.units); }

// Walks the segments of one CTA in the order every role uses.
struct DecIter {
    const DecParams& p;
    int cta;
    int64_t u0, u, u1;
    __device__ DecIter(const DecParams& p_, int cta_, int nctas) : p(p_), cta(cta_) {
        u0 = u = dec_begin(p, cta, nctas);
        u1 = dec_begin(p, cta + 1, nctas);
    }
    __device__ bool next(DecSeg& s) {
        if (u >= u1) return false;
        int q = 0;
#pragma unroll 1
        while (q + 1 < p.nprob && u >= p.pr[q + 1].unit_base) ++q;
        const int64_t rel = u - p.pr[q].unit_base;
        const int G = p.pr[q].G;
        const int tl = (int)(rel / G);
        s.prob = q;
        s.tile = p.pr[q].tile_base + tl;
        s.n0 = tl * kDecRows;
        s.kb0 = (int)(rel - (int64_t)tl * G);
        s.nkb = (int)min((int64_t)(G - s.kb0), u1 - u);
        s.partial = s.nkb < G;
        s.slot = 2 * cta + (u == u0 ? 0 : 1);
        u += s.nkb;
        return true;
    }
};

__device__ __forceinline__ void dec_timeout(DeviceStatus* st, int where) {
    if (atomicCAS(&st->code, 0, (int)RESQ_ERR_TIMEOUT) == 0) {
        st->where = 32 + where;
        st->block = (int)blockIdx.x;
    }
}

template <int FMT, bool RES>
__global__ void __launch_bounds__(kDecThreads, 1)
gemm_decode_kernel(const __grid_constant__ DecMaps maps, const __grid_constant__ DecParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    // A pipeline stage is a "quad" of up to four consecutive k-blocks of a segment: one wait, one proxy fence and one
    // arrive per quad and warp, one commit per quad (with a k-block per stage the loop runs at the latency of a warp's
    // wait -> expand -> fence -> arrive chain, about 2000 cycles per k-block).
    const int SR = p.sr;  // raw-code quads; the token and expanded-weight rings have two stages each
    const int a_quad = kDecQuad * p.a_stage;
    uint8_t* ring_a = smem;
    uint8_t* ring_e = ring_a + (size_t)kDecStages * a_quad;
    uint8_t* ring_r = ring_e + (size_t)kDecStages * kDecExpQuad;
    uint64_t* bars = reinterpret_cast<uint64_t*>(ring_r + (size_t)SR * kDecRawQuad);
    uint64_t* a_full = bars;                      // [2] token quad landed
    uint64_t* q_empty = bars + kDecMaxRing;       // [2] the MMAs that read the token quad and the expanded quad completed
    uint64_t* r_full = bars + 2 * kDecMaxRing;    // raw codes landed
    uint64_t* r_empty = bars + 3 * kDecMaxRing;   // the expanders consumed them
    uint64_t* e_full = bars + 4 * kDecMaxRing;    // [2] expanded quad written
    uint64_t* acc_full = bars + 6 * kDecMaxRing;  // [2]
    uint64_t* acc_empty = acc_full + 2;           // [2]
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    volatile int* s_last = reinterpret_cast<volatile int*>(tmem_slot + 2);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int cta = (int)blockIdx.x, nctas = (int)gridDim.x;
    const int ntok = p.ntok;
    const int tok_bytes = ntok * 128;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kDecMaxRing; ++s) {
            ptx::mbar_init(&a_full[s], 1);
            ptx::mbar_init(&q_empty[s], 1);
            ptx::mbar_init(&r_full[s], 1);
            ptx::mbar_init(&r_empty[s], kDecExpWarps);
            ptx::mbar_init(&e_full[s], kDecExpWarps);
        }
        for (int b = 0; b < 2; ++b) {
            ptx::mbar_init(&acc_full[b], 1);
            ptx::mbar_init(&acc_empty[b], 4);
        }
        *abort_flag = 0;
        ptx::mbar_fence_init();
    }
    if (warp == kDecMmaWarp) ptx::tmem_alloc(tmem_slot, kDecTmemCols);
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // Programmatic dependent launch: the weight side reads only the packed weights, which no kernel since the start of the
    // quantizer writes, and starts at once; the token producer and the epilogue wait for the quantizer's outputs.
    pdl_trigger();
    if (warp >= kDecTokWarp) pdl_wait();

    if (warp < kDecExpWarps) {
        // ------------------------------------------------------------------ expanders
        // thread -> weight row tid / 4 of the tile and the 16-byte chunks 2 (tid % 4), 2 (tid % 4) + 1 of its 128-byte row
        const int row = (int)threadIdx.x >> 2, ch0 = ((int)threadIdx.x & 3) * 2;
        const uint32_t st0 = (uint32_t)(row * 128 + ((ch0 ^ (row & 7)) << 4)), st1 = (uint32_t)(row * 128 + (((ch0 + 1) ^ (row & 7)) << 4));
        // the raw quad is a 128-byte-swizzled tile [128 rows][4 k-blocks x 32 bytes]: this thread's 8 bytes of k-block s
        // are in the logical 16-byte chunk 2 s + ch0 / 4
        const uint32_t rd_row = (uint32_t)(row * 128 + (ch0 & 3) * 4);
        // The integer pipe is what this loop runs on (two cycles per warp instruction): everything but the expansion itself
        // is kept out of it -- ring indices and phases advance by additions, the metadata pointer by a constant.
        uint32_t st = 0, st_ph = 0, sr = 0, sr_ph = 0;  // stage of the expanded / token rings and its phase; same for the raw ring
        bool ok = true;
        DecIter di(p, cta, nctas);
        DecSeg sg;
        while (ok && di.next(sg)) {
            const DecProblem& pb = p.pr[sg.prob];
            const int64_t n = (int64_t)sg.n0 + row;
            const bool row_ok = n < pb.N;
            const int G = pb.G;
            // metadata words of this thread's row, from the segment's first k-block on (rows past N read row 0 and are never stored)
            const uint8_t* side = static_cast<const uint8_t*>(pb.w_side) + ((row_ok ? n : 0) * (int64_t)G + sg.kb0) * (FMT == kHiF4 ? 4 : 2);
            const int kb_left = G - sg.kb0;  // k-blocks up to the end of the row
            auto load_quad = [&](int first, uint32_t (&m)[kDecQuad]) {
#pragma unroll
                for (int s = 0; s < kDecQuad; ++s) {
                    if (first + s < kb_left) {
                        if (FMT == kHiF4) m[s] = ptx::ld_nc_u32(reinterpret_cast<const uint32_t*>(side) + first + s);
                        else m[s] = ptx::ld_nc_u16(reinterpret_cast<const uint16_t*>(side) + first + s);
                    } else {
                        m[s] = 0u;
                    }
                }
            };
            const int nq = (sg.nkb + kDecQuad - 1) / kDecQuad;
            // the metadata words of a quad are fetched while the previous quad is expanded
            uint32_t mn[kDecQuad];
            load_quad(0, mn);
            for (int j = 0; j < nq; ++j) {
                uint32_t mw[kDecQuad];
#pragma unroll
                for (int s = 0; s < kDecQuad; ++s) mw[s] = mn[s];
                if (j + 1 < nq) load_quad((j + 1) * kDecQuad, mn);
                const int valid = min(kDecQuad, sg.nkb - j * kDecQuad);
                // one lane polls the two barriers for its warp
                int got = 1;
                if (lane == 0)
                    got = (ptx::mbar_wait_spin(&q_empty[st], st_ph ^ 1u, abort_flag) && ptx::mbar_wait_spin(&r_full[sr], sr_ph, abort_flag)) ? 1 : 0;
                ok = __shfl_sync(0xFFFFFFFFu, got, 0) != 0;
                if (!ok) {
                    dec_timeout(p.status, 3);
                    break;
                }
                const uint8_t* rq = ring_r + (size_t)sr * kDecRawQuad + rd_row;
                uint8_t* eq = ring_e + (size_t)st * kDecExpQuad;
                uint2 cw[kDecQuad];
#pragma unroll
                for (int s = 0; s < kDecQuad; ++s)
                    cw[s] = *reinterpret_cast<const uint2*>(rq + ((((uint32_t)(2 * s + (ch0 >> 2))) ^ (uint32_t)(row & 7)) << 4));
#pragma unroll
                for (int s = 0; s < kDecQuad; ++s) {
                    if (s < valid) {
                        uint4 v0, v1;
                        if (FMT == kHiF4) {
                            v0 = expand_hif4_chunk(cw[s].x, mw[s], ch0);
                            v1 = expand_hif4_chunk(cw[s].y, mw[s], ch0 + 1);
                        } else {
                            v0 = expand_mxfp4_chunk(cw[s].x, (mw[s] >> (8 * (ch0 >> 2))) & 255u);
                            v1 = expand_mxfp4_chunk(cw[s].y, (mw[s] >> (8 * ((ch0 + 1) >> 2))) & 255u);
                        }
                        *reinterpret_cast<uint4*>(eq + s * kDecExpStage + st0) = v0;
                        *reinterpret_cast<uint4*>(eq + s * kDecExpStage + st1) = v1;
                    }
                }
                // One proxy fence for both hand-offs: it makes the stores above visible to the tensor pipe, and it orders the
                // reads of the raw codes (whose values the stores depend on, so they have completed) before the TMA refill.
                ptx::fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) {
                    ptx::mbar_arrive(&e_full[st]);
                    ptx::mbar_arrive(&r_empty[sr]);
                }
                st ^= 1u;
                if (st == 0) st_ph ^= 1u;
                if (++sr == (uint32_t)SR) {
                    sr = 0;
                    sr_ph ^= 1u;
                }
            }
        }
    } else if (warp == kDecRawWarp) {
        // ------------------------------------------------------------------ raw weight-code producer
        if (lane == 0) {
            for (int q = 0; q < p.nprob; ++q) ptx::tma_prefetch_desc(&maps.w[q]);
            uint32_t qi = 0;
            bool ok = true;
            DecIter di(p, cta, nctas);
            DecSeg sg;
            while (ok && di.next(sg)) {
                const int nq = (sg.nkb + kDecQuad - 1) / kDecQuad;
                for (int j = 0; j < nq; ++j, ++qi) {
                    const uint32_t s = qi % (uint32_t)SR;
                    if (!ptx::mbar_wait_spin(&r_empty[s], ((qi / (uint32_t)SR) & 1u) ^ 1u, abort_flag)) {
                        dec_timeout(p.status, 5);
                        ok = false;
                        break;
                    }
                    // (a quad at the end of a segment loads k-blocks it does not use; past K the box is zero-filled)
                    ptx::mbar_arrive_expect_tx(&r_full[s], (uint32_t)kDecRawQuad);
                    ptx::tma_load_2d(ring_r + (size_t)s * kDecRawQuad, &maps.w[sg.prob], &r_full[s], (sg.kb0 + j * kDecQuad) * (kBK / 2), sg.n0);
                }
            }
        }
    } else if (warp == kDecTokWarp) {
        // ------------------------------------------------------------------ token-tile producer
        if (lane == 0) {
            for (int q = 0; q < p.nprob; ++q) {
                ptx::tma_prefetch_desc(&maps.a[q]);
                if (RES) ptx::tma_prefetch_desc(&maps.r[q]);
            }
            uint32_t qi = 0;
            bool ok = true;
            DecIter di(p, cta, nctas);
            DecSeg sg;
            while (ok && di.next(sg)) {
                const int nq = (sg.nkb + kDecQuad - 1) / kDecQuad;
                for (int j = 0; j < nq; ++j, ++qi) {
                    const uint32_t st = qi & 1u;
                    if (!ptx::mbar_wait_spin(&q_empty[st], ((qi >> 1) & 1u) ^ 1u, abort_flag)) {
                        dec_timeout(p.status, 1);
                        ok = false;
                        break;
                    }
                    const int valid = min(kDecQuad, sg.nkb - j * kDecQuad);
                    uint8_t* base = ring_a + (size_t)st * a_quad;
                    ptx::mbar_arrive_expect_tx(&a_full[st], (uint32_t)(valid * p.a_stage));
                    for (int s = 0; s < valid; ++s) {
                        const int kx = (sg.kb0 + j * kDecQuad + s) * kBK;
                        ptx::tma_load_2d(base + (size_t)s * p.a_stage, &maps.a[sg.prob], &a_full[st], kx, 0);
                        if (RES) ptx::tma_load_2d(base + (size_t)s * p.a_stage + tok_bytes, &maps.r[sg.prob], &a_full[st], kx, 0);
                    }
                }
            }
        }
    } else if (warp == kDecMmaWarp) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            // The residual operand's rows follow the main image's rows in a token stage: one MMA over both (N = 2 ntok)
            // accumulates the two terms side by side, and the epilogue adds them -- half as many instructions, each of
            // which costs the read of its 128 x 32-byte weight operand whatever N is.
            const uint32_t idesc = ptx::idesc_bf16_f32(kDecRows, RES ? 2 * ntok : ntok);
            const uint64_t desc0 = ptx::smem_desc_sw128_kmajor(0);  // everything but the start address
            const uint32_t w16 = (ptx::smem_u32(ring_e) & 0x3FFFFu) >> 4, t16 = (ptx::smem_u32(ring_a) & 0x3FFFFu) >> 4;
            const uint32_t a_quad16 = (uint32_t)(a_quad >> 4);
            const uint64_t a_stage16 = (uint64_t)(p.a_stage >> 4);
            uint32_t qi = 0;
            int lt = 0;
            bool ok = true;
            DecIter di(p, cta, nctas);
            DecSeg sg;
            while (ok && di.next(sg)) {
                const int buf = lt & 1;
                const uint32_t use = (uint32_t)(lt >> 1);
                ++lt;
                if (!ptx::mbar_wait_spin(&acc_empty[buf], (use & 1) ^ 1, abort_flag)) {
                    dec_timeout(p.status, 6);
                    break;
                }
                ptx::tc_fence_after();
                const uint32_t d = tmem_base + (uint32_t)(buf * 2 * kDecMaxTok);
                const int nq = (sg.nkb + kDecQuad - 1) / kDecQuad;
                for (int j = 0; j < nq; ++j, ++qi) {
                    const uint32_t st = qi & 1u;
                    ok = ptx::mbar_wait_spin(&e_full[st], (qi >> 1) & 1u, abort_flag) && ptx::mbar_wait_spin(&a_full[st], (qi >> 1) & 1u, abort_flag);
                    if (!ok) {
                        dec_timeout(p.status, 2);
                        break;
                    }
                    ptx::tc_fence_after();
                    const int valid = min(kDecQuad, sg.nkb - j * kDecQuad);
                    // This thread shares its scheduler with four expander warps: its instruction stream is kept short
                    // (descriptors advance by additions; a full quad is sixteen MMAs without a branch in between).
                    uint64_t wd = desc0 + (uint64_t)(w16 + st * (uint32_t)(kDecExpQuad >> 4));
                    uint64_t td = desc0 + (uint64_t)(t16 + st * a_quad16);
                    if (valid == kDecQuad) {
#pragma unroll
                        for (int s = 0; s < kDecQuad; ++s) {
#pragma unroll
                            for (int k = 0; k < kBK / 16; ++k)
                                ptx::umma_bf16(d, wd + (uint64_t)((s * kDecExpStage + k * 32) >> 4), td + (uint64_t)(2 * k), idesc,
                                               (j > 0 || s > 0 || k > 0) ? 1u : 0u);
                            td += a_stage16;
                        }
                    } else {
                        for (int s = 0; s < valid; ++s) {
#pragma unroll
                            for (int k = 0; k < kBK / 16; ++k)
                                ptx::umma_bf16(d, wd + (uint64_t)(2 * k), td + (uint64_t)(2 * k), idesc, (j > 0 || s > 0 || k > 0) ? 1u : 0u);
                            wd += (uint64_t)(kDecExpStage >> 4);
                            td += a_stage16;
                        }
                    }
                    ptx::umma_commit(&q_empty[st]);  // frees the token quad and the expanded quad
                }
                if (ok) ptx::umma_commit(&acc_full[buf]);
            }
        }
    } else if (warp >= kDecFirstEpiWarp) {
        // ------------------------------------------------------------------ epilogue: lane = weight row, column = token
        const int quad = warp & 3;
        const int row = quad * 32 + lane;
        const int et = row;  // thread index among the 128 epilogue threads
        int lt = 0;
        DecIter di(p, cta, nctas);
        DecSeg sg;
        while (di.next(sg)) {
            const DecProblem& pb = p.pr[sg.prob];
            const int buf = lt & 1;
            const uint32_t use = (uint32_t)(lt >> 1);
            ++lt;
            if (!ptx::mbar_wait(&acc_full[buf], use & 1, abort_flag)) {
                dec_timeout(p.status, 4);
                break;
            }
            ptx::tc_fence_after();
            const int64_t n = (int64_t)sg.n0 + row;
            float* slot = p.slots + (size_t)sg.slot * (size_t)ntok * kDecRows;
            const int nchunks = ntok / 16;
#pragma unroll 1
            for (int c = 0; c < nchunks; ++c) {
                uint32_t v[16];
                ptx::tmem_ld_32x16(tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(buf * 2 * kDecMaxTok + c * 16), v);
                if (RES) {
                    uint32_t vr[16];
                    ptx::tmem_ld_32x16(tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(buf * 2 * kDecMaxTok + ntok + c * 16), vr);
                    ptx::tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 16; ++j) v[j] = __float_as_uint(__uint_as_float(v[j]) + __uint_as_float(vr[j]));
                }
                ptx::tmem_ld_wait();
                if (c == nchunks - 1) {
                    ptx::tc_fence_before();
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive(&acc_empty[buf]);
                }
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const int m = c * 16 + j;
                    if (m >= pb.M) continue;
                    if (sg.partial) {
                        slot[(size_t)m * kDecRows + row] = __uint_as_float(v[j]);
                    } else if (n < pb.N) {
                        if (p.out_f32) reinterpret_cast<float*>(pb.Y)[(int64_t)m * pb.ldy + n] = __uint_as_float(v[j]);
                        else reinterpret_cast<__nv_bfloat16*>(pb.Y)[(int64_t)m * pb.ldy + n] = __float2bfloat16_rn(__uint_as_float(v[j]));
                    }
                }
            }
            if (sg.partial) {
                // count the segment in; the last arrival of the tile adds its segments in k order and writes Y
                const int64_t tb = pb.unit_base + (int64_t)(sg.tile - pb.tile_base) * pb.G, te = tb + pb.G;
                const int pf = dec_cta_of(p, tb, nctas), pl = dec_cta_of(p, te - 1, nctas);
                __threadfence();
                asm volatile("bar.sync 1, 128;" ::: "memory");
                if (et == 0) *s_last = (atomicAdd(&p.flags[sg.tile], 1u) + 1u == (unsigned)(pl - pf + 1)) ? 1 : 0;
                asm volatile("bar.sync 1, 128;" ::: "memory");
                const bool last = *s_last != 0;
                asm volatile("bar.sync 1, 128;" ::: "memory");  // (the flag is rewritten for the next segment)
                if (last) {
                    __threadfence();
                    if (n < pb.N) {
                        // eight tokens at a time, the loads of up to four segments in flight together; added in k order
                        for (int mb = 0; mb < pb.M; mb += 8) {
                            float acc[8];
#pragma unroll
                            for (int j = 0; j < 8; ++j) acc[j] = 0.f;
                            for (int c0 = pf; c0 <= pl; c0 += 4) {
                                float v[4][8];
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    const int c = c0 + e;
                                    const int sl = 2 * c + (dec_begin(p, c, nctas) >= tb ? 0 : 1);
                                    const float* src = p.slots + ((size_t)sl * ntok + mb) * kDecRows + row;
#pragma unroll
                                    for (int j = 0; j < 8; ++j) v[e][j] = (c <= pl && mb + j < pb.M) ? __ldcg(src + j * kDecRows) : 0.f;
                                }
#pragma unroll
                                for (int e = 0; e < 4; ++e)
#pragma unroll
                                    for (int j = 0; j < 8; ++j) acc[j] += v[e][j];
                            }
#pragma unroll
                            for (int j = 0; j < 8; ++j) {
                                const int m = mb + j;
                                if (m >= pb.M) continue;
                                if (p.out_f32) reinterpret_cast<float*>(pb.Y)[(int64_t)m * pb.ldy + n] = acc[j];
                                else reinterpret_cast<__nv_bfloat16*>(pb.Y)[(int64_t)m * pb.ldy + n] = __float2bfloat16_rn(acc[j]);
                            }
                        }
                    }
                }
            }
        }
    }
    ptx::tc_fence_before();
    __syncthreads();
    if (warp == kDecMmaWarp) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, kDecTmemCols);
    }
}

int res_of(const GemmArgs& g) { return g.r_bf16 ? 1 : 0; }

template <int FMT, bool RES>
int launch_decode(const GemmArgs* g, int count, cudaStream_t stream) {
    DecMaps maps;
    DecParams p;
    memset(&maps, 0, sizeof(maps));
    memset(&p, 0, sizeof(p));
    int ntok = 16;
    for (int i = 0; i < count; ++i) ntok = std::max(ntok, (int)((g[i].M + 15) / 16 * 16));
    p.nprob = count;
    p.ntok = ntok;
    int tile_base = 0;
    int64_t unit_base = 0;
    for (int i = 0; i < count; ++i) {
        const GemmArgs& a = g[i];
        const uint64_t pitch = (uint64_t)(a.lda ? a.lda : a.K) * 2;
        int rc = make_tmap_2d(&maps.a[i], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, a.a_bf16, (uint64_t)a.K, (uint64_t)a.M, pitch, kBK, (uint32_t)ntok,
                              CU_TENSOR_MAP_SWIZZLE_128B);
        if (rc) return rc;
        rc = make_tmap_2d(&maps.r[i], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, RES ? a.r_bf16 : a.a_bf16, (uint64_t)a.K, (uint64_t)a.M, pitch, kBK,
                          (uint32_t)ntok, CU_TENSOR_MAP_SWIZZLE_128B);
        if (rc) return rc;
        // packed codes of four k-blocks (128 bytes) x 128 rows, 128-byte swizzle (the expanders' reads are conflict-free)
        rc = make_tmap_2d(&maps.w[i], CU_TENSOR_MAP_DATA_TYPE_UINT8, a.w_codes, (uint64_t)a.K / 2, (uint64_t)a.N, (uint64_t)a.K / 2,
                          kDecQuad * (kBK / 2), (uint32_t)kDecRows, CU_TENSOR_MAP_SWIZZLE_128B);
        if (rc) return rc;
        DecProblem& pb = p.pr[i];
        pb.w_side = a.w_side;
        pb.Y = a.Y;
        pb.ldy = a.ldy;
        pb.M = (int)a.M;
        pb.N = (int)a.N;
        pb.G = (int)(a.K / kBK);
        pb.tile_base = tile_base;
        pb.unit_base = unit_base;
        const int tiles = (int)((a.N + kDecRows - 1) / kDecRows);
        tile_base += tiles;
        unit_base += (int64_t)tiles * pb.G;
    }
    for (int i = count; i < kMaxQuantGroup; ++i) {  // unused entries: never matched by the look-up
        maps.a[i] = maps.a[0];
        maps.r[i] = maps.r[0];
        maps.w[i] = maps.w[0];
        p.pr[i] = p.pr[count - 1];
        p.pr[i].tile_base = tile_base;
        p.pr[i].unit_base = unit_base;
    }
    p.units = unit_base;
    p.out_f32 = g[0].out_dtype == RESQ_OUT_F32;
    p.flags = g[0].sk_flags;
    p.slots = g[0].splitk_partials;
    p.status = g[0].status;
    p.a_stage = (RES ? 2 : 1) * ntok * 128;
    const int fixed = 2048 + kDecStages * kDecQuad * p.a_stage + kDecStages * kDecExpQuad;
    p.sr = std::min(4, (kDecSmem - fixed) / kDecRawQuad);
    const int smem_bytes = fixed + p.sr * kDecRawQuad;
    // every CTA gets at least four k-blocks
    const int nctas = (int)std::max<int64_t>(1, std::min<int64_t>(device_sm_count(), p.units / 4));
    if ((size_t)2 * nctas * ntok * kDecRows * sizeof(float) > g[0].partial_bytes || tile_base > kDecMaxTiles || p.sr < 2 ||
        smem_bytes > kDecSmem) {
        set_last_error("internal: decode GEMM launched outside its domain");
        return RESQ_ERR_CUDA;
    }
    auto kern = gemm_decode_kernel<FMT, RES>;
    int rc = ensure_dynamic_smem(reinterpret_cast<const void*>(kern), kDecSmem, "cudaFuncSetAttribute(gemm decode)");
    if (rc) return rc;
    LaunchScope scope(kKindGemm, stream);
    return cuda_fail(launch_kernel(kern, dim3((unsigned)nctas), dim3(kDecThreads), (size_t)smem_bytes, stream, maps, p),
                     "gemm_decode_kernel launch");
}

}  // namespace

// RESQ_GEMM_DECODE = 0 is the debugging override that keeps such calls on the other kernels.
bool gemm_decode_supported(const GemmArgs* g, int count) {
    if (count < 1 || count > kMaxQuantGroup || !env_int("RESQ_GEMM_DECODE", 1)) return false;
    int64_t tiles = 0;
    for (int i = 0; i < count; ++i) {
        const GemmArgs& a = g[i];
        if (a.M > kDecMaxTok || a.r_comp || a.w_bf16 || a.K % kBK != 0 || !a.sk_flags || !a.splitk_partials) return false;
        if (a.fmt != g[0].fmt || res_of(a) != res_of(g[0]) || a.out_dtype != g[0].out_dtype) return false;
        tiles += (a.N + kDecRows - 1) / kDecRows;
    }
    return tiles <= kDecMaxTiles && g[0].partial_bytes >= (size_t)2 * 148 * kDecMaxTok * kDecRows * sizeof(float);
}

int launch_gemm_decode(const GemmArgs* g, int count, cudaStream_t stream) {
    if (!gemm_decode_supported(g, count)) {
        set_last_error("internal: decode GEMM asked for outside its domain");
        return RESQ_ERR_CUDA;
    }
    const bool res = res_of(g[0]) != 0;
    if (g[0].fmt == kMXFP4) return res ? launch_decode<kMXFP4, true>(g, count, stream) : launch_decode<kMXFP4, false>(g, count, stream);
    return res ? launch_decode<kHiF4, true>(g, count, stream) : launch_decode<kHiF4, false>(g, count, stream);
}

}  // namespace resq
