// CTA-pair version of the HiF4 / MXFP4 GEMM of Eq. (5) (see gemm_hif4.cu for the numerics).
//
// Two CTAs on neighbouring SMs (a cluster of 2) compute one 256 x TN output tile with
// tcgen05.mma.cta_group::2: each CTA supplies the activation rows of its own 128 token rows and expands
// only HALF of the weight tile; the tensor cores read the other half from the peer's shared memory.
// Against the single-CTA kernel this halves the expansion work and the weight-side shared-memory fill per
// SM, which is what bounds that kernel.  No TMA multicast is used: every TMA load targets the issuing
// CTA's own shared memory; only mbarrier arrivals and tcgen05.commit cross the pair.
//
// Roles per CTA (8 + 4 * NG warps): warp 0 activation TMA, warp 1 MMA issue (leader CTA only) + TMEM alloc,
// warp 2 raw weight-code TMA, warps 4..7 epilogue, warps 8.. expanders in NG groups of four.  The leader's
// "full" barriers collect arrivals from both CTAs; "empty" barriers are released in both CTAs by a commit
// multicast.  Two schedules: whole tiles per pair (optionally with a K split and a separate reduce kernel), or
// K-streamed (the k-blocks of few tiles dealt out evenly; partial tiles go to fp32 slots and are summed in a
// fixed order at the end of the same kernel).  Residual term: a second dense A operand, or (2:4) the compressed
// operand on the structured-sparse MMA.  Weights: packed 4-bit codes expanded here, or plain bf16 by TMA.
#include "common.cuh"
#include "ptx.cuh"
#include "expand.cuh"

#include <algorithm>
#include <atomic>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <vector>

namespace resq {

namespace {

constexpr int kBM = 128;
constexpr int kBK = 64;
constexpr int kMaxBN = 256;
constexpr int kGroupWarps = 4;                       // expander warps per group
// Expander groups take k-blocks round-robin; k-block i uses slot i mod depth of each of the three rings
// (activation stages, raw codes, expanded weights; depths of at least NG, chosen in launch_pair_variant).  The
// number of groups NG (four warps each) is a template parameter of the kernel: more groups tolerate more
// hand-off latency, fewer groups fit wider tiles into shared memory (three slots of a 512-wide tile with a
// residual operand take 216 KB).
constexpr int kFirstEpiWarp = 4;
constexpr int kFirstExpWarp = 8;
constexpr int pair_threads(int groups) { return 32 * (kFirstExpWarp + kGroupWarps * groups); }
constexpr int kATileBytes = kBM * kBK * 2;
constexpr int kMaxRing = 8;
constexpr int kSmemBudget = 232448;
constexpr int kTmemCols = 512;

// One launch computes one problem (NP = 1) or a group of independent problems that share the residual mode, the weight
// format and the output type (NP = kMaxGroup): the tiles of all problems form one list, problem after problem.
constexpr int kMaxGroup = kMaxQuantGroup;

struct PairProblem {
    const void* w_side;
    void* Y;
    int64_t ldy;
    int M, N, G;             // token rows, output columns, k-blocks (K / 64)
    int ntiles_n;
    int tile_base;           // position of the problem's first tile in the launch's tile list
    int dealt_first;         // K-streamed schedule: first tile of the problem whose k-blocks are dealt out (else whole)
    int64_t unit_base;       //   and the (tile, k-block) units of the dealt tiles of the problems before it
    int meta_ka;             // sparse residual: metadata blocks (128 K positions) per 128-row band
    const uint8_t* blk_flags;  // dense residual from an unmasked image: keep flags [(M / 32), G] of the 32 x 64 blocks, or null
};

template <int NP>
struct PairMaps {
    CUtensorMap a[NP], r[NP], e[NP], w[NP];
};

template <int NP>
struct PairParams {
    PairProblem pr[NP];
    int nprob;
    int kblocks_per_split, splits;
    int num_tiles;
    int sa, sr, se, acc_bufs;
    int out_f32;
    float* partials;
    DeviceStatus* status;
#ifdef RESQ_TIMELINE
    int debug;
    unsigned int* timeline;  // device buffer for a per-role event log of pair 0 (or null)
    int timeline_first;      // first k-block iteration that is logged
    int timeline_pair;       // the pair that logs
#endif
    // K-streamed schedule (streamk != 0): the first dp_tiles tiles of the list are computed whole, tile t by pair
    // t mod npairs, and written out directly; the sk_units (tile, k-block) units of the remaining tiles are dealt
    // out in contiguous ranges: the pairs below sk_first (those that hold one whole tile more) take sk_hi units
    // each, the pairs sk_first .. sk_first + sk_pairs - 1 share the rest evenly.  A range may start and end inside
    // a tile's K range: such segments go to fp32 slots and are summed at the end of the kernel.
    int streamk;
    int dp_tiles;
    int sk_first, sk_hi, sk_pairs;
    int64_t sk_units;
    float* sk_slots;         // [2 * npairs][256][TN] fp32: slot 2p = first segment of pair p, 2p + 1 = its last
    unsigned int* sk_flags;  // [dealt tiles][2]: segments of the tile written, per CTA rank (zeroed before launch)
    int sk_poll_limit;       // polls (about 0.3 us each) before the wait for a tile's segments gives up
    int sk_extra;            // test hook (resq_debug_expire_next_wait): arrivals awaited beyond those that can come
};

__device__ __forceinline__ void report_timeout(DeviceStatus* st, int where) {
    if (atomicCAS(&st->code, 0, (int)RESQ_ERR_TIMEOUT) == 0) {
        st->where = where;
        st->block = (int)blockIdx.x;
    }
}

// In-kernel instrumentation (cycle counters per role, an event log of pair 0) exists only in builds with
// -DRESQ_TIMELINE, which the profiling experiments use; the shipped kernels carry none of it.
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
    int prob;      // problem of the tile
    int tile_id;   // K-streamed schedule: index of the segment's tile among the dealt tiles
    int slot;      //   and where its fp32 partial goes
    bool partial;  // the segment does not cover the whole K range (or K is split): fp32 partial output
};

// Problem that holds tile t of the launch's tile list (t below the total).
template <int NP>
__device__ __forceinline__ int problem_of_tile(const PairParams<NP>& p, int t) {
    int q = 0;
    if constexpr (NP > 1) {
#pragma unroll 1
        while (q + 1 < p.nprob && t >= p.pr[q + 1].tile_base) ++q;
    }
    return q;
}

// Whole-tile schedule of a single problem (tile list entry = (output tile, K split)).
template <int TN, int NP>
__device__ __forceinline__ TileCoord decode_tile(const PairParams<NP>& p, int tile) {
    TileCoord t;
    t.split = tile % p.splits;
    const int rest = tile / p.splits;
    t.prob = 0;
    t.n0 = (int64_t)(rest % p.pr[0].ntiles_n) * TN;
    t.m0 = (int64_t)(rest / p.pr[0].ntiles_n) * (2 * kBM);
    const int G = p.pr[0].G;
    t.kb_begin = t.split * p.kblocks_per_split;
    t.nkb = min(G, t.kb_begin + p.kblocks_per_split) - t.kb_begin;
    if (t.nkb < 0) t.nkb = 0;
    t.tile_id = rest;
    t.slot = 0;
    t.partial = p.splits > 1;
    return t;
}

// K-streamed schedule: first dealt unit of pair q (q may be one past the last pair), and the pair that owns unit u.
template <int NP>
__device__ __forceinline__ int64_t sk_begin(const PairParams<NP>& p, int q) {
    if (q < p.sk_first) return (int64_t)q * p.sk_hi;
    const int64_t head = (int64_t)p.sk_first * p.sk_hi;
    if (q >= p.sk_first + p.sk_pairs) return p.sk_units;
    return head + (int64_t)(q - p.sk_first) * (p.sk_units - head) / p.sk_pairs;
}
template <int NP>
__device__ __forceinline__ int sk_pair_of(const PairParams<NP>& p, int64_t u) {
    const int64_t head = (int64_t)p.sk_first * p.sk_hi;
    if (u < head) return (int)(u / p.sk_hi);
    return p.sk_first + (int)((((u - head + 1) * p.sk_pairs) - 1) / (p.sk_units - head));
}
// Dealt unit u -> problem, tile of the launch's list and k-block.
template <int NP>
__device__ __forceinline__ void sk_locate(const PairParams<NP>& p, int64_t u, int& prob, int& tile, int& kb) {
    int q = 0;
    if constexpr (NP > 1) {
#pragma unroll 1
        while (q + 1 < p.nprob && u >= p.pr[q + 1].unit_base) ++q;
    }
    const int64_t rel = u - p.pr[q].unit_base;
    const int tr = (int)(rel / p.pr[q].G);
    prob = q;
    tile = p.pr[q].dealt_first + tr;
    kb = (int)(rel - (int64_t)tr * p.pr[q].G);
}

// Walks the work of one pair in the order every role of the kernel uses.
template <int TN, int NP>
struct SegIter {
    const PairParams<NP>& p;
    int pair, npairs;
    int tile;            // next whole tile
    int64_t u0, u, u1;   // K-streamed schedule: this pair's dealt units
    __device__ SegIter(const PairParams<NP>& p_, int pair_, int npairs_) : p(p_), pair(pair_), npairs(npairs_) {
        tile = pair;
        u0 = u = u1 = 0;
        if (p.streamk) {
            u0 = u = sk_begin(p, pair);
            u1 = sk_begin(p, pair + 1);
        }
    }
    __device__ bool next(TileCoord& tc) {
        if (!p.streamk) {
            if (tile >= p.num_tiles) return false;
            tc = decode_tile<TN>(p, tile);
            tile += npairs;
            return true;
        }
        if (tile < p.dp_tiles) {  // whole tiles first
            const int q = problem_of_tile(p, tile);
            const int tl = tile - p.pr[q].tile_base;
            tc.prob = q;
            tc.tile_id = 0;
            tc.split = 0;
            tc.kb_begin = 0;
            tc.nkb = p.pr[q].G;
            tc.n0 = (int64_t)(tl % p.pr[q].ntiles_n) * TN;
            tc.m0 = (int64_t)(tl / p.pr[q].ntiles_n) * (2 * kBM);
            tc.partial = false;
            tc.slot = 0;
            tile += npairs;
            return true;
        }
        if (u >= u1) return false;
        int q, t, kb;
        sk_locate(p, u, q, t, kb);
        const int tl = t - p.pr[q].tile_base;
        tc.prob = q;
        tc.tile_id = t - p.dp_tiles;
        tc.split = 0;
        tc.kb_begin = kb;
        tc.nkb = (int)min((int64_t)(p.pr[q].G - kb), u1 - u);
        tc.n0 = (int64_t)(tl % p.pr[q].ntiles_n) * TN;
        tc.m0 = (int64_t)(tl / p.pr[q].ntiles_n) * (2 * kBM);
        tc.partial = tc.nkb < p.pr[q].G;
        tc.slot = 2 * pair + (u == u0 ? 0 : 1);
        u += tc.nkb;
        return true;
    }
};

__device__ __forceinline__ unsigned int ld_acquire_u32(const unsigned int* p) {
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ float4 ld_cg_f4(const float* p) {
    float4 v;
    asm volatile("ld.global.cg.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p));
    return v;
}

// End of the K-streamed kernel: the tiles whose K range this pair shared with other pairs are summed here.
// The pairs that hold segments of a tile each reduce one column slice of it: they wait until all segments of
// the tile are in their slots, then add them in k order (a fixed order: the result does not depend on timing).
// Called by all threads of the CTA; the CTA of rank r handles rows r * 128 .. r * 128 + 127 of the tile.
template <int TN, int NP>
__device__ __forceinline__ void streamk_fixup(const PairParams<NP>& p, int pair, int rank, volatile int* abort_flag,
                                              volatile int* s_ok, int* s_slots, unsigned int* evt, long long t0) {
    const int64_t u0 = sk_begin(p, pair), u1 = sk_begin(p, pair + 1);
    if (u1 <= u0) return;
    int q_first, t_first, q_last, t_last, kb_unused;
    sk_locate(p, u0, q_first, t_first, kb_unused);
    sk_locate(p, u1 - 1, q_last, t_last, kb_unused);
    for (int which = 0; which < 2; ++which) {
        const int t = which == 0 ? t_first : t_last;  // tile of the launch's list
        const int q = which == 0 ? q_first : q_last;
        if (which == 1 && t_last == t_first) break;
        const PairProblem& pb = p.pr[q];
        const int64_t tb = pb.unit_base + (int64_t)(t - pb.dealt_first) * pb.G, te = tb + pb.G;
        if (u0 <= tb && u1 >= te) continue;  // this pair computed the whole tile and wrote it out directly
        const int pf = sk_pair_of(p, tb), pl = sk_pair_of(p, te - 1);
        const int nseg = pl - pf + 1, j = pair - pf;
        if (threadIdx.x == 0) {
            int ok = *abort_flag ? 0 : 1;
            const unsigned int* flag = p.sk_flags + (t - p.dp_tiles) * 2 + rank;
            for (int polls = 0; ok && ld_acquire_u32(flag) < (unsigned)(nseg + p.sk_extra); ++polls) {
                __nanosleep(200);
                if (polls > p.sk_poll_limit) {
                    report_timeout(p.status, 7);
                    ok = 0;
                }
            }
            *s_ok = ok;
        }
        __syncthreads();
        const bool ok = *s_ok != 0;
        __syncthreads();
        if (!ok) return;
        if (evt && threadIdx.x == 0) evt[which] = (unsigned int)(clock64() - t0);
        // slot of every segment (k order), worked out once per tile
        if ((int)threadIdx.x < nseg) {
            const int sq = pf + (int)threadIdx.x;
            s_slots[threadIdx.x] = 2 * sq + (sk_begin(p, sq) >= tb ? 0 : 1);
        }
        __syncthreads();
        // column slice j of nseg, in units of 4 columns
        const int c0 = (int)((int64_t)j * (TN / 4) / nseg) * 4, c1 = (int)((int64_t)(j + 1) * (TN / 4) / nseg) * 4;
        const int w4 = (c1 - c0) / 4;
        const int tl = t - pb.tile_base;
        const int64_t m_base = (int64_t)(tl / pb.ntiles_n) * (2 * kBM) + rank * kBM;
        const int64_t n_base = (int64_t)(tl % pb.ntiles_n) * TN;
        for (int item = threadIdx.x; item < kBM * w4; item += (int)blockDim.x) {
            const int row = item / w4, c = c0 + (item % w4) * 4;
            const int64_t m = m_base + row, n = n_base + c;
            if (m >= pb.M || n >= pb.N) continue;
            const float* src = p.sk_slots + ((size_t)rank * kBM + row) * TN + c;
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int s0 = 0; s0 < nseg; s0 += 4) {
                float4 v[4];
#pragma unroll
                for (int e = 0; e < 4; ++e)  // the loads of a group of four segments are in flight together
                    v[e] = s0 + e < nseg ? ld_cg_f4(src + (size_t)s_slots[s0 + e] * (2 * kBM) * TN) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    acc.x += v[e].x; acc.y += v[e].y; acc.z += v[e].z; acc.w += v[e].w;
                }
            }
            const float o[4] = {acc.x, acc.y, acc.z, acc.w};
            if (p.out_f32) {
                float* dst = reinterpret_cast<float*>(pb.Y) + m * pb.ldy + n;
                if (n + 3 < pb.N) *reinterpret_cast<float4*>(dst) = acc;
                else for (int e = 0; e < 4; ++e) if (n + e < pb.N) dst[e] = o[e];
            } else {
                __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(pb.Y) + m * pb.ldy + n;
                if (n + 3 < pb.N) {
                    __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y), hi = __floats2bfloat162_rn(acc.z, acc.w);
                    *reinterpret_cast<uint2*>(dst) = make_uint2(*reinterpret_cast<uint32_t*>(&lo), *reinterpret_cast<uint32_t*>(&hi));
                } else {
                    for (int e = 0; e < 4; ++e) if (n + e < pb.N) dst[e] = __float2bfloat16_rn(o[e]);
                }
            }
        }
        __syncthreads();  // the slot list is rewritten for the next tile
    }
}

// Weight formats of the kernel: the two packed 4-bit formats (expanded in the kernel), or plain bf16 weights that
// TMA writes straight into the slots of the expanded-weight ring (activation-only quantization, "W16A4").
constexpr int kPlainW = 2;

// Residual term of the kernel: none, a dense second A operand (the masked bf16 image), or the 2:4 compressed image
// with its index metadata on the structured-sparse MMA (half the tensor work of the dense form).
enum ResMode : int { kResNone = 0, kResDense = 1, kResSparse24 = 2 };
constexpr int kSpTileBytes = kATileBytes / 2;  // compressed residual tile: 128 rows x 32 kept values (64-byte rows)
constexpr int kSpMetaBytes = 2048;             // index metadata of 128 rows x 128 K positions (two k-blocks)
constexpr int kSpTmemCol = kTmemCols - 8;      // two metadata buffers of four columns at the end of tensor memory
__host__ __device__ constexpr int a_stage_bytes(int res) {
    return res == kResDense ? 2 * kATileBytes : res == kResSparse24 ? kATileBytes + kSpTileBytes + kSpMetaBytes : kATileBytes;
}

// TN: width of the pair's output tile (the pair computes 256 x TN); bn = MMA N; each CTA expands TN/2 rows.
template <int RES, int TN, int FMT, int NG, int NP>
__global__ void __launch_bounds__(pair_threads(NG), 1)
gemm_pair_kernel(const __grid_constant__ PairMaps<NP> maps, const __grid_constant__ PairParams<NP> p) {
    constexpr int kExpGroups = NG;
    constexpr int kAStage = a_stage_bytes(RES);
    constexpr int nt = TN > kMaxBN ? 2 : 1;           // MMAs side by side in N
    constexpr int bn = TN / nt;                    // MMA N
    constexpr int half = bn / 2;                   // rows of each MMA's weight tile held by one CTA
    constexpr int my_rows = nt * half;             // rows this CTA expands per k-block
    constexpr int exp_stage = my_rows * 128, raw_stage = FMT == kPlainW ? 0 : my_rows * 32;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int SA = p.sa, SR = p.sr, SE = p.se;
    uint8_t* ring_a = smem;
    uint8_t* ring_e = ring_a + (size_t)SA * kAStage;
    uint8_t* ring_r = ring_e + (size_t)SE * exp_stage;
    uint64_t* bars = reinterpret_cast<uint64_t*>(ring_r + (size_t)SR * raw_stage);
    // All three rings have one slot per expander group, and slot s of each holds k-block it = s (mod NG): one
    // "full" barrier per slot collects the activation bytes of both CTAs and the arrivals of both CTAs' expander
    // group, and one "empty" barrier per slot (a single commit) releases the activation stage and the expanded
    // stage together.  The MMA thread thus does one wait and one commit per k-block.
    uint64_t* a_full = bars;                   // leader: both CTAs' activation stages landed and expanded halves written
    uint64_t* a_empty = bars + kMaxRing;       // each CTA: the MMAs that read the slot completed
    uint64_t* r_full = bars + 2 * kMaxRing;    // each CTA: own raw codes landed
    uint64_t* r_empty = bars + 3 * kMaxRing;   // each CTA: own expanders consumed them
    uint64_t* e_full = a_full;                 // (same barriers: see above)
    uint64_t* e_empty = a_empty;
    uint64_t* acc_full = bars + 6 * kMaxRing;  // [2] each CTA
    uint64_t* acc_empty = acc_full + 2;        // [2] leader: both epilogues drained
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
#ifdef RESQ_TIMELINE
    unsigned int* tlog = reinterpret_cast<unsigned int*>(tmem_slot + 4);  // [8 roles][32 iterations] (512 B)
    const bool tl = p.timeline != nullptr && (int)(blockIdx.x >> 1) == p.timeline_pair;
    const int kTl0 = p.timeline_first;  // first logged iteration
#define EVT(k) do { if (tl) p.timeline[512 + (int)rank * 16 + (k)] = (unsigned int)(clock64() - t_kernel0); } while (0)
#define TLOG(role, it) do { if (tl && (it) >= kTl0 && (it) < kTl0 + 32) tlog[(role) * 32 + ((it) - kTl0)] = (unsigned int)clock64(); } while (0)
    const long long t_entry = clock64();
#else
#define EVT(k) do { } while (0)
#define TLOG(role, it) do { } while (0)
#endif
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = ptx::cluster_ctarank();  // 0 = leader
    const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kMaxRing; ++s) {
            // an arrive.expect_tx per CTA for the activations, and one expander group per CTA (packed weights) or a
            // second arrive.expect_tx per CTA (bf16 weights)
            ptx::mbar_init(&a_full[s], FMT == kPlainW ? 4 : 2 + 2 * kGroupWarps);
            ptx::mbar_init(&a_empty[s], 1);
            ptx::mbar_init(&r_full[s], 1);
            ptx::mbar_init(&r_empty[s], kGroupWarps);
        }
        for (int b = 0; b < 2; ++b) {
            ptx::mbar_init(&acc_full[b], 1);
            ptx::mbar_init(&acc_empty[b], 8);              // four epilogue warps per CTA
        }
        *abort_flag = 0;
        ptx::mbar_fence_init();
    }
    if (warp == 1) ptx::tmem_alloc_pair(tmem_slot, kTmemCols);
    ptx::tc_fence_before();
    __syncthreads();
    ptx::cluster_sync();  // the peer's barriers exist before anything arrives on them
    ptx::tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
#ifdef RESQ_TIMELINE
    const long long t_kernel0 = clock64();
    Trace tr{(p.debug & 16) ? reinterpret_cast<unsigned long long*>(p.status) + 8 : nullptr, 0};
    if (tl && threadIdx.x == 0) p.timeline[512 + (int)rank * 16] = (unsigned int)(t_kernel0 - t_entry);
#else
    Trace tr;
#endif
    // Programmatic dependent launch: the set-up above overlaps the tail of the quantizer kernel.  The weight side
    // (raw-code producer, expanders) reads only the packed weights, which no kernel since the start of the
    // quantizer writes, and starts at once; everything else waits for the quantizer's outputs.
    pdl_trigger();
    if (!(warp == 2 || warp >= kFirstExpWarp)) pdl_wait();

    if (warp == 0) {
        // ------------------------------------------------------------------ activation producer (both CTAs)
        if (lane == 0) {
            for (int q = 0; q < (NP > 1 ? p.nprob : 1); ++q) {
                ptx::tma_prefetch_desc(&maps.a[q]);
                if (RES != kResNone) ptx::tma_prefetch_desc(&maps.r[q]);
                if (RES == kResSparse24 || (RES == kResDense && p.pr[q].blk_flags)) ptx::tma_prefetch_desc(&maps.e[q]);
            }
            uint32_t it = 0;
            bool ok = true;
            SegIter<TN, NP> si(p, pair, npairs);
            TileCoord tc;
            while (ok && si.next(tc)) {
                const int my_m = (int)(tc.m0 + rank * kBM);
                const CUtensorMap* tmap_a = &maps.a[tc.prob];
                const CUtensorMap* tmap_r = &maps.r[tc.prob];
                const CUtensorMap* tmap_e = &maps.e[tc.prob];
                const int meta_ka = p.pr[tc.prob].meta_ka;
                // Block-wise selection: the residual tile is loaded as four boxes of 32 rows, a dropped block from beyond the
                // tensor's last row (TMA fills it with zeros and reads nothing).  The flags of a k-block are fetched while
                // the previous one waits for its slot.
                const uint8_t* blk_flags = RES == kResDense ? p.pr[tc.prob].blk_flags : nullptr;
                const int blk_G = p.pr[tc.prob].G, blk_M = p.pr[tc.prob].M;
                const int oob_row = (blk_M + 2 * kBM - 1) / (2 * kBM) * (2 * kBM);
                uint32_t fl[4] = {0u, 0u, 0u, 0u};
                auto fetch_flags = [&](int kb) {
#pragma unroll
                    for (int g = 0; g < 4; ++g) {
                        const int row = my_m + 32 * g;
                        fl[g] = row < blk_M ? ptx::ld_nc_u8(blk_flags + (size_t)(row >> 5) * blk_G + kb) : 0u;
                    }
                };
                if (blk_flags && tc.nkb > 0) fetch_flags(tc.kb_begin);
                for (int i = 0; i < tc.nkb; ++i, ++it) {
                    // The activation ring may be shallower than the ring of expanded weights whose barriers it shares
                    // (barrier slot = k-block mod SE): slot it % SA is free once the MMAs of k-block it - SA, which
                    // signal barrier (it - SA) % SE, completed.  (That barrier cannot run a phase ahead: its next
                    // phase needs the k-block it - SA + SE >= it, which this thread has not loaded yet.)
                    const int s = it % SA, sb = it % SE;
                    tr.begin();
                    const uint32_t prev = it - (uint32_t)SA;
                    const bool got = it < (uint32_t)SA || ptx::mbar_wait_spin(&a_empty[prev % SE], (prev / SE) & 1, abort_flag);
                    tr.end(0);
                    if (!got) {
                        report_timeout(p.status, 1);
                        ok = false;
                        break;
                    }
                    uint8_t* st = ring_a + (size_t)s * kAStage;
                    TLOG(0, it);
                    if (it == 0) EVT(1);
                    const uint32_t full = ptx::map_to_cta(&a_full[sb], 0);
                    const int kb = tc.kb_begin + i;
                    // the metadata of two k-blocks travels with the even one (or with the first of a K range)
                    const bool with_meta = RES == kResSparse24 && ((kb & 1) == 0 || i == 0);
                    ptx::mbar_arrive_expect_tx_cluster_relaxed(  // publishes nothing itself
                        full, (uint32_t)(kAStage - (RES == kResSparse24 && !with_meta ? kSpMetaBytes : 0)));
                    const int kx = kb * kBK;
                    ptx::tma_load_2d_pair(st, tmap_a, full, kx, my_m);
                    if (RES == kResDense) {
                        if (blk_flags) {
#pragma unroll
                            for (int g = 0; g < 4; ++g)
                                ptx::tma_load_2d_pair(st + kATileBytes + g * 32 * 128, tmap_e, full, kx, fl[g] ? my_m + 32 * g : oob_row);
                            if (i + 1 < tc.nkb) fetch_flags(kb + 1);
                        } else {
                            ptx::tma_load_2d_pair(st + kATileBytes, tmap_r, full, kx, my_m);
                        }
                    }
                    if (RES == kResSparse24) {
                        ptx::tma_load_2d_pair(st + kATileBytes, tmap_r, full, kx / 2, my_m);
                        if (with_meta)  // rows of 256 bytes, eight per 128 x 128 block
                            ptx::tma_load_2d_pair(st + kATileBytes + kSpTileBytes, tmap_e, full, 0,
                                                  ((my_m >> 7) * meta_ka + (kb >> 1)) * 8);
                    }
                }
            }
        }
    } else if (warp == 2) {
        // ------------------------------------------------------------------ raw weight-code producer (both CTAs)
        if (lane == 0) {
            for (int q = 0; q < (NP > 1 ? p.nprob : 1); ++q) ptx::tma_prefetch_desc(&maps.w[q]);
            uint32_t it = 0;
            bool ok = true;
            SegIter<TN, NP> si(p, pair, npairs);
            TileCoord tc;
            while (ok && si.next(tc)) {
                const CUtensorMap* tmap_w = &maps.w[tc.prob];
                if constexpr (FMT == kPlainW) {
                    // bf16 weights: this CTA's rows of the k-block go straight into the expanded-weight slot
                    for (int i = 0; i < tc.nkb; ++i, ++it) {
                        const int se = it % SE;
                        if (!ptx::mbar_wait_spin(&e_empty[se], ((it / SE) & 1) ^ 1, abort_flag)) {
                            report_timeout(p.status, 5);
                            ok = false;
                            break;
                        }
                        const uint32_t full = ptx::map_to_cta(&e_full[se], 0);
                        ptx::mbar_arrive_expect_tx_cluster_relaxed(full, (uint32_t)exp_stage);
#pragma unroll
                        for (int j = 0; j < nt; ++j)
                            ptx::tma_load_2d_pair(ring_e + (size_t)se * exp_stage + (size_t)j * half * 128, tmap_w, full,
                                                  (tc.kb_begin + i) * kBK, (int)(tc.n0 + j * bn + rank * half));
                    }
                } else {
                for (int i = 0; i < tc.nkb; ++i, ++it) {
                    const int s = it % SR;
                    tr.begin();
                    const bool got = ptx::mbar_wait_spin(&r_empty[s], ((it / SR) & 1) ^ 1, abort_flag);
                    tr.end(1);
                    if (!got) {
                        report_timeout(p.status, 5);
                        ok = false;
                        break;
                    }
                    TLOG(1, it);
                    ptx::mbar_arrive_expect_tx(&r_full[s], (uint32_t)raw_stage);
#pragma unroll
                    for (int j = 0; j < nt; ++j)
                        ptx::tma_load_2d(ring_r + (size_t)s * raw_stage + (size_t)j * half * 32, tmap_w, &r_full[s],
                                         (tc.kb_begin + i) * (kBK / 2), (int)(tc.n0 + j * bn + rank * half));
                }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (leader CTA only)
        if (lane == 0 && rank == 0) {
            const uint32_t idesc = ptx::idesc_bf16_f32(2 * kBM, bn);
            const uint64_t desc0 = ptx::smem_desc_sw128_kmajor(0);  // everything but the start address
            const uint64_t desc0_sp = ptx::smem_desc_sw64_kmajor(0);
            const uint64_t desc0_e = ptx::smem_desc_rows16(0);
            uint32_t ebuf = 0;  // metadata buffer (four tensor-memory columns) in use
            const uint32_t a_base16 = (ptx::smem_u32(ring_a) & 0x3FFFFu) >> 4, e_base16 = (ptx::smem_u32(ring_e) & 0x3FFFFu) >> 4;
            uint32_t it = 0, sa = 0, se = 0, pha = 0;  // activation slot, barrier / weight slot and its phase parity
            int local_tile = 0;
            bool ok = true;
            SegIter<TN, NP> si(p, pair, npairs);
            TileCoord tc;
            while (ok && si.next(tc)) {
                const int lt = local_tile++;
                if (tc.nkb == 0) continue;
                const int buf = p.acc_bufs == 2 ? (lt & 1) : 0;
                const uint32_t use = p.acc_bufs == 2 ? (uint32_t)(lt >> 1) : (uint32_t)lt;
                tr.begin();
                const bool got_acc = ptx::mbar_wait_spin(&acc_empty[buf], (use & 1) ^ 1, abort_flag);
                tr.end(4);
                if (!got_acc) {
                    report_timeout(p.status, 6);
                    break;
                }
                ptx::tc_fence_after();
                const uint32_t d0 = tmem_base + (uint32_t)(buf * TN);
                for (int i = 0; i < tc.nkb; ++i, ++it) {
                    // This thread's instruction stream sits between the MMAs of consecutive k-blocks: stage
                    // indices, phases and descriptors advance by additions only.
                    tr.begin();
                    ok = ptx::mbar_wait_spin(&a_full[se], pha, abort_flag);
                    tr.end(2);
                    if (!ok) {
                        report_timeout(p.status, 2);
                        break;
                    }
                    tr.begin();
                    TLOG(2, it);
                    if (it == 0) EVT(2);
                    ptx::tc_fence_after();
                    const uint32_t a16 = a_base16 + sa * (uint32_t)(kAStage >> 4);
                    const uint64_t adesc = desc0 + (uint64_t)a16;
                    const uint64_t bdesc = desc0 + (uint64_t)(e_base16 + se * (uint32_t)(exp_stage >> 4));
                    uint32_t e_col = 0;
                    if (RES == kResSparse24) {
                        const int kb = tc.kb_begin + i;
                        if ((kb & 1) == 0 || i == 0) {
                            ebuf ^= 1u;
                            ptx::tmem_cp_128x128b_pair(tmem_base + (uint32_t)kSpTmemCol + 4u * ebuf,
                                                       desc0_e + (uint64_t)(a16 + (uint32_t)((kATileBytes + kSpTileBytes) >> 4)));
                        }
                        e_col = tmem_base + (uint32_t)kSpTmemCol + 4u * ebuf + 2u * (uint32_t)(kb & 1);
                    }
#pragma unroll
                    for (int k = 0; k < kBK / 16; ++k) {
#pragma unroll
                        for (int j = 0; j < nt; ++j) {
                            const uint64_t bd = bdesc + (uint64_t)((j * half * 128 + k * 32) >> 4);
                            const uint32_t d = d0 + (uint32_t)(j * bn);
                            ptx::umma_bf16_pair(d, adesc + (uint64_t)((k * 32) >> 4), bd, idesc, (i > 0 || k > 0) ? 1u : 0u);
                            if (RES == kResDense)
                                ptx::umma_bf16_pair(d, adesc + (uint64_t)((kATileBytes + k * 32) >> 4), bd, idesc, 1u);
                            if (RES == kResSparse24 && (k & 1)) {
                                // 32 K positions per instruction: 32 bytes of the compressed rows, 64 bytes of the weight rows
                                const int k2 = k >> 1;
                                ptx::umma_bf16_sp_pair(d, desc0_sp + (uint64_t)(a16 + (uint32_t)((kATileBytes + k2 * 32) >> 4)),
                                                       bdesc + (uint64_t)((j * half * 128 + k2 * 64) >> 4), e_col,
                                                       ptx::sparse_idesc(idesc, (uint32_t)k2), 1u);
                            }
                        }
                    }
                    ptx::umma_commit_pair(&a_empty[se], 3);  // frees the slots in both CTAs
                    if (++sa == (uint32_t)SA) sa = 0;
                    if (++se == (uint32_t)SE) { se = 0; pha ^= 1u; }
                    TLOG(3, it);
                    tr.end(5);
                }
                if (ok) ptx::umma_commit_pair(&acc_full[buf], 3);
                EVT(3);
            }
        }
    } else if (warp >= kFirstExpWarp && FMT != kPlainW) {
        // ------------------------------------------------------------------ expanders (both CTAs, own half)
        // NG groups of four warps take k-blocks round-robin, so each group has NG MMA periods for one block:
        // the per-block synchronisation latency (two waits, two arrives, one proxy fence) stays off the
        // critical path.
        const int ew = (warp - kFirstExpWarp) % kGroupWarps;
        const int grp = (warp - kFirstExpWarp) / kGroupWarps;
        constexpr int rows_per_warp = my_rows / kGroupWarps;  // 8, 16 or 32
        const int r_begin = ew * rows_per_warp;
        const int sub_row = lane >> 3, chunk = lane & 7;
        // Byte offsets of this lane's 16-byte stores into an expanded slot, for even and odd q (row r = r_begin + 4 q +
        // sub_row, chunk column chunk ^ (r & 7)): rows four apart flip bit 2 of the swizzle, rows eight apart share it.
        const uint32_t st_even = (uint32_t)((r_begin + sub_row) * 128 + ((chunk ^ ((r_begin + sub_row) & 7)) << 4));
        const uint32_t st_odd = (uint32_t)((r_begin + sub_row + 4) * 128 + ((chunk ^ ((r_begin + sub_row + 4) & 7)) << 4));
        uint32_t it0 = 0;  // k-block counter at the start of the current tile
        bool ok = true;
        SegIter<TN, NP> si(p, pair, npairs);
        TileCoord tc;
        while (ok && si.next(tc)) {
            // local row l (< my_rows) is weight row n0 + (l / half) * bn + rank * half + (l % half);
            // lane l owns the metadata of rows l and 32 + l of this warp's slice
            auto row_of = [&](int l) -> int64_t { return tc.n0 + (int64_t)(l / half) * bn + rank * half + (l % half); };
            const int64_t n_a = row_of(r_begin + lane);
            const int64_t n_b = row_of(r_begin + (rows_per_warp > 32 ? 32 + lane : lane));
            const PairProblem& pb = p.pr[tc.prob];
            const int64_t G = pb.G;
            const void* w_side = pb.w_side;
            const bool ok_a = lane < rows_per_warp && n_a < pb.N;
            const bool ok_b = rows_per_warp > 32 && n_b < pb.N;
            auto load_side = [&](int64_t n, int kb) -> uint32_t {
                if (FMT == kHiF4) return ptx::ld_nc_u32(reinterpret_cast<const uint32_t*>(w_side) + n * G + kb);
                return ptx::ld_nc_u16(reinterpret_cast<const uint16_t*>(w_side) + n * G + kb);
            };
            // first k-block of this tile that belongs to this group
            int i = (int)((grp + kExpGroups - (it0 % kExpGroups)) % kExpGroups);
            uint32_t ma_next = (ok_a && i < tc.nkb) ? load_side(n_a, tc.kb_begin + i) : 0u;
            uint32_t mb_next = (ok_b && i < tc.nkb) ? load_side(n_b, tc.kb_begin + i) : 0u;
            for (; i < tc.nkb; i += kExpGroups) {
                const uint32_t it = it0 + (uint32_t)i;
                const uint32_t ma = ma_next, mb = mb_next;
                if (i + kExpGroups < tc.nkb) {
                    ma_next = ok_a ? load_side(n_a, tc.kb_begin + i + kExpGroups) : 0u;
                    mb_next = ok_b ? load_side(n_b, tc.kb_begin + i + kExpGroups) : 0u;
                }
                const int sr = it % SR, se = it % SE;
                if (ew == 0 && lane == 0 && grp == 0) tr.begin();
                ok = ptx::mbar_wait(&e_empty[se], ((it / SE) & 1) ^ 1, abort_flag);
                if (ew == 0 && lane == 0 && grp == 0) { tr.end(6); tr.begin(); TLOG(4, it); }
                ok = ok && ptx::mbar_wait(&r_full[sr], (it / SR) & 1, abort_flag);
                if (ew == 0 && lane == 0 && grp == 0) { tr.end(7); tr.begin(); TLOG(5, it); }
                if (!ok) {
                    report_timeout(p.status, 3);
                    break;
                }
                const uint32_t* raw = reinterpret_cast<const uint32_t*>(ring_r + (size_t)sr * raw_stage);
                uint8_t* bexp = ring_e + (size_t)se * exp_stage;
                constexpr int kIters = rows_per_warp / 4;
                uint32_t cw[kIters], mw[kIters];
#pragma unroll
                for (int q = 0; q < kIters; ++q) {
                    const int rl = q * 4 + sub_row;
                    mw[q] = __shfl_sync(0xFFFFFFFFu, q < 8 ? ma : mb, rl & 31);
                    cw[q] = raw[(r_begin + rl) * 8 + chunk];
                }
                // The raw slot goes back to the TMA producer, whose next load overwrites it through the async proxy: the
                // reads above (generic proxy) are ordered before that by a proxy fence.  Without it the loads of the
                // later rows were found to execute after the arrive, late enough to read 128-byte pieces of the next
                // k-block's codes (wrong expanded rows in groups of four).
                ptx::fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&r_empty[sr]);
#pragma unroll
                for (int q = 0; q < kIters; ++q) {
                    const uint4 v = FMT == kHiF4 ? expand_hif4_chunk(cw[q], mw[q], chunk)
                                                 : expand_mxfp4_chunk(cw[q], (mw[q] >> (8 * (chunk >> 2))) & 255u);
                    *reinterpret_cast<uint4*>(bexp + ((q & 1) ? st_odd : st_even) + (q >> 1) * 1024) = v;
                }
                ptx::fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive_cluster(ptx::map_to_cta(&e_full[se], 0));
                if (ew == 0 && lane == 0 && grp == 0) { tr.end(8); TLOG(6, it); }
            }
            it0 += (uint32_t)tc.nkb;
        }
    } else if (warp >= kFirstEpiWarp && warp < kFirstExpWarp) {
        // ------------------------------------------------------------------ epilogue (both CTAs, own 128 rows)
        const int quad = warp & 3;
        constexpr int nchunks = TN / 32;
        int local_tile = 0;
        SegIter<TN, NP> si(p, pair, npairs);
        TileCoord tc;
        while (si.next(tc)) {
            const int lt = local_tile++;
            if (tc.nkb == 0) continue;
            const PairProblem& pb = p.pr[tc.prob];
            const int64_t pM = pb.M, pN = pb.N, ldy = pb.ldy;
            const int buf = p.acc_bufs == 2 ? (lt & 1) : 0;
            const uint32_t use = p.acc_bufs == 2 ? (uint32_t)(lt >> 1) : (uint32_t)lt;
            if (quad == 0 && lane == 0) tr.begin();
            const bool got_full = ptx::mbar_wait(&acc_full[buf], use & 1, abort_flag);
            if (quad == 0 && lane == 0) { tr.end(9); tr.begin(); EVT(4); }
            if (!got_full) {
                report_timeout(p.status, 4);
                break;
            }
            ptx::tc_fence_after();
            const int64_t m = tc.m0 + rank * kBM + quad * 32 + lane;
            // a warp whose 32 rows all lie past M (decode-sized calls fill a fraction of the 256-row tile) has
            // nothing to read or store: it only hands the accumulator back
            const bool warp_has_rows = tc.m0 + rank * kBM + quad * 32 < pM;
#pragma unroll 1
            for (int cc = warp_has_rows ? 0 : nchunks - 1; cc < nchunks; ++cc) {
                uint32_t v[32];
                if (warp_has_rows) {
                    ptx::tmem_ld_32x32(tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(buf * TN + cc * 32), v);
                    ptx::tmem_ld_wait();
                }
                if (cc == nchunks - 1) {
                    ptx::tc_fence_before();
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive_cluster(ptx::map_to_cta(&acc_empty[buf], 0));
                }
                if (!warp_has_rows) continue;
                if (p.streamk && tc.partial) {
                    // fp32 slot [256][TN]; the sum reads rows below M only, so rows past M are not written
                    if (m >= pM) continue;
                    float* dst = p.sk_slots + ((size_t)tc.slot * (2 * kBM) + rank * kBM + quad * 32 + lane) * TN + cc * 32;
#pragma unroll
                    for (int j = 0; j < 32; j += 8)
                        ptx::st_global_v8(dst + j, v[j], v[j + 1], v[j + 2], v[j + 3], v[j + 4], v[j + 5], v[j + 6], v[j + 7]);
                    continue;
                }
                if (m >= pM) continue;
                const int64_t nb = tc.n0 + cc * 32;
                const int64_t left = pN - nb;
                if (left <= 0) continue;
                if (p.splits > 1) {
                    float* dst = p.partials + ((int64_t)tc.split * pM + m) * pN + nb;
                    if (left >= 32 && (reinterpret_cast<uintptr_t>(dst) & 31u) == 0) {
#pragma unroll
                        for (int j = 0; j < 32; j += 8)
                            ptx::st_global_v8(dst + j, v[j], v[j + 1], v[j + 2], v[j + 3], v[j + 4], v[j + 5], v[j + 6], v[j + 7]);
                    } else if (left >= 32 && (pN & 3) == 0) {
#pragma unroll
                        for (int j = 0; j < 32; j += 4)
                            *reinterpret_cast<uint4*>(dst + j) = make_uint4(v[j], v[j + 1], v[j + 2], v[j + 3]);
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (j < left) dst[j] = __uint_as_float(v[j]);
                    }
                } else if (p.out_f32) {
                    float* dst = reinterpret_cast<float*>(pb.Y) + m * ldy + nb;
                    if (left >= 32 && (reinterpret_cast<uintptr_t>(dst) & 31u) == 0) {
#pragma unroll
                        for (int j = 0; j < 32; j += 8)
                            ptx::st_global_v8(dst + j, v[j], v[j + 1], v[j + 2], v[j + 3], v[j + 4], v[j + 5], v[j + 6], v[j + 7]);
                    } else if (left >= 32) {
#pragma unroll
                        for (int j = 0; j < 32; j += 4)
                            *reinterpret_cast<uint4*>(dst + j) = make_uint4(v[j], v[j + 1], v[j + 2], v[j + 3]);
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (j < left) dst[j] = __uint_as_float(v[j]);
                    }
                } else {
                    __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(pb.Y) + m * ldy + nb;
                    if (left >= 32) {
                        uint32_t o[16];
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            __nv_bfloat162 b = __floats2bfloat162_rn(__uint_as_float(v[2 * j]), __uint_as_float(v[2 * j + 1]));
                            o[j] = *reinterpret_cast<uint32_t*>(&b);
                        }
                        if ((reinterpret_cast<uintptr_t>(dst) & 31u) == 0) {  // two full 32-byte sectors per thread
                            ptx::st_global_v8(dst, o[0], o[1], o[2], o[3], o[4], o[5], o[6], o[7]);
                            ptx::st_global_v8(dst + 16, o[8], o[9], o[10], o[11], o[12], o[13], o[14], o[15]);
                        } else {
#pragma unroll
                            for (int j = 0; j < 16; j += 4)
                                *reinterpret_cast<uint4*>(dst + 2 * j) = make_uint4(o[j], o[j + 1], o[j + 2], o[j + 3]);
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (j < left) dst[j] = __float2bfloat16_rn(__uint_as_float(v[j]));
                    }
                }
            }
            if (p.streamk && tc.partial) {
                // publish the slot: every epilogue thread fences its stores, then one thread counts the segment in
                __threadfence();
                asm volatile("bar.sync 1, 128;" ::: "memory");
                if (quad == 0 && lane == 0) atomicAdd(&p.sk_flags[tc.tile_id * 2 + (int)rank], 1u);
            }
            if (quad == 0 && lane == 0) { tr.end(10); EVT(5); }
        }
    }
    ptx::tc_fence_before();
    __syncthreads();
    if (p.streamk) {
        if (threadIdx.x == 0) tr.begin();
        // the activation ring is idle by now: its first bytes hold the slot list of the tile being summed
#ifdef RESQ_TIMELINE
        streamk_fixup<TN>(p, pair, (int)rank, abort_flag, reinterpret_cast<volatile int*>(tmem_slot + 2),
                          reinterpret_cast<int*>(ring_a), tl ? p.timeline + 512 + (int)rank * 16 + 8 : nullptr, t_kernel0);
#else
        streamk_fixup<TN>(p, pair, (int)rank, abort_flag, reinterpret_cast<volatile int*>(tmem_slot + 2),
                          reinterpret_cast<int*>(ring_a), nullptr, 0);
#endif
        if (threadIdx.x == 0) { tr.end(13); EVT(7); }
    }
#ifdef RESQ_TIMELINE
    if (tl && threadIdx.x < 256) p.timeline[rank * 256 + threadIdx.x] = tlog[threadIdx.x];
#endif
    ptx::cluster_sync();  // no CTA leaves while the peer may still signal its barriers or read its shared memory
#ifdef RESQ_TIMELINE
    if (tr.out && threadIdx.x == 0) {
        atomicAdd(tr.out + 11, (unsigned long long)(clock64() - t_kernel0));
        atomicAdd(tr.out + 12, 1ull);
    }
#endif
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc_pair(tmem_base, kTmemCols);
    }
}

std::atomic<int> g_expire_next_wait{0};

constexpr int kStreamKTN = 256;    // tile width of the K-streamed schedule (two accumulators fit in tensor memory)
constexpr int kStreamKMaxPairs = 74;

// Tensor maps of one problem: activation image, residual operand (dense image, or compressed image + index metadata),
// weights (packed codes, or plain bf16 rows).
template <int RES, int TN, int FMT>
int make_problem_maps(const GemmArgs& g, CUtensorMap* ta, CUtensorMap* tr, CUtensorMap* te, CUtensorMap* tw) {
    constexpr int nt = TN > kMaxBN ? 2 : 1;
    constexpr int half = TN / nt / 2;
    int rc = make_tmap_2d(ta, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, g.a_bf16, (uint64_t)g.K, (uint64_t)g.M, (uint64_t)(g.lda ? g.lda : g.K) * 2,
                          kBK, kBM, CU_TENSOR_MAP_SWIZZLE_128B);
    if (rc) return rc;
    if (RES == kResSparse24) {
        // compressed residual image [M, K/2] in boxes of 32 values x 128 rows (64-byte rows, 64-byte swizzle) and its
        // metadata blocks (2 KB per 128 rows x 128 K positions) as rows of 256 bytes
        rc = make_tmap_2d(tr, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, g.r_comp, (uint64_t)g.K / 2, (uint64_t)g.M, (uint64_t)g.K,
                          kBK / 2, kBM, CU_TENSOR_MAP_SWIZZLE_64B);
        if (rc) return rc;
        rc = make_tmap_2d(te, CU_TENSOR_MAP_DATA_TYPE_UINT8, g.r_meta, 256, (uint64_t)g.meta_rows128 * (uint64_t)g.meta_ka * 8, 256,
                          256, 8, CU_TENSOR_MAP_SWIZZLE_NONE);
    } else {
        rc = make_tmap_2d(tr, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, RES == kResDense ? g.r_bf16 : g.a_bf16, (uint64_t)g.K, (uint64_t)g.M,
                          (uint64_t)(g.lda ? g.lda : g.K) * 2, kBK, kBM, CU_TENSOR_MAP_SWIZZLE_128B);
        *te = *ta;
        if (RES == kResDense && g.blk_flags && !rc)  // the same image in boxes of 32 rows (one block of the selection)
            rc = make_tmap_2d(te, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, g.r_bf16, (uint64_t)g.K, (uint64_t)g.M,
                              (uint64_t)(g.lda ? g.lda : g.K) * 2, kBK, 32, CU_TENSOR_MAP_SWIZZLE_128B);
    }
    if (rc) return rc;
    if (FMT == kPlainW)
        return make_tmap_2d(tw, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, g.w_bf16, (uint64_t)g.K, (uint64_t)g.N, (uint64_t)g.ldw * 2, kBK,
                            (uint32_t)half, CU_TENSOR_MAP_SWIZZLE_128B);
    return make_tmap_2d(tw, CU_TENSOR_MAP_DATA_TYPE_UINT8, g.w_codes, (uint64_t)g.K / 2, (uint64_t)g.N, (uint64_t)g.K / 2,
                        kBK / 2, (uint32_t)half, CU_TENSOR_MAP_SWIZZLE_NONE);
}

template <int TN>
void fill_problem(PairProblem& pb, const GemmArgs& g) {
    pb.w_side = g.w_side;
    pb.Y = g.Y;
    pb.ldy = g.ldy;
    pb.M = (int)g.M;
    pb.N = (int)g.N;
    pb.G = (int)(g.K / kBK);
    pb.ntiles_n = (int)((g.N + TN - 1) / TN);
    pb.tile_base = 0;
    pb.dealt_first = 0;
    pb.unit_base = 0;
    pb.meta_ka = (int)g.meta_ka;
    pb.blk_flags = g.r_bf16 ? g.blk_flags : nullptr;
}

// Ring depths from the shared-memory budget.  Ring slots: a multiple of the number of expander groups (group g works
// on the slots s = g mod NG, so a slot is only ever written by one group).  With one slot per group the group's
// expansion of a k-block and the MMAs that read its previous k-block alternate; with two slots per group they
// overlap.  `kb_per_pair`: k-blocks a pair walks in a row (a deeper ring only pays once the pipeline is in steady state).
template <int RES, int TN, int FMT, int NG, int NP>
int pick_rings(PairParams<NP>& p, int64_t kb_per_pair, int* smem_bytes) {
    constexpr int kExpGroups = NG;
    constexpr int kAStage = a_stage_bytes(RES);
    constexpr int nt = TN > kMaxBN ? 2 : 1;
    constexpr int my_rows = nt * (TN / nt / 2);
    constexpr int exp_stage = my_rows * 128, raw_stage = FMT == kPlainW ? 0 : my_rows * 32;  // (the kernel's raw ring is unused then)
    const int fixed = 1024 + 1024;
    const int slot_bytes = kAStage + exp_stage + raw_stage;
    int per_group = (fixed + 2 * kExpGroups * slot_bytes <= kSmemBudget) ? 2 : 1;
    per_group = std::max(1, std::min(per_group, env_int("RESQ_GEMM_SLOTS_PER_GROUP", 2)));
    p.se = p.sr = p.sa = kExpGroups * per_group;
    // If two full slots per group do not fit, two expanded-weight slots per group with shallower activation and
    // raw-code rings may: what matters is that a group can expand its next k-block while the MMAs still read
    // its previous one.
    if (per_group == 1 && kb_per_pair >= 8 && env_int("RESQ_GEMM_DEEP_E", 1)) {
        // three activation slots cover the latency of their loads, one raw-code slot per group is enough, and
        // the rest goes to expanded-weight slots (any number: a k-block's barrier slot is k-block mod SE)
        // (the 512-wide tile with a dense residual operand fits a fourth expanded-weight slot only next to two activation
        // slots: measured 2 % faster there, slower everywhere else)
        const int sa2 = env_int("RESQ_GEMM_MIN_SA", (RES == kResDense && TN == 512) ? 2 : 3), sr2 = std::max(kExpGroups, std::min(env_int("RESQ_GEMM_MIN_SR", kExpGroups), kMaxRing));
        const int left = kSmemBudget - fixed - sa2 * kAStage - sr2 * raw_stage;
        const int se2 = std::min(std::min(left / exp_stage, 2 * kExpGroups), kMaxRing);
        if (se2 > kExpGroups) {
            p.se = se2;
            p.sr = sr2;
            p.sa = sa2;
            // what is left over deepens the activation ring (its loads have ~2000 cycles of latency to cover)
            while (p.sa < p.se && fixed + (p.sa + 1) * kAStage + p.se * exp_stage + p.sr * raw_stage <= kSmemBudget) ++p.sa;
        }
    }
    if (p.sa > kMaxRing || fixed + p.sa * kAStage + p.se * exp_stage + p.sr * raw_stage > kSmemBudget) {
        set_last_error("internal: shared-memory rings do not fit (pair tile %d)", TN);
        return RESQ_ERR_CUDA;
    }
    *smem_bytes = fixed + p.sa * kAStage + p.se * exp_stage + p.sr * raw_stage;
    return RESQ_OK;
}

template <int NG>
void pair_launch_config(cudaLaunchConfig_t& cfg, cudaLaunchAttribute (&attr)[2], int npairs, int smem_bytes, cudaStream_t stream) {
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3((unsigned)(2 * npairs), 1, 1);
    cfg.blockDim = dim3(pair_threads(NG), 1, 1);
    cfg.dynamicSmemBytes = (size_t)smem_bytes;
    cfg.stream = stream;
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl_enabled() ? 2 : 1;
}

template <int NP>
void common_params(PairParams<NP>& p, const GemmArgs& g, bool streamk) {
    p.streamk = streamk ? 1 : 0;
    p.dp_tiles = 0;
    p.sk_first = 0;
    p.sk_hi = 0;
    p.sk_pairs = 0;
    p.sk_units = 0;
    p.sk_slots = g.splitk_partials;
    p.sk_flags = g.sk_flags;
    p.sk_poll_limit = 1 << 20;
    p.sk_extra = 0;
    if (streamk && g_expire_next_wait.exchange(0)) {  // test hook: this launch's wait for the segments cannot be met
        p.sk_poll_limit = 1 << 12;
        p.sk_extra = 1;
    }
    p.out_f32 = g.out_dtype == RESQ_OUT_F32;
    p.partials = g.splitk_partials;
    p.status = g.status;
#ifdef RESQ_TIMELINE
    p.debug = env_int("RESQ_GEMM_DEBUG", 0);
    {
        const char* tp = getenv("RESQ_GEMM_TIMELINE_PTR");
        p.timeline = tp && *tp ? reinterpret_cast<unsigned int*>(strtoull(tp, nullptr, 0)) : nullptr;
        p.timeline_first = env_int("RESQ_GEMM_TIMELINE_FIRST", 96);
        p.timeline_pair = env_int("RESQ_GEMM_TIMELINE_PAIR", 0);
    }
#endif
}

template <int RES, int TN, int FMT, int NG>
int launch_pair_variant(const GemmArgs& g, int splits, cudaStream_t stream, bool streamk = false) {
    PairMaps<1> maps;
    int rc = make_problem_maps<RES, TN, FMT>(g, &maps.a[0], &maps.r[0], &maps.e[0], &maps.w[0]);
    if (rc) return rc;
    PairParams<1> p;
    memset(&p, 0, sizeof(p));
    p.nprob = 1;
    fill_problem<TN>(p.pr[0], g);
    const int G = p.pr[0].G;
    p.splits = splits;
    p.kblocks_per_split = (G + splits - 1) / splits;
    const int ntiles_m = (int)((g.M + 2 * kBM - 1) / (2 * kBM));
    p.num_tiles = ntiles_m * p.pr[0].ntiles_n * splits;
    if (g.tile_limit > 0 && !streamk) p.num_tiles = std::min(p.num_tiles, g.tile_limit * splits);
    p.acc_bufs = TN * 2 <= (RES == kResSparse24 ? kSpTmemCol : kTmemCols) ? 2 : 1;
    if (RES == kResSparse24 && TN > kSpTmemCol) {
        set_last_error("internal: no tensor-memory columns left for the sparse metadata (pair tile %d)", TN);
        return RESQ_ERR_CUDA;
    }
    common_params(p, g, streamk);
    auto kern = gemm_pair_kernel<RES, TN, FMT, NG, 1>;
    rc = ensure_dynamic_smem(reinterpret_cast<const void*>(kern), kSmemBudget, "cudaFuncSetAttribute(gemm pair)");
    if (rc) return rc;
    const int max_pairs = device_sm_count() / 2;
    int npairs = std::min(p.num_tiles, max_pairs);
    if (streamk) {
        // every pair gets at least two k-blocks; the pairs wait for one another at the end, so all of them
        // must be resident at once
        const int64_t units = (int64_t)p.num_tiles * G;
        const int cap = std::min(max_pairs, kStreamKMaxPairs);
        npairs = (int)std::min<int64_t>(cap, std::max<int64_t>(1, units / 2));
        // Few tiles: the same number of pairs for every tile, so that a pair works on one tile only -- unless that
        // leaves more than 15 % of the pairs idle on long K ranges (measured: 18944 -> 3584 at M = 512, 28 tiles:
        // 154 -> 134 us with the units dealt out evenly; short K ranges lose more in the second partial tile).
        const int per_tile_aligned = std::max(1, std::min(cap / std::max(1, p.num_tiles), G / 2));
        const bool idle_pairs = p.num_tiles * per_tile_aligned * 100 < cap * 85 && units / cap >= 64;
        const int force_unaligned = env_int("RESQ_GEMM_SK_UNALIGNED", -1);  // debugging override
        if (p.num_tiles <= cap && !(force_unaligned >= 0 ? force_unaligned != 0 : idle_pairs)) {
            int per_tile = std::max(1, std::min(cap / p.num_tiles, G / 2));
            const int forced = env_int("RESQ_GEMM_SK_PAIRS", 0);  // debugging override: pairs per tile
            if (forced > 0) per_tile = std::max(1, std::min(forced, per_tile));
            npairs = p.num_tiles * per_tile;
        }
    }
    const int64_t kb_per_pair = streamk ? ((int64_t)p.num_tiles * G + npairs - 1) / npairs : p.kblocks_per_split;
    int smem_bytes = 0;
    rc = pick_rings<RES, TN, FMT, NG>(p, kb_per_pair, &smem_bytes);
    if (rc) return rc;
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[2];
    pair_launch_config<NG>(cfg, attr, npairs, smem_bytes, stream);
    cudaError_t e;
    if (streamk) {
        int max_clusters = 0;  // co-resident clusters of this variant with this much shared memory
        rc = max_active_clusters(reinterpret_cast<const void*>(kern), &cfg, &max_clusters);
        if (rc) return rc;
        if (npairs > max_clusters) {
            npairs = max_clusters;
            cfg.gridDim = dim3((unsigned)(2 * npairs), 1, 1);
        }
        if (npairs < 1) {
            set_last_error("gemm pair kernel: no cluster of two CTAs fits on this device");
            return RESQ_ERR_CUDA;
        }
        // more tiles than pairs: whole rounds of tiles first, only the last, incomplete round is dealt out by k-blocks
        if (p.num_tiles > npairs) p.dp_tiles = (p.num_tiles / npairs) * npairs;
        const int dealt_tiles = p.num_tiles - p.dp_tiles;
        p.pr[0].dealt_first = p.dp_tiles;
        p.sk_units = (int64_t)dealt_tiles * G;
        p.sk_pairs = (int)std::max<int64_t>(1, std::min<int64_t>(npairs, p.sk_units / 2));
        if ((size_t)dealt_tiles * 2 * sizeof(unsigned int) > kWsFlags) {
            set_last_error("internal: %d dealt tiles exceed the arrival counters of the K-streamed schedule", dealt_tiles);
            return RESQ_ERR_CUDA;
        }
    }
    {
        LaunchScope scope(kKindGemm, stream);
        e = cudaLaunchKernelEx(&cfg, kern, maps, p);
    }
    if (e != cudaSuccess) return cuda_fail(e, "gemm_pair_kernel launch");
    if (streamk) return RESQ_OK;
    return launch_splitk_reduce(g, splits, stream);
}

// ---- a group of independent problems in one launch ----------------------------------------------------------
// The tiles of all problems (256 x 256) form one list; the launch walks it with the K-streamed schedule.  Which
// tiles are computed whole and which are dealt out by k-blocks is chosen here, by simulating the candidates:
// a pair's time is its k-blocks plus a fixed cost per partial tile it writes and helps to sum.
struct GroupPlan {
    int order[kMaxGroup];   // problems in the order of the tile list (ascending K: whole tiles first)
    int dp_tiles, sk_first, sk_hi, sk_pairs;
    int64_t sk_units;
    double cost;
};

GroupPlan plan_group(const GemmArgs* g, int count, int npairs) {
    constexpr double kPartialCost = 10.0;  // a partial tile (fp32 write, wait, share of the sum) in k-block periods
    GroupPlan best;
    memset(&best, 0, sizeof(best));
    best.cost = 1e300;
    int order[kMaxGroup];
    for (int i = 0; i < count; ++i) order[i] = i;
    std::stable_sort(order, order + count, [&](int a, int b) { return g[a].K < g[b].K; });
    int T[kMaxGroup], G[kMaxGroup], base[kMaxGroup + 1];
    base[0] = 0;
    for (int i = 0; i < count; ++i) {
        const GemmArgs& a = g[order[i]];
        T[i] = (int)(((a.M + 2 * kBM - 1) / (2 * kBM)) * ((a.N + kStreamKTN - 1) / kStreamKTN));
        G[i] = (int)(a.K / kBK);
        base[i + 1] = base[i] + T[i];
    }
    const int total = base[count];
    auto g_of_tile = [&](int t) { int q = 0; while (q + 1 < count && t >= base[q + 1]) ++q; return G[q]; };
    // candidates for the number of whole tiles: the problem boundaries, and each rounded down to whole rounds
    int cand[2 * kMaxGroup + 2], nc = 0;
    for (int i = 0; i <= count; ++i) {
        cand[nc++] = base[i];
        cand[nc++] = base[i] / npairs * npairs;
    }
    // debugging overrides (tests reach both classes of ranges with them): the number of whole tiles and the units of
    // the pairs that hold one whole tile more
    const int force_dp = env_int("RESQ_GEMM_GROUP_DP", -1), force_hi = env_int("RESQ_GEMM_GROUP_HI", -1);
    if (force_dp >= 0 && force_dp <= total) {
        cand[0] = force_dp;
        nc = 1;
    }
    std::vector<double> whole((size_t)npairs);
    for (int ci = 0; ci < nc; ++ci) {
        const int dp = cand[ci];
        if ((size_t)(total - dp) * 2 * sizeof(unsigned int) > kWsFlags) continue;  // an arrival counter per dealt tile and rank
        std::fill(whole.begin(), whole.end(), 0.0);
        for (int t = 0; t < dp; ++t) whole[(size_t)(t % npairs)] += g_of_tile(t);
        int64_t D = 0;
        for (int t = dp; t < total; ++t) D += g_of_tile(t);
        const int b = dp % npairs;
        // units per pair of the first b pairs (which hold one whole tile more): balance the two classes
        for (int pass = 0; pass < 2; ++pass) {
            int H = 0;
            if (pass == 1) {
                if (b == 0 || D == 0) break;
                const double extra = whole[0] - whole[(size_t)(npairs - 1)];
                const double h = ((double)D - extra * (npairs - b)) / npairs;  // H with equal loads
                H = force_hi >= 0 ? force_hi : (int)h;
                if (H < 4) break;
            }
            const int64_t rest = D - (int64_t)b * H;
            int sk_pairs = b == npairs ? 0 : npairs - b;
            if (D > 0) {
                if (sk_pairs == 0 || rest < 0) continue;
                sk_pairs = (int)std::max<int64_t>(1, std::min<int64_t>(sk_pairs, rest / 2));
                if (rest == 0) continue;
            }
            // simulate: dealt ranges and the partial tiles they cut
            double worst = 0.0;
            auto beg = [&](int q) -> int64_t {
                if (q < b) return (int64_t)q * H;
                if (q >= b + sk_pairs) return D;
                return (int64_t)b * H + (int64_t)(q - b) * rest / sk_pairs;
            };
            // tile boundaries of the dealt units (prefix sums)
            std::vector<int64_t> tb;
            tb.push_back(0);
            for (int t = dp; t < total; ++t) tb.push_back(tb.back() + g_of_tile(t));
            for (int q = 0; q < npairs; ++q) {
                double c = whole[(size_t)q];
                if (D > 0) {
                    const int64_t u0 = beg(q), u1 = beg(q + 1);
                    if (u1 > u0) {
                        c += (double)(u1 - u0);
                        const bool cut0 = !std::binary_search(tb.begin(), tb.end(), u0);
                        const bool cut1 = !std::binary_search(tb.begin(), tb.end(), u1);
                        // first and last tile of the range: partial if the range cuts them
                        const auto i0 = std::upper_bound(tb.begin(), tb.end(), u0) - tb.begin() - 1;
                        const auto i1 = std::upper_bound(tb.begin(), tb.end(), u1 - 1) - tb.begin() - 1;
                        int partial = 0;
                        if (i0 == i1) partial = (cut0 || cut1) ? 1 : 0;
                        else partial = (cut0 ? 1 : 0) + (cut1 ? 1 : 0);
                        c += kPartialCost * partial;
                    }
                }
                worst = std::max(worst, c);
            }
            if (force_hi >= 0 && pass == 1) worst = 0.0;  // (forced)
            // (at equal cost the plan with more whole tiles wins: less partial-tile traffic)
            if (worst < best.cost || (worst == best.cost && dp > best.dp_tiles)) {
                best.cost = worst;
                best.dp_tiles = dp;
                best.sk_first = D > 0 ? b : 0;
                best.sk_hi = H;
                best.sk_pairs = D > 0 ? sk_pairs : 0;
                best.sk_units = D;
            }
        }
    }
    for (int i = 0; i < count; ++i) best.order[i] = order[i];
    return best;
}

template <int RES, int FMT, int NG>
int launch_pair_group(const GemmArgs* g, int count, cudaStream_t stream) {
    constexpr int TN = kStreamKTN, NP = kMaxGroup;
    if (count < 1 || count > kMaxGroup) {
        set_last_error("a group holds 1 to %d problems (got %d)", kMaxGroup, count);
        return RESQ_ERR_SHAPE;
    }
    auto kern = gemm_pair_kernel<RES, TN, FMT, NG, NP>;
    int rc = ensure_dynamic_smem(reinterpret_cast<const void*>(kern), kSmemBudget, "cudaFuncSetAttribute(gemm pair group)");
    if (rc) return rc;
    PairParams<NP> p;
    memset(&p, 0, sizeof(p));
    int64_t units = 0;
    for (int i = 0; i < count; ++i)
        units += ((g[i].M + 2 * kBM - 1) / (2 * kBM)) * ((g[i].N + TN - 1) / TN) * (g[i].K / kBK);
    p.splits = 1;
    p.acc_bufs = 2;
    common_params(p, g[0], true);
    int npairs = (int)std::min<int64_t>(std::min(device_sm_count() / 2, kStreamKMaxPairs), std::max<int64_t>(1, units / 2));
    int smem_bytes = 0;
    rc = pick_rings<RES, TN, FMT, NG>(p, (units + npairs - 1) / npairs, &smem_bytes);
    if (rc) return rc;
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[2];
    pair_launch_config<NG>(cfg, attr, npairs, smem_bytes, stream);
    int max_clusters = 0;  // the pairs wait for one another at the end: all of them must be resident at once
    rc = max_active_clusters(reinterpret_cast<const void*>(kern), &cfg, &max_clusters);
    if (rc) return rc;
    if (npairs > max_clusters) {
        npairs = max_clusters;
        cfg.gridDim = dim3((unsigned)(2 * npairs), 1, 1);
    }
    if (npairs < 1) {
        set_last_error("gemm pair kernel: no cluster of two CTAs fits on this device");
        return RESQ_ERR_CUDA;
    }
    const GroupPlan plan = plan_group(g, count, npairs);
    if (plan.cost >= 1e300) {
        set_last_error("gemm pair group: no schedule fits the arrival counters (too many output tiles with long K)");
        return RESQ_ERR_SHAPE;
    }
    PairMaps<NP> maps;
    memset(&maps, 0, sizeof(maps));
    p.nprob = count;
    int tile_base = 0;
    int64_t unit_base = 0;
    for (int i = 0; i < count; ++i) {
        const GemmArgs& a = g[plan.order[i]];
        rc = make_problem_maps<RES, TN, FMT>(a, &maps.a[i], &maps.r[i], &maps.e[i], &maps.w[i]);
        if (rc) return rc;
        fill_problem<TN>(p.pr[i], a);
        const int tiles = (int)((a.M + 2 * kBM - 1) / (2 * kBM)) * p.pr[i].ntiles_n;
        p.pr[i].tile_base = tile_base;
        p.pr[i].dealt_first = std::min(std::max(tile_base, plan.dp_tiles), tile_base + tiles);
        p.pr[i].unit_base = unit_base;
        unit_base += (int64_t)(tile_base + tiles - p.pr[i].dealt_first) * p.pr[i].G;
        tile_base += tiles;
    }
    for (int i = count; i < NP; ++i) {  // unused entries: never matched by the lookups
        maps.a[i] = maps.a[0];
        maps.r[i] = maps.r[0];
        maps.e[i] = maps.e[0];
        maps.w[i] = maps.w[0];
        p.pr[i] = p.pr[count - 1];
        p.pr[i].tile_base = tile_base;
        p.pr[i].dealt_first = tile_base;
        p.pr[i].unit_base = unit_base;
    }
    p.num_tiles = tile_base;
    p.dp_tiles = plan.dp_tiles;
    p.sk_first = plan.sk_first;
    p.sk_hi = plan.sk_hi;
    p.sk_pairs = plan.sk_pairs;
    p.sk_units = plan.sk_units;
    if (unit_base != plan.sk_units) {
        set_last_error("internal: group schedule is inconsistent (%lld dealt units planned, %lld laid out)", (long long)plan.sk_units,
                       (long long)unit_base);
        return RESQ_ERR_CUDA;
    }
    if ((size_t)(p.num_tiles - p.dp_tiles) * 2 * sizeof(unsigned int) > kWsFlags) {
        set_last_error("internal: %d dealt tiles exceed the arrival counters of the K-streamed schedule", p.num_tiles - p.dp_tiles);
        return RESQ_ERR_CUDA;
    }
    if (env_int("RESQ_GEMM_DEBUG", 0) & 1)
        fprintf(stderr, "resq gemm group: %d problems, %d tiles, %d pairs: %d whole tiles, %lld dealt units (first %d pairs take %d each, %d pairs share the rest)\n",
                count, p.num_tiles, npairs, p.dp_tiles, (long long)p.sk_units, p.sk_first, p.sk_hi, p.sk_pairs);
    cudaError_t e;
    {
        LaunchScope scope(kKindGemm, stream);
        e = cudaLaunchKernelEx(&cfg, kern, maps, p);
    }
    return e == cudaSuccess ? RESQ_OK : cuda_fail(e, "gemm_pair_kernel (group) launch");
}

template <int RES, int FMT>
int dispatch_pair(const GemmArgs& g, int tn, int splits, cudaStream_t stream) {
    const int ng = env_int("RESQ_GEMM_GROUPS", 3);
    if (tn == 128) return launch_pair_variant<RES, 128, FMT, 4>(g, splits, stream);
    if (tn == 256 && ng == 3) return launch_pair_variant<RES, 256, FMT, 3>(g, splits, stream);
    if (tn == 256) return launch_pair_variant<RES, 256, FMT, 4>(g, splits, stream);
    if (tn == 320) return launch_pair_variant<RES, 320, FMT, 3>(g, splits, stream);
    if (tn == 384) return launch_pair_variant<RES, 384, FMT, 3>(g, splits, stream);
    if constexpr (RES != kResSparse24) {  // 512 accumulator columns leave none for the sparse metadata
        if (tn == 512) return launch_pair_variant<RES, 512, FMT, 3>(g, splits, stream);  // four slots would not fit
    } else {
        if (tn == 480) return launch_pair_variant<RES, 480, FMT, 3>(g, splits, stream);
    }
    set_last_error("internal: unsupported pair tile width %d", tn);
    return RESQ_ERR_CUDA;
}

}  // namespace

void debug_expire_next_wait(int on) { g_expire_next_wait.store(on ? 1 : 0); }

size_t gemm_pair_streamk_scratch_bytes() {
    return (size_t)2 * kStreamKMaxPairs * (2 * kBM) * kStreamKTN * sizeof(float);
}

namespace {
int res_mode(const GemmArgs& g) { return g.r_comp ? kResSparse24 : g.r_bf16 ? kResDense : kResNone; }
template <int FMT>
int streamk_fmt(const GemmArgs& g, cudaStream_t stream) {
    // Four expander groups (768 threads, 80 registers) once a pair walks a dozen k-blocks or more: long runs are bound by
    // the expanders' latency per k-block (M = 512, 7B shapes: step 494 -> 476 us; 3B down projection at M = 256: 49.3 ->
    // 47.9 us), short ones lose a microsecond to the larger CTA (qkv at M = 256: 27.9 -> 29.0 us).
    const int64_t units = ((g.M + 2 * kBM - 1) / (2 * kBM)) * ((g.N + kStreamKTN - 1) / kStreamKTN) * (g.K / kBK);
    if (env_int("RESQ_GEMM_SK_GROUPS", units / kStreamKMaxPairs >= 12 ? 4 : 3) == 4) {
        switch (res_mode(g)) {
            case kResSparse24: return launch_pair_variant<kResSparse24, kStreamKTN, FMT, 4>(g, 1, stream, true);
            case kResDense: return launch_pair_variant<kResDense, kStreamKTN, FMT, 4>(g, 1, stream, true);
            default: return launch_pair_variant<kResNone, kStreamKTN, FMT, 4>(g, 1, stream, true);
        }
    }
    switch (res_mode(g)) {
        case kResSparse24: return launch_pair_variant<kResSparse24, kStreamKTN, FMT, 3>(g, 1, stream, true);
        case kResDense: return launch_pair_variant<kResDense, kStreamKTN, FMT, 3>(g, 1, stream, true);
        default: return launch_pair_variant<kResNone, kStreamKTN, FMT, 3>(g, 1, stream, true);
    }
}
template <int FMT>
int group_fmt(const GemmArgs* g, int count, cudaStream_t stream) {
    // four expander groups (768 threads, 80 registers): the long k-block runs of a group are bound by the expanders'
    // latency per k-block, and a fourth group shortens the period (config 1 step 98.4 -> 93.4 us); RESQ_GEMM_GROUPS=3
    // is the debugging override
    const bool four = env_int("RESQ_GEMM_GROUPS", 4) == 4;
    switch (res_mode(g[0])) {
        case kResSparse24:
            set_last_error("internal: a group takes the dense residual image");
            return RESQ_ERR_CUDA;
        case kResDense: return four ? launch_pair_group<kResDense, FMT, 4>(g, count, stream) : launch_pair_group<kResDense, FMT, 3>(g, count, stream);
        default: return four ? launch_pair_group<kResNone, FMT, 4>(g, count, stream) : launch_pair_group<kResNone, FMT, 3>(g, count, stream);
    }
}
template <int FMT>
int pair_fmt(const GemmArgs& g, int tn, int splits, cudaStream_t stream) {
    switch (res_mode(g)) {
        case kResSparse24: return dispatch_pair<kResSparse24, FMT>(g, tn, splits, stream);
        case kResDense: return dispatch_pair<kResDense, FMT>(g, tn, splits, stream);
        default: return dispatch_pair<kResNone, FMT>(g, tn, splits, stream);
    }
}
}  // namespace

// bf16 weights (no expansion): 256-wide tiles on the K-streamed schedule or for small problems, else 512-wide.
int launch_gemm_pair_plainw(const GemmArgs& g, int tn, int splits, bool streamk, cudaStream_t stream) {
    const int mode = res_mode(g);
    if (mode == kResSparse24) {
        set_last_error("internal: the bf16-weight GEMM takes the dense residual image");
        return RESQ_ERR_CUDA;
    }
    if (streamk || tn <= 256)
        return mode == kResDense ? launch_pair_variant<kResDense, 256, kPlainW, 3>(g, splits, stream, streamk)
                                 : launch_pair_variant<kResNone, 256, kPlainW, 3>(g, splits, stream, streamk);
    return mode == kResDense ? launch_pair_variant<kResDense, 512, kPlainW, 3>(g, splits, stream)
                             : launch_pair_variant<kResNone, 512, kPlainW, 3>(g, splits, stream);
}

int launch_gemm_pair_streamk(const GemmArgs& g, cudaStream_t stream) {
    return g.fmt == kMXFP4 ? streamk_fmt<kMXFP4>(g, stream) : streamk_fmt<kHiF4>(g, stream);
}

// All problems share the weight format, the residual mode, the output type, the status word, the arrival counters and
// the partial-tile slots of g[0].
int launch_gemm_pair_group(const GemmArgs* g, int count, cudaStream_t stream) {
    for (int i = 1; i < count; ++i)
        if (g[i].fmt != g[0].fmt || res_mode(g[i]) != res_mode(g[0]) || g[i].out_dtype != g[0].out_dtype || g[i].w_bf16 || g[i].blk_flags) {
            set_last_error("internal: the problems of a group must share format, residual mode and output type");
            return RESQ_ERR_CUDA;
        }
    return g[0].fmt == kMXFP4 ? group_fmt<kMXFP4>(g, count, stream) : group_fmt<kHiF4>(g, count, stream);
}

int launch_gemm_pair(const GemmArgs& g, int tn, int splits, cudaStream_t stream) {
    return g.fmt == kMXFP4 ? pair_fmt<kMXFP4>(g, tn, splits, stream) : pair_fmt<kHiF4>(g, tn, splits, stream);
}

}  // namespace resq
