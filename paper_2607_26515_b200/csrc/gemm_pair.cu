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
#include <cstdlib>
#include <cstring>
#include <mutex>

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

struct PairParams {
    const void* w_side;
    int64_t M, N, K;
    int kblocks_per_split, splits;
    int ntiles_m, ntiles_n, num_tiles;
    int sa, sr, se, acc_bufs;
    int meta_ka;             // sparse residual: metadata blocks (128 K positions) per 128-row band
    void* Y;
    int out_f32;
    int64_t ldy;
    float* partials;
    DeviceStatus* status;
#ifdef RESQ_TIMELINE
    int debug;
    unsigned int* timeline;  // device buffer for a per-role event log of pair 0 (or null)
    int timeline_first;      // first k-block iteration that is logged
#endif
    // K-streamed schedule (streamk != 0): the num_tiles * G (tile, k-block) units are dealt out evenly to the
    // pairs; a pair's first and last segment may cover only part of a tile's K range and then go to fp32 slots
    int streamk;
    // With more tiles than pairs the first dp_tiles tiles (a multiple of the number of pairs) are computed whole,
    // one per pair and round, and written out directly; only the k-blocks of the remaining tiles are dealt out.
    int dp_tiles;
    int sk_pairs;            // pairs 0 .. sk_pairs-1 share the dealt-out units (at least two k-blocks each)
    float* sk_slots;         // [2 * npairs][256][TN] fp32: slot 2p = first segment of pair p, 2p + 1 = its last
    unsigned int* sk_flags;  // [num_tiles][2]: segments of the tile written, per CTA rank (zeroed before launch)
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
    int tile_id;   // K-streamed schedule: output tile of the segment
    int slot;      //   and where its fp32 partial goes
    bool partial;  // the segment does not cover the whole K range (or K is split): fp32 partial output
};

template <int TN>
__device__ __forceinline__ TileCoord decode_tile(const PairParams& p, int tile) {
    TileCoord t;
    t.split = tile % p.splits;
    const int rest = tile / p.splits;
    t.n0 = (int64_t)(rest % p.ntiles_n) * TN;
    t.m0 = (int64_t)(rest / p.ntiles_n) * (2 * kBM);
    const int G = (int)(p.K / kBK);
    t.kb_begin = t.split * p.kblocks_per_split;
    t.nkb = min(G, t.kb_begin + p.kblocks_per_split) - t.kb_begin;
    if (t.nkb < 0) t.nkb = 0;
    t.tile_id = rest;
    t.slot = 0;
    t.partial = p.splits > 1;
    return t;
}

// K-streamed schedule: pair q owns units [q * U / P, (q + 1) * U / P) of the U = num_tiles * G (tile, k-block)
// units, tile-major.
__device__ __forceinline__ int64_t sk_begin(int64_t U, int P, int q) { return (int64_t)q * U / P; }
__device__ __forceinline__ int sk_pair_of(int64_t U, int P, int64_t u) { return (int)((((u + 1) * P) - 1) / U); }

// Walks the work of one pair in the order every role of the kernel uses.
template <int TN>
struct SegIter {
    const PairParams& p;
    int pair, npairs, G;
    int tile;            // tile schedule: next tile
    int64_t u0, u, u1;   // K-streamed schedule: this pair's units
    __device__ SegIter(const PairParams& p_, int pair_, int npairs_) : p(p_), pair(pair_), npairs(npairs_) {
        G = (int)(p.K / kBK);
        tile = pair;
        if (p.streamk) {
            const int64_t U = (int64_t)(p.num_tiles - p.dp_tiles) * G;  // units of the tiles that are dealt out
            u0 = u = u1 = 0;
            if (pair < p.sk_pairs) {
                u0 = u = sk_begin(U, p.sk_pairs, pair);
                u1 = sk_begin(U, p.sk_pairs, pair + 1);
            }
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
            tc.tile_id = tile;
            tc.split = 0;
            tc.kb_begin = 0;
            tc.nkb = G;
            tc.n0 = (int64_t)(tile % p.ntiles_n) * TN;
            tc.m0 = (int64_t)(tile / p.ntiles_n) * (2 * kBM);
            tc.partial = false;
            tc.slot = 0;
            tile += npairs;
            return true;
        }
        if (u >= u1) return false;
        const int tr = (int)(u / G);     // among the tiles that are dealt out
        const int t = p.dp_tiles + tr;
        tc.tile_id = t;
        tc.split = 0;
        tc.kb_begin = (int)(u - (int64_t)tr * G);
        tc.nkb = (int)min((int64_t)(G - tc.kb_begin), u1 - u);
        tc.n0 = (int64_t)(t % p.ntiles_n) * TN;
        tc.m0 = (int64_t)(t / p.ntiles_n) * (2 * kBM);
        tc.partial = tc.nkb < G;
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
template <int TN>
__device__ __forceinline__ void streamk_fixup(const PairParams& p, int pair, int npairs, int rank, volatile int* abort_flag,
                                              volatile int* s_ok, int* s_slots, unsigned int* evt, long long t0) {
    const int G = (int)(p.K / kBK);
    const int64_t U = (int64_t)(p.num_tiles - p.dp_tiles) * G;
    if (pair >= p.sk_pairs) return;
    npairs = p.sk_pairs;  // the pairs that share the dealt-out units
    const int64_t u0 = sk_begin(U, npairs, pair), u1 = sk_begin(U, npairs, pair + 1);
    if (u1 <= u0) return;
    const int t_first = (int)(u0 / G), t_last = (int)((u1 - 1) / G);  // among the tiles that are dealt out
    for (int which = 0; which < 2; ++which) {
        const int tr = which == 0 ? t_first : t_last;
        if (which == 1 && t_last == t_first) break;
        const int t = p.dp_tiles + tr;  // output tile
        const int64_t tb = (int64_t)tr * G, te = tb + G;
        if (u0 <= tb && u1 >= te) continue;  // this pair computed the whole tile and wrote it out directly
        const int pf = sk_pair_of(U, npairs, tb), pl = sk_pair_of(U, npairs, te - 1);
        const int nseg = pl - pf + 1, j = pair - pf;
        if (threadIdx.x == 0) {
            int ok = *abort_flag ? 0 : 1;
            const unsigned int* flag = p.sk_flags + t * 2 + rank;
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
            const int q = pf + (int)threadIdx.x;
            s_slots[threadIdx.x] = 2 * q + (sk_begin(U, npairs, q) >= tb ? 0 : 1);
        }
        __syncthreads();
        // column slice j of nseg, in units of 4 columns
        const int c0 = (int)((int64_t)j * (TN / 4) / nseg) * 4, c1 = (int)((int64_t)(j + 1) * (TN / 4) / nseg) * 4;
        const int w4 = (c1 - c0) / 4;
        const int64_t m_base = (int64_t)(t / p.ntiles_n) * (2 * kBM) + rank * kBM;
        const int64_t n_base = (int64_t)(t % p.ntiles_n) * TN;
        for (int item = threadIdx.x; item < kBM * w4; item += (int)blockDim.x) {
            const int row = item / w4, c = c0 + (item % w4) * 4;
            const int64_t m = m_base + row, n = n_base + c;
            if (m >= p.M || n >= p.N) continue;
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
                float* dst = reinterpret_cast<float*>(p.Y) + m * p.ldy + n;
                if (n + 3 < p.N) *reinterpret_cast<float4*>(dst) = acc;
                else for (int e = 0; e < 4; ++e) if (n + e < p.N) dst[e] = o[e];
            } else {
                __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(p.Y) + m * p.ldy + n;
                if (n + 3 < p.N) {
                    __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y), hi = __floats2bfloat162_rn(acc.z, acc.w);
                    *reinterpret_cast<uint2*>(dst) = make_uint2(*reinterpret_cast<uint32_t*>(&lo), *reinterpret_cast<uint32_t*>(&hi));
                } else {
                    for (int e = 0; e < 4; ++e) if (n + e < p.N) dst[e] = __float2bfloat16_rn(o[e]);
                }
            }
        }
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
template <int RES, int TN, int FMT, int NG>
__global__ void __launch_bounds__(pair_threads(NG), 1)
gemm_pair_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_r,
                 const __grid_constant__ CUtensorMap tmap_e, const __grid_constant__ CUtensorMap tmap_w, const PairParams p) {
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
    const bool tl = p.timeline != nullptr && (blockIdx.x >> 1) == 0;
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
    const int G = (int)(p.K / kBK);

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
    Trace tr{(p.debug & 16) ? reinterpret_cast<unsigned long long*>(p.status) + 8 : nullptr, 0};
    const long long t_kernel0 = clock64();
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
            ptx::tma_prefetch_desc(&tmap_a);
            if (RES != kResNone) ptx::tma_prefetch_desc(&tmap_r);
            if (RES == kResSparse24) ptx::tma_prefetch_desc(&tmap_e);
            uint32_t it = 0;
            bool ok = true;
            SegIter<TN> si(p, pair, npairs);
            TileCoord tc;
            while (ok && si.next(tc)) {
                const int my_m = (int)(tc.m0 + rank * kBM);
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
                    ptx::tma_load_2d_pair(st, &tmap_a, full, kx, my_m);
                    if (RES == kResDense) ptx::tma_load_2d_pair(st + kATileBytes, &tmap_r, full, kx, my_m);
                    if (RES == kResSparse24) {
                        ptx::tma_load_2d_pair(st + kATileBytes, &tmap_r, full, kx / 2, my_m);
                        if (with_meta)  // rows of 256 bytes, eight per 128 x 128 block
                            ptx::tma_load_2d_pair(st + kATileBytes + kSpTileBytes, &tmap_e, full, 0,
                                                  ((my_m >> 7) * p.meta_ka + (kb >> 1)) * 8);
                    }
                }
            }
        }
    } else if (warp == 2) {
        // ------------------------------------------------------------------ raw weight-code producer (both CTAs)
        if (lane == 0) {
            ptx::tma_prefetch_desc(&tmap_w);
            uint32_t it = 0;
            bool ok = true;
            SegIter<TN> si(p, pair, npairs);
            TileCoord tc;
            while (ok && si.next(tc)) {
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
                            ptx::tma_load_2d_pair(ring_e + (size_t)se * exp_stage + (size_t)j * half * 128, &tmap_w, full,
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
                        ptx::tma_load_2d(ring_r + (size_t)s * raw_stage + (size_t)j * half * 32, &tmap_w, &r_full[s],
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
            SegIter<TN> si(p, pair, npairs);
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
        uint32_t it0 = 0;  // k-block counter at the start of the current tile
        bool ok = true;
        SegIter<TN> si(p, pair, npairs);
        TileCoord tc;
        while (ok && si.next(tc)) {
            // local row l (< my_rows) is weight row n0 + (l / half) * bn + rank * half + (l % half);
            // lane l owns the metadata of rows l and 32 + l of this warp's slice
            auto row_of = [&](int l) -> int64_t { return tc.n0 + (int64_t)(l / half) * bn + rank * half + (l % half); };
            const int64_t n_a = row_of(r_begin + lane);
            const int64_t n_b = row_of(r_begin + (rows_per_warp > 32 ? 32 + lane : lane));
            const bool ok_a = lane < rows_per_warp && n_a < p.N;
            const bool ok_b = rows_per_warp > 32 && n_b < p.N;
            auto load_side = [&](int64_t n, int kb) -> uint32_t {
                if (FMT == kHiF4) return ptx::ld_nc_u32(reinterpret_cast<const uint32_t*>(p.w_side) + n * G + kb);
                return ptx::ld_nc_u16(reinterpret_cast<const uint16_t*>(p.w_side) + n * G + kb);
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
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&r_empty[sr]);
#pragma unroll
                for (int q = 0; q < kIters; ++q) {
                    const int r = r_begin + q * 4 + sub_row;
                    const uint4 v = FMT == kHiF4 ? expand_hif4_chunk(cw[q], mw[q], chunk)
                                                 : expand_mxfp4_chunk(cw[q], (mw[q] >> (8 * (chunk >> 2))) & 255u);
                    *reinterpret_cast<uint4*>(bexp + r * 128 + ((chunk ^ (r & 7)) << 4)) = v;
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
        SegIter<TN> si(p, pair, npairs);
        TileCoord tc;
        while (si.next(tc)) {
            const int lt = local_tile++;
            if (tc.nkb == 0) continue;
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
            const bool warp_has_rows = tc.m0 + rank * kBM + quad * 32 < p.M;
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
                    if (m >= p.M) continue;
                    float* dst = p.sk_slots + ((size_t)tc.slot * (2 * kBM) + rank * kBM + quad * 32 + lane) * TN + cc * 32;
#pragma unroll
                    for (int j = 0; j < 32; j += 8)
                        ptx::st_global_v8(dst + j, v[j], v[j + 1], v[j + 2], v[j + 3], v[j + 4], v[j + 5], v[j + 6], v[j + 7]);
                    continue;
                }
                if (m >= p.M) continue;
                const int64_t nb = tc.n0 + cc * 32;
                const int64_t left = p.N - nb;
                if (left <= 0) continue;
                if (p.splits > 1) {
                    float* dst = p.partials + ((int64_t)tc.split * p.M + m) * p.N + nb;
                    if (left >= 32 && (reinterpret_cast<uintptr_t>(dst) & 31u) == 0) {
#pragma unroll
                        for (int j = 0; j < 32; j += 8)
                            ptx::st_global_v8(dst + j, v[j], v[j + 1], v[j + 2], v[j + 3], v[j + 4], v[j + 5], v[j + 6], v[j + 7]);
                    } else if (left >= 32 && (p.N & 3) == 0) {
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
                    __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(p.Y) + m * p.ldy + nb;
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
        streamk_fixup<TN>(p, pair, npairs, (int)rank, abort_flag, reinterpret_cast<volatile int*>(tmem_slot + 2),
                          reinterpret_cast<int*>(ring_a), tl ? p.timeline + 512 + (int)rank * 16 + 8 : nullptr, t_kernel0);
#else
        streamk_fixup<TN>(p, pair, npairs, (int)rank, abort_flag, reinterpret_cast<volatile int*>(tmem_slot + 2),
                          reinterpret_cast<int*>(ring_a), nullptr, 0);
#endif
        if (threadIdx.x == 0) { tr.end(13); EVT(7); }
    }
#ifdef RESQ_TIMELINE
    if (tl && threadIdx.x < 256) p.timeline[blockIdx.x * 256 + threadIdx.x] = tlog[threadIdx.x];
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

template <int RES, int TN, int FMT, int NG>
int launch_pair_variant(const GemmArgs& g, int splits, cudaStream_t stream, bool streamk = false) {
    constexpr int kExpGroups = NG;
    constexpr int kAStage = a_stage_bytes(RES);
    constexpr int nt = TN > kMaxBN ? 2 : 1;
    constexpr int bn = TN / nt;
    constexpr int half = bn / 2;
    constexpr int my_rows = nt * half;
    CUtensorMap ta, tr, te, tw;
    int rc = make_tmap_2d(&ta, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, g.a_bf16, (uint64_t)g.K, (uint64_t)g.M, (uint64_t)(g.lda ? g.lda : g.K) * 2,
                          kBK, kBM, CU_TENSOR_MAP_SWIZZLE_128B);
    if (rc) return rc;
    if (RES == kResSparse24) {
        // compressed residual image [M, K/2] in boxes of 32 values x 128 rows (64-byte rows, 64-byte swizzle) and its
        // metadata blocks (2 KB per 128 rows x 128 K positions) as rows of 256 bytes
        rc = make_tmap_2d(&tr, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, g.r_comp, (uint64_t)g.K / 2, (uint64_t)g.M, (uint64_t)g.K,
                          kBK / 2, kBM, CU_TENSOR_MAP_SWIZZLE_64B);
        if (rc) return rc;
        rc = make_tmap_2d(&te, CU_TENSOR_MAP_DATA_TYPE_UINT8, g.r_meta, 256, (uint64_t)g.meta_rows128 * (uint64_t)g.meta_ka * 8, 256,
                          256, 8, CU_TENSOR_MAP_SWIZZLE_NONE);
    } else {
        rc = make_tmap_2d(&tr, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, RES == kResDense ? g.r_bf16 : g.a_bf16, (uint64_t)g.K, (uint64_t)g.M,
                          (uint64_t)(g.lda ? g.lda : g.K) * 2, kBK, kBM, CU_TENSOR_MAP_SWIZZLE_128B);
        te = ta;
    }
    if (rc) return rc;
    if (FMT == kPlainW)
        rc = make_tmap_2d(&tw, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, g.w_bf16, (uint64_t)g.K, (uint64_t)g.N, (uint64_t)g.ldw * 2, kBK,
                          (uint32_t)half, CU_TENSOR_MAP_SWIZZLE_128B);
    else
        rc = make_tmap_2d(&tw, CU_TENSOR_MAP_DATA_TYPE_UINT8, g.w_codes, (uint64_t)g.K / 2, (uint64_t)g.N, (uint64_t)g.K / 2,
                          kBK / 2, (uint32_t)half, CU_TENSOR_MAP_SWIZZLE_NONE);
    if (rc) return rc;
    PairParams p;
    p.meta_ka = g.meta_ka;
    p.w_side = g.w_side;
    p.M = g.M;
    p.N = g.N;
    p.K = g.K;
    const int G = (int)(g.K / kBK);
    p.splits = splits;
    p.kblocks_per_split = (G + splits - 1) / splits;
    p.ntiles_m = (int)((g.M + 2 * kBM - 1) / (2 * kBM));
    p.ntiles_n = (int)((g.N + TN - 1) / TN);
    p.num_tiles = p.ntiles_m * p.ntiles_n * splits;
    if (g.tile_limit > 0 && !streamk) p.num_tiles = std::min(p.num_tiles, g.tile_limit * splits);
    p.acc_bufs = TN * 2 <= (RES == kResSparse24 ? kSpTmemCol : kTmemCols) ? 2 : 1;
    if (RES == kResSparse24 && TN > kSpTmemCol) {
        set_last_error("internal: no tensor-memory columns left for the sparse metadata (pair tile %d)", TN);
        return RESQ_ERR_CUDA;
    }
    p.streamk = streamk ? 1 : 0;
    p.dp_tiles = 0;
    p.sk_pairs = 0;
    p.sk_slots = g.splitk_partials;
    p.sk_flags = g.sk_flags;
    p.sk_poll_limit = 1 << 20;
    p.sk_extra = 0;
    if (streamk && g_expire_next_wait.exchange(0)) {  // test hook: this launch's wait for the segments cannot be met
        p.sk_poll_limit = 1 << 12;
        p.sk_extra = 1;
    }
    p.Y = g.Y;
    p.out_f32 = g.out_dtype == RESQ_OUT_F32;
    p.ldy = g.ldy;
    p.partials = g.splitk_partials;
    p.status = g.status;
#ifdef RESQ_TIMELINE
    p.debug = env_int("RESQ_GEMM_DEBUG", 0);
    {
        const char* tp = getenv("RESQ_GEMM_TIMELINE_PTR");
        p.timeline = tp && *tp ? reinterpret_cast<unsigned int*>(strtoull(tp, nullptr, 0)) : nullptr;
        p.timeline_first = env_int("RESQ_GEMM_TIMELINE_FIRST", 96);
    }
#endif
    auto kern = gemm_pair_kernel<RES, TN, FMT, NG>;
    rc = ensure_dynamic_smem(reinterpret_cast<const void*>(kern), kSmemBudget, "cudaFuncSetAttribute(gemm pair)");
    if (rc) return rc;
    const int max_pairs = device_sm_count() / 2;
    int npairs = std::min(p.num_tiles, max_pairs);
    if (streamk && (size_t)p.num_tiles * 2 * sizeof(unsigned int) > kWsFlags) {
        set_last_error("internal: %d output tiles exceed the arrival counters of the K-streamed schedule", p.num_tiles);
        return RESQ_ERR_CUDA;
    }
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
    constexpr int exp_stage = my_rows * 128, raw_stage = FMT == kPlainW ? 0 : my_rows * 32;  // (the kernel's raw ring is unused then)
    const int fixed = 1024 + 1024;
    // Ring slots: a multiple of the number of expander groups (group g works on the slots s = g mod NG, so a slot
    // is only ever written by one group).  With one slot per group the group's expansion of a k-block and the
    // MMAs that read its previous k-block alternate; with two slots per group they overlap.  All three rings have
    // the same depth (they share the slot's full / empty barriers).
    const int slot_bytes = kAStage + exp_stage + raw_stage;
    int per_group = (fixed + 2 * kExpGroups * slot_bytes <= kSmemBudget) ? 2 : 1;
    per_group = std::max(1, std::min(per_group, env_int("RESQ_GEMM_SLOTS_PER_GROUP", 2)));
    p.se = p.sr = p.sa = kExpGroups * per_group;
    // If two full slots per group do not fit, two expanded-weight slots per group with shallower activation and
    // raw-code rings may: what matters is that a group can expand its next k-block while the MMAs still read
    // its previous one.
    // (Not for a handful of k-blocks per pair: the deeper ring only pays once the pipeline is in steady state.)
    const int64_t kb_per_pair = streamk ? ((int64_t)p.num_tiles * G + npairs - 1) / npairs : p.kblocks_per_split;
    if (per_group == 1 && kb_per_pair >= 8 && env_int("RESQ_GEMM_DEEP_E", 1)) {
        // three activation slots cover the latency of their loads, one raw-code slot per group is enough, and
        // the rest goes to expanded-weight slots (any number: a k-block's barrier slot is k-block mod SE)
        const int sa2 = env_int("RESQ_GEMM_MIN_SA", 3), sr2 = std::max(kExpGroups, std::min(env_int("RESQ_GEMM_MIN_SR", kExpGroups), kMaxRing));
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
    const int smem_bytes = fixed + p.sa * kAStage + p.se * exp_stage + p.sr * raw_stage;
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3((unsigned)(2 * npairs), 1, 1);
    cfg.blockDim = dim3(pair_threads(NG), 1, 1);
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
        p.sk_pairs = (int)std::max<int64_t>(1, std::min<int64_t>(npairs, (int64_t)(p.num_tiles - p.dp_tiles) * G / 2));
    }
    {
        LaunchScope scope(kKindGemm, stream);
        e = cudaLaunchKernelEx(&cfg, kern, ta, tr, te, tw, p);
    }
    if (e != cudaSuccess) return cuda_fail(e, "gemm_pair_kernel launch");
    if (streamk) return RESQ_OK;
    return launch_splitk_reduce(g, splits, stream);
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
    switch (res_mode(g)) {
        case kResSparse24: return launch_pair_variant<kResSparse24, kStreamKTN, FMT, 3>(g, 1, stream, true);
        case kResDense: return launch_pair_variant<kResDense, kStreamKTN, FMT, 3>(g, 1, stream, true);
        default: return launch_pair_variant<kResNone, kStreamKTN, FMT, 3>(g, 1, stream, true);
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

int launch_gemm_pair(const GemmArgs& g, int tn, int splits, cudaStream_t stream) {
    return g.fmt == kMXFP4 ? pair_fmt<kMXFP4>(g, tn, splits, stream) : pair_fmt<kHiF4>(g, tn, splits, stream);
}

}  // namespace resq
