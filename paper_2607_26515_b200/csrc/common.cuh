// Shared declarations of the ResQ CUDA library (sm_100a).  Internal; the public contract is include/resq.h.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>
#include <string.h>
#include "../../include/resq.h"

namespace resq {

enum Format : int { kHiF4 = 0, kMXFP4 = 1 };

constexpr int kHif4Block = 64;
constexpr int kMxBlock = 32;
constexpr int kE6M2Bias = 48;      // S1 = (1 + Mn/4) * 2^(E - 48)
constexpr int kBlkRows = 32;       // S^{32x64}: 32 token rows ...
constexpr int kBlkCols = 64;       // ... by 64 channels
constexpr size_t kWsHeader = 256;  // status word + padding at the start of every workspace
constexpr size_t kWsFlags = 2048;  // linear-layer workspaces: arrival counters of the K-streamed GEMM, right after the header

// Device status word layout (first 16 bytes of the workspace).
struct DeviceStatus {
    int code;    // resq_status
    int where;   // which wait gave up (kernel-specific tag)
    int block;   // blockIdx.x of the reporter
    int pad;
};

void set_last_error(const char* fmt, ...);
int cuda_fail(cudaError_t e, const char* what);

// Debugging overrides (tile widths, schedules, kernel choices: the RESQ_* variables the tests use to reach every
// variant) are honoured only when RESQ_DEBUG is set to a non-zero value in the environment at the library's first
// call; otherwise no call reads the environment and every override has its default.
bool debug_overrides();
int env_int(const char* name, int dflt);       // the variable's integer value if overrides are on and it is set
bool env_is_zero(const char* name);            // overrides on and the variable starts with '0'

// Per-device facts the launchers need (looked up once per device, under a mutex).
int device_sm_count();                         // of the current device
// Opts `func` into `bytes` of dynamic shared memory on the current device (once per device and function).
int ensure_dynamic_smem(const void* func, int bytes, const char* what);
// cudaOccupancyMaxActiveClusters of `func` under `cfg`, cached per device, function and shared-memory size.
int max_active_clusters(const void* func, const cudaLaunchConfig_t* cfg, int* out);

// Argument checks shared by the entry points (api.cu).
int split_pattern(int* pattern, int* quarters, int* per_strip);  // strips RESQ_KEEP_QUARTERS / RESQ_BLOCK_PER_STRIP
int check_pattern(int base_pattern, int64_t M);
// Packed outputs are written with 32-bit stores (codes, HiF4 metadata) or 16-bit stores (MXFP4 scales): every
// non-null packed output must be 4-byte aligned, else RESQ_ERR_ALIGN.
int check_packed_outputs(const void* x_codes, const void* x_side, const void* r_codes, const void* r_side);

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Diagnostics (api.cu): every kernel launch of the library is counted; when profiling is enabled a
// pair of CUDA events brackets each launch on its stream so that per-kernel device time can be read.
enum KernelKind : int { kKindQuant = 0, kKindSelect = 1, kKindGemm = 2, kKindReduce = 3, kNumKinds = 4 };
struct LaunchScope {
    LaunchScope(int kind, cudaStream_t stream);
    ~LaunchScope();
    int kind_;
    cudaStream_t stream_;
    void* rec_;
};

// ---- programmatic dependent launch ----------------------------------------------------------------
// The kernels of one linear-layer call (and of consecutive calls on a stream) are launched with programmatic
// stream serialization: a kernel may be scheduled, and run its set-up, while its predecessor drains.  Every
// kernel launched this way executes pdl_wait() before it first touches global memory that an earlier kernel may
// have written (or may still read), and pdl_trigger() as early as it likes.
bool pdl_enabled();  // api.cu: environment switch RESQ_PDL (default on)
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                 Args... args) {
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = pdl_enabled() ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
}
#endif

// ---- quantizer launch description (quantize.cu) ------------------------------------------------
struct QuantArgs {
    const __nv_bfloat16* X;
    const __nv_bfloat16* X_up;  // non-null: fused producer, the input is bf16(SiLU(X) * X_up) (same M, K, ldx)
    // non-null: fused RMSNorm producer, the input is bf16((X * row_scale[m]) * gamma[k]); row_scale [M] fp32 is
    // written by the row kernel that launch_quantize runs first (1 / sqrt(mean(X^2) + eps))
    const __nv_bfloat16* gamma;
    float* row_scale;
    float eps;
    // rht != 0: randomized Hadamard pre-transform, the input is bf16((1/8) H64 (s * X)) per block of 64 channels,
    // bit j of rht_signs negates channel j of every block (K % 64 == 0)
    int rht;
    unsigned long long rht_signs;
    int64_t M, K, ldx;
    int pattern;            // resq_pattern (base value); RESQ_S_NONE => no residual work at all
    int keep_quarters;      // kept share of the selection in quarters: 1, 2 (the paper's 50 %; also for 0) or 3
    int per_strip;          // block pattern: select inside every strip of 32 rows instead of over the tensor
    // canonical packed outputs (any may be null)
    uint8_t* x_codes;
    void* x_side;           // u32 meta (HiF4) or u8 scale (MXFP4)
    uint8_t* r_codes;
    void* r_side;
    uint8_t* mask_bits;
    int mask_r_codes;       // nonzero: r_codes receives S(Q(dX)) (dropped codes zeroed) instead of the canonical Q(dX)
    // expanded operands for the GEMM (any may be null): exact bf16 images of deq Q(X) and S(deq Q(dX))
    __nv_bfloat16* a_bf16;  // [M, K]
    __nv_bfloat16* r_bf16;  // [M, K]
    // pattern 2:4 only, instead of r_bf16: the compressed image and its index metadata (see GemmArgs)
    __nv_bfloat16* r_comp;  // [M, K/2]
    uint8_t* r_meta;
    int64_t meta_rows128, meta_ka;
    // BLOCK only: leave r_bf16 unmasked (the GEMM takes the keep flags and loads zero tiles for the dropped blocks)
    int skip_image_mask;
    // scratch
    double* scores;         // CHAN50: [K]; BLOCK: [(M/32) * (K/64)]
    uint8_t* keep_flags;    // CHAN50: [K]; BLOCK: [(M/32) * (K/64)]
    // more than kSelGridMin scores: the selection runs as a few grid-wide kernels over 16-bit digits and needs a
    // histogram of 65536 counters plus a small state block (kSelGridScratch bytes); null: single-CTA selection
    uint32_t* sel_hist;
    DeviceStatus* status;
    // words at the start of the workspace (status, counters of the GEMM) that the first kernel of the call clears
    uint32_t* clear_words;
    int n_clear_words;
};

int launch_quantize(int fmt, const QuantArgs& a, cudaStream_t stream);
constexpr int kMaxQuantGroup = 8;  // problems per grouped launch (quantizer and GEMM alike)
int launch_quantize_group(int fmt, const QuantArgs* a, int count, cudaStream_t stream);
// "W4A8": the decoded bf16 image of MXFP8-E4M3 quantized activations (blocks of 32, E8M0 scale), for the GEMM
int launch_quantize_mxfp8_image(const __nv_bfloat16* X, int64_t M, int64_t K, int64_t ldx, __nv_bfloat16* img, uint32_t* clear_words,
                                int n_clear_words, cudaStream_t stream);
// dst [cols, rows] (row pitch ld_dst) = transpose of src [rows, cols] (row pitch ld_src)
int launch_transpose_bf16(const __nv_bfloat16* src, int64_t rows, int64_t cols, int64_t ld_src, __nv_bfloat16* dst, int64_t ld_dst,
                          cudaStream_t stream);
int launch_dequantize(int fmt, const uint8_t* codes, const void* side, int64_t rows, int64_t K, float* out,
                      cudaStream_t stream);
size_t quant_scratch_bytes(int64_t M, int64_t K, int pattern);  // scores + keep flags [+ histogram] (without header)
constexpr int64_t kSelGridMin = 24576;                         // selections with more scores than this use the grid-wide kernels
constexpr size_t kSelGridScratch = 65536 * 4 + 256;            // histogram + state

// ---- GEMM launch description (gemm_hif4.cu / gemm_mxfp4.cu) -------------------------------------
struct GemmArgs {
    int fmt;                       // kHiF4 or kMXFP4: how w_codes / w_side are decoded
    const __nv_bfloat16* a_bf16;   // [M, K] exact bf16 image of deq Q(X)
    const __nv_bfloat16* r_bf16;   // [M, K] masked residual image, or null (pattern NONE, or r_comp given)
    // 2:4 residual in compressed form for the structured-sparse MMA (CTA-pair kernel only), instead of r_bf16:
    const __nv_bfloat16* r_comp;   // [M, K/2] the two kept values of every four consecutive channels, in channel order
    const uint8_t* r_meta;         // index metadata, sparse24_meta_offset() layout: meta_rows128 x meta_ka blocks of 2 KB
    int64_t meta_rows128, meta_ka;
    // block-wise selection, with r_bf16 (CTA-pair kernel only): r_bf16 is the unmasked image of deq Q(dX) and
    // blk_flags [(M/32), K/64] says which blocks of 32 rows x 64 channels are kept (nonzero); the kernel loads a zero tile
    // in place of a dropped block
    const uint8_t* blk_flags;
    const uint8_t* w_codes;        // [N, K/2]
    const void* w_side;            // [N, K/64] u32 or [N, K/32] u8
    const __nv_bfloat16* w_bf16;   // instead of w_codes / w_side: plain bf16 weights [N, K], row pitch ldw ("W16A4")
    int64_t ldw;
    int64_t M, N, K;
    int64_t lda;                   // row pitch of a_bf16 / r_bf16 in elements (0: K, the workspace images)
    void* Y;
    int out_dtype;
    int64_t ldy;
    float* splitk_partials;        // fp32 scratch for partial tiles: [splits, M, N] slabs, or tile slots (K-streamed schedule)
    int splits;                    // slabs that fit in splitk_partials
    size_t partial_bytes;          // size of splitk_partials
    unsigned int* sk_flags;        // kWsFlags bytes of zeroed counters (K-streamed schedule)
    int tile_limit;                // > 0: whole-tile schedule of the pair kernel stops after this many output tiles
    DeviceStatus* status;
};
int launch_gemm_hif4(const GemmArgs& g, cudaStream_t stream);
// A group of independent problems (same format, residual mode and output type) as one launch of the CTA-pair kernel on
// the K-streamed schedule; status word, arrival counters and partial-tile slots are those of g[0] (gemm_pair.cu).
int launch_gemm_pair_group(const GemmArgs* g, int count, cudaStream_t stream);
size_t gemm_pair_streamk_scratch_bytes();
// Decode-sized calls (every M <= 64): one launch with the weights as the MMA's M dimension and the tokens as its N
// (gemm_decode.cu).  The problems share format, residual mode (none or the dense image), output type, and the status word,
// arrival counters (kWsFlags zeroed bytes) and partial-tile scratch of g[0].
bool gemm_decode_supported(const GemmArgs* g, int count);
int launch_gemm_decode(const GemmArgs* g, int count, cudaStream_t stream);
// Test hook behind resq_debug_expire_next_wait (gemm_pair.cu).
void debug_expire_next_wait(int on);
// Whether launch_gemm_hif4 takes the keep flags of the block-wise selection for this shape (see GemmArgs::blk_flags).
bool gemm_block_lists_supported(int64_t M, int64_t N, int64_t K);
// Whether launch_gemm_hif4 takes the compressed 2:4 residual for this shape (the CTA-pair kernel runs it).
bool gemm_sparse24_supported(int64_t M, int64_t N, int64_t K);
// Layout of the 2:4 index metadata, fixed by the sparse MMA: blocks of 128 rows x 128 K positions (2 KB, row bands
// outermost); inside a block, rows of 16 bytes: byte 16 * (m % 8 + 8 * ((k / 16) % 2) + 16 * (m / 16)) + 4 * (k / 32)
// + 2 * ((m / 8) % 2) + (k / 8) % 2 holds the two 4-bit index pairs (idx0 | idx1 << 2, lower channels in the low
// nibble) of channels k .. k + 7 of row m (m, k relative to the block).
__host__ __device__ inline int64_t sparse24_meta_offset(int64_t m, int64_t k, int64_t ka) {
    return ((m >> 7) * ka + (k >> 7)) * 2048 + ((m >> 4) & 7) * 256 + ((k >> 4) & 1) * 128 + (m & 7) * 16 + ((k >> 5) & 3) * 4 +
           ((m >> 3) & 1) * 2 + ((k >> 3) & 1);
}
inline int64_t sparse24_rows128(int64_t M) { return (M + 255) / 256 * 2; }  // whole 256-row tiles of the pair kernel
inline int64_t sparse24_ka(int64_t K) { return (K + 127) / 128; }

// MXFP4 on the block-scaled FP4 tensor pipe (gemm_mxfp4.cu): operands stay packed E2M1 codes + E8M0 scales.
struct Mxfp4NativeArgs {
    const uint8_t* a_codes;   // [M, K/2]  Q(X)
    const uint8_t* a_scale;   // [M, K/32]
    const uint8_t* r_codes;   // [M, K/2]  S(Q(dX)) with the dropped codes zeroed, or null (pattern NONE)
    const uint8_t* r_scale;   // [M, K/32]
    const uint8_t* w_codes;   // [N, K/2]
    const uint8_t* w_scale;   // [N, K/32]
    int64_t M, N, K;
    void* Y;
    int out_dtype;
    int64_t ldy;
    float* partials;          // fp32 scratch for the partial tiles of a K split (decode-sized calls), or null
    size_t partial_bytes;
    DeviceStatus* status;
};
bool gemm_mxfp4_native_supported(int64_t M, int64_t N, int64_t K, bool res);
int launch_gemm_mxfp4_native(const Mxfp4NativeArgs& g, cudaStream_t stream);
int make_tmap_2d(CUtensorMap* m, CUtensorMapDataType dt, const void* base, uint64_t inner, uint64_t rows,
                 uint64_t row_stride_bytes, uint32_t box_inner, uint32_t box_rows, CUtensorMapSwizzle sw);
int launch_splitk_reduce(const GemmArgs& g, int splits, cudaStream_t stream);
int gemm_hif4_pick_splits(int64_t M, int64_t N, int64_t K);
size_t gemm_hif4_scratch_bytes(int64_t M, int64_t N, int64_t K);  // what splitk_partials must hold for this shape

}  // namespace resq
