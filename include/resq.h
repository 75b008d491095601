/*
 * resq.h -- C ABI of the B200 (sm_100a) Rollout-ResQ FP4 linear layer.
 *
 *     Y  =  Q(X) Q(W)^T  +  S(Q(X - deq Q(X))) Q(W)^T            (paper Eq. (5))
 *
 * X is the activation [M, K] (paper: m x d), W the weight [N, K] (paper: n x d), Y [M, N]
 * (Section 3, "Block-Scaled Quantization": Y = X W^T).  Q is a block-scaled 4-bit quantizer whose
 * blocks run along K.  Two formats are provided, as in the paper: HiF4 (blocks of 64, E6M2 level-1
 * scaler, E1 level-2 and level-3 scalers, S1P2 elements) and MXFP4 (blocks of 32, E8M0 scale,
 * E2M1 elements), the latter as the comparison twin (`mxfp4_*`).
 *
 * Conventions for every call
 *   - All tensor pointers are DEVICE pointers (the library never touches host data); row-major;
 *     `ld*` is the row stride in ELEMENTS of the pointed-to type.  bf16 inputs must be 16-byte
 *     aligned with ld a multiple of 8.  Packed outputs are dense (no stride); codes, metadata and
 *     scale outputs must be 4-byte aligned (they are written with 32-bit / 16-bit stores), mask_bits
 *     may start at any byte.  A misaligned pointer is RESQ_ERR_ALIGN, found on the host.
 *   - The RESQ_* environment variables are debugging overrides of the kernel choices; they are read only
 *     when RESQ_DEBUG is set to a non-zero value at the library's first call, otherwise never.
 *   - The caller owns every buffer; the library allocates no device memory.  Scratch comes from
 *     the `workspace` argument, sized by the matching *_workspace_bytes query (256-byte aligned).
 *   - Calls are asynchronous on `stream` (a cudaStream_t passed as void*; NULL = default stream).
 *   - The return value is a resq_status.  Shape / null / alignment / workspace errors are detected
 *     on the host before anything is launched.  Nothing throws.  resq_last_error() returns a
 *     thread-local description of the most recent failure.
 *   - Device-side waits are bounded; if one expires the kernel records RESQ_ERR_TIMEOUT in the
 *     status word at the start of the workspace and exits normally; resq_check() reads it.
 *
 * Packed layouts (bit-exact contract; the paper fixes the field widths only, the rest is this
 * library's reading, see the notes at each call)
 *   HiF4   codes[row][K/2] u8 : element 2j in bits 3:0, element 2j+1 in bits 7:4; a code is
 *                               sign<<3 | q, magnitude q/4 (S1P2 == E1M2: 0, .25, ..., 1.75).
 *          meta [row][K/64] u32: bits 7:0 level-1 E6M2 code s = E<<2|Mn, S1 = (1+Mn/4) 2^(E-48);
 *                               bit 8+i  = level-2 exponent of elements 8i..8i+7   (i = 0..7);
 *                               bit 16+j = level-3 exponent of elements 4j..4j+3   (j = 0..15).
 *          value = (-1)^sign (q/4) 2^(e2+e3) S1.
 *   MXFP4  codes as above with E2M1 codes (0,.5,1,1.5,2,3,4,6); scale[row][K/32] u8 E8M0 (2^(c-127)).
 *   mask   mask_bits[m][K/8] u8: bit (k&7) of byte k>>3 is 1 where S keeps element k of row m.
 */
#ifndef RESQ_H_
#define RESQ_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define RESQ_API __attribute__((visibility("default")))
#else
#define RESQ_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    RESQ_OK = 0,
    RESQ_ERR_NULL = 1,      /* a required pointer is NULL */
    RESQ_ERR_SHAPE = 2,     /* M,N,K <= 0; K % 64 (HiF4) or K % 32 (MXFP4); block pattern needs M % 32 == 0 */
    RESQ_ERR_ALIGN = 3,     /* base pointer not 16-byte aligned, or ld not a multiple of 8 / smaller than K */
    RESQ_ERR_WORKSPACE = 4, /* workspace NULL, misaligned or smaller than the query says */
    RESQ_ERR_PATTERN = 5,   /* unknown pattern or output type */
    RESQ_ERR_CUDA = 6,      /* a CUDA call or launch failed; text in resq_last_error() */
    RESQ_ERR_TIMEOUT = 7    /* a bounded device-side wait expired (reported by resq_check) */
} resq_status;

/* The sparsity function S of Eq. (5) (Section 4.3). */
typedef enum {
    RESQ_S_NONE = 0,          /* no residual term: Eq. (1) */
    RESQ_S_DENSE = 1,         /* S = identity: Eq. (4), "Rollout-ResQ-Dense" */
    RESQ_S_2_4 = 2,           /* keep the 2 largest magnitudes of every 4 contiguous elements along K;
                                 ties keep the lower index; always exactly 2 kept */
    RESQ_S_ROW50 = 3,         /* per row, keep the K/2 largest magnitudes (ties: lower index) */
    RESQ_S_CHAN50 = 4,        /* keep the K/2 channels (columns) with the largest L2 norm over all M rows */
    RESQ_S_BLOCK32x64_50 = 5  /* keep floor(nb/2) of the nb aligned blocks of 32 rows x 64 channels with the
                                 largest L2 norm, chosen over the whole tensor */
} resq_pattern;

/* Sparsity sweep (the paper evaluates 50 % and names other ratios as open, Section 6): a selecting pattern combined
 * with RESQ_KEEP_QUARTERS(q), q = 1, 2 or 3, keeps q/4 instead of 1/2: the q largest of every 4 (RESQ_S_2_4, i.e.
 * 1:4 / 2:4 / 3:4), floor(K q / 4) entries per row (RESQ_S_ROW50), floor(K q / 4) channels (RESQ_S_CHAN50),
 * floor(nb q / 4) blocks (RESQ_S_BLOCK32x64_50); same tie rules.  Accepted wherever a pattern argument is; q = 2 is
 * the pattern itself. */
#define RESQ_KEEP_QUARTERS(q) ((int)(q) << 8)

/* Load-balanced alternative of the block pattern (Section 4.3 item 3 selects over the whole tensor):
 * RESQ_S_BLOCK32x64_50 | RESQ_BLOCK_PER_STRIP selects inside every strip of 32 token rows -- each strip keeps the
 * floor((K/64) q / 4) of its own K/64 blocks with the largest sum of squares (ties: lower column block first), so
 * every strip of an M tile carries the same residual work.  May be combined with RESQ_KEEP_QUARTERS; with any other
 * pattern it is RESQ_ERR_PATTERN. */
#define RESQ_BLOCK_PER_STRIP (1 << 12)

typedef enum { RESQ_OUT_BF16 = 0, RESQ_OUT_F32 = 1 } resq_out;

/* ---- size queries (host only, no CUDA calls) -------------------------------------------------- */
RESQ_API size_t hif4_codes_bytes(int64_t rows, int64_t K);  /* rows*K/2 */
RESQ_API size_t hif4_meta_bytes(int64_t rows, int64_t K);   /* rows*(K/64)*4 */
RESQ_API size_t mxfp4_codes_bytes(int64_t rows, int64_t K); /* rows*K/2 */
RESQ_API size_t mxfp4_scale_bytes(int64_t rows, int64_t K); /* rows*(K/32) */
RESQ_API size_t resq_mask_bytes(int64_t M, int64_t K);      /* M*K/8 */
/* Scratch for *_residual_mask (status word, channel / block scores, selection buffers). */
RESQ_API size_t resq_residual_mask_workspace_bytes(int64_t M, int64_t K, int pattern);
/* Scratch for *_resq_linear (the above plus the expanded activation operands of the GEMM and,
 * for small M, split-K partial tiles). */
RESQ_API size_t hif4_resq_workspace_bytes(int64_t M, int64_t N, int64_t K, int pattern);
RESQ_API size_t mxfp4_resq_workspace_bytes(int64_t M, int64_t N, int64_t K, int pattern);

/* ---- Q(W): pack a weight once per policy update (Section 3, Eq. (1): W_hat = Q(W)) -------------
 * W_bf16 [N, K] with row stride ldw -> w_codes [N, K/2], w_meta [N, K/64] (HiF4) or w_scale [N, K/32].
 * HiF4 scale rule (this library's reading; the paper gives the field formats only): level 1 is the
 * smallest E6M2 value with 7*S1 >= max|block|; a level-2 / level-3 exponent is raised exactly when
 * the group would otherwise clip; elements round to nearest, ties to even.  MXFP4: scale exponent
 * floor(log2 max|block|) - 2, elements round to nearest even and saturate at 6. */
RESQ_API int hif4_pack_weight(const void* W_bf16, int64_t N, int64_t K, int64_t ldw, void* w_codes, void* w_meta, void* stream);
RESQ_API int mxfp4_pack_weight(const void* W_bf16, int64_t N, int64_t K, int64_t ldw, void* w_codes, void* w_scale, void* stream);

/* ---- Q(X): on-the-fly activation quantizer (same operator Q applied to X, Eq. (1)) ------------- */
RESQ_API int hif4_quantize_act(const void* X_bf16, int64_t M, int64_t K, int64_t ldx, void* x_codes, void* x_meta, void* stream);
RESQ_API int mxfp4_quantize_act(const void* X_bf16, int64_t M, int64_t K, int64_t ldx, void* x_codes, void* x_scale, void* stream);

/* ---- deq: decode packed data to fp32 [rows, K] (test helper; every HiF4 / MXFP4 value is fp32-exact) */
RESQ_API int hif4_dequantize(const void* codes, const void* meta, int64_t rows, int64_t K, float* out, void* stream);
RESQ_API int mxfp4_dequantize(const void* codes, const void* scale, int64_t rows, int64_t K, float* out, void* stream);

/* ---- Q(X), dX = X - deq Q(X) (Eq. (3)), Q(dX) (Eq. (4)) and the selection S (Eq. (5), Section 4.3)
 * in one pass over X.  Outputs (any of them may be NULL to skip it): Q(X), Q(dX) in the canonical
 * dense layout, and mask_bits.  S acts on the decoded magnitudes of Q(dX); kept elements keep their
 * value, dropped ones contribute zero.  For RESQ_S_NONE only Q(X) is written. */
RESQ_API int resq_residual_mask(const void* X_bf16, int64_t M, int64_t K, int64_t ldx, int pattern,
                       void* x_codes, void* x_meta, void* r_codes, void* r_meta, void* mask_bits,
                       void* workspace, size_t ws_bytes, void* stream);
RESQ_API int mxfp4_residual_mask(const void* X_bf16, int64_t M, int64_t K, int64_t ldx, int pattern,
                        void* x_codes, void* x_scale, void* r_codes, void* r_scale, void* mask_bits,
                        void* workspace, size_t ws_bytes, void* stream);

/* ---- the same pass for callers that cannot allocate device memory (the paper has no counterpart) ----
 * Meant for hosts that cannot give the library a workspace: a server that handed all device memory to its
 * own pool at start-up, a plugin invoked inside a serving loop where an allocation would stall the device,
 * or a foreign-function caller that owns only its inputs and outputs.  Same inputs, outputs, patterns (the
 * RESQ_KEEP_QUARTERS and RESQ_BLOCK_PER_STRIP modifiers included) and results as resq_residual_mask (HiF4), but the scratch of the channel-wise and block-wise selections lives
 * in a fixed device array inside the library image (about 290 KB, held by every GPU that loads the
 * library until the process exits).  The call performs no cudaMalloc / cudaFree and uses no allocating
 * library routine.
 *   - Limit: at most RESQ_STATIC_SCRATCH_MAX_SCORES selection scores, i.e. K for RESQ_S_CHAN50 and
 *     (M/32)*(K/64) for RESQ_S_BLOCK32x64_50 (with or without RESQ_BLOCK_PER_STRIP); larger problems return RESQ_ERR_WORKSPACE with a message
 *     (the other patterns need no scores and have no limit).
 *   - The first call on each device looks up the array's device address (with that device current); make
 *     that first call before starting any stream capture.
 *   - All calls on a device share the one array, which keeps the previous call's contents; the call clears
 *     what has to start from zero itself.  Two calls whose kernels overlap on the GPU (different streams,
 *     or different host threads) race on it: serialise them. */
#define RESQ_STATIC_SCRATCH_MAX_SCORES 32768
RESQ_API int resq_residual_mask_static(const void* X_bf16, int64_t M, int64_t K, int64_t ldx, int pattern,
                                       void* x_codes, void* x_meta, void* r_codes, void* r_meta, void* mask_bits,
                                       void* stream);

/* ---- the rollout projection, Eq. (5):  Y = Q(X) Q(W)^T + S(Q(dX)) Q(W)^T ------------------------
 * X_bf16 [M, K] (ldx), packed weight from *_pack_weight, Y [M, N] (ldy) as bf16 (round-to-nearest-
 * even of the fp32 accumulator) or fp32.  Products of decoded values are exact in fp32; only the
 * accumulation rounds.  Both terms are accumulated into the same output tile.
 *   - The workspace holds the status word, arrival counters, the quantizer's outputs and fp32 partial
 *     tiles of the call: a workspace must not be shared by calls whose kernels may overlap on the GPU.
 *   - For decode-sized problems the GEMM kernel's CTAs wait for one another at its end (bounded) and are
 *     sized to be resident all at once on an otherwise idle device.  Calls whose kernels overlap on the
 *     same device (different streams) can therefore delay each other up to the bound and then end with
 *     RESQ_ERR_TIMEOUT in the status word instead of a result: issue them on one stream.
 *   - Consecutive calls on one stream overlap their kernels' set-up through programmatic dependent
 *     launch; every kernel waits for its predecessor before it touches memory that one may have written.
 *   - MXFP4 with K a multiple of 256 runs on the block-scaled FP4 tensor pipe where that is faster (all but
 *     long-K calls with few output tiles); everything else on the bf16 pipe.  Both are exact in the products;
 *     they differ in accumulation order only. */
RESQ_API int hif4_resq_linear(const void* X_bf16, int64_t M, int64_t K, int64_t ldx,
                     const void* w_codes, const void* w_meta, int64_t N,
                     int pattern, void* Y, int out_dtype, int64_t ldy,
                     void* workspace, size_t ws_bytes, void* stream);
RESQ_API int mxfp4_resq_linear(const void* X_bf16, int64_t M, int64_t K, int64_t ldx,
                      const void* w_codes, const void* w_scale, int64_t N,
                      int pattern, void* Y, int out_dtype, int64_t ldy,
                      void* workspace, size_t ws_bytes, void* stream);

/* ---- several independent projections of Eq. (5) in one call (the paper treats one projection; the grouping is this
 * library's, for decode-sized problems) -----------------------------------------------------------------------------
 * At a few hundred token rows a single projection cannot fill the device: its launch, pipeline fill and the sum of its
 * partial tiles cost more than its arithmetic.  A group of up to RESQ_MAX_GROUP projections that do not depend on one
 * another (the q/k/v, gate and up projections of a block, the experts of a mixture, the layers of several models)
 * runs as ONE quantizer launch and ONE GEMM launch whose CTA pairs walk the output tiles of all problems: whole tiles
 * first, the k-blocks of the remaining tiles dealt out evenly, partial tiles summed in a fixed order inside the kernel
 * (bit-identical results run to run).  A group whose problems all have at most 32 token rows takes a kernel of its own:
 * 128 weight rows are the M dimension of the MMA and the tokens its N, the (tile, k-block) units of all problems are cut
 * into equal ranges, one per CTA, and the last CTA to finish a tile adds its partial tiles in k order (no CTA waits for
 * another there).  Each problem is exactly *_resq_linear: same quantizer, residual and selection, results within the same
 * tolerance (the fp32 summation order over K differs from the single call's).
 *   - `problems` is a HOST array read during the call; its tensor pointers are device pointers with the alignment
 *     rules of *_resq_linear; M, N, K may differ from problem to problem; any M >= 1.
 *   - pattern: RESQ_S_NONE, RESQ_S_DENSE or RESQ_S_2_4 (with RESQ_KEEP_QUARTERS), one for the whole group; the
 *     selections that look beyond a token row (ROW50, CHAN50, BLOCK) are RESQ_ERR_PATTERN here.
 *   - workspace of *_resq_group_workspace_bytes(problems, count, pattern) bytes, owned by the caller; status word,
 *     bounded waits and resq_check as for *_resq_linear (the CTAs of the GEMM wait for one another at its end: issue
 *     overlapping calls on one stream). */
#define RESQ_MAX_GROUP 8
typedef struct resq_problem {
    const void* X_bf16;  /* [M, K] device, row pitch ldx */
    int64_t M, K, ldx;
    const void* w_codes; /* [N, K/2] from *_pack_weight */
    const void* w_side;  /* HiF4: w_meta [N, K/64] u32; MXFP4: w_scale [N, K/32] u8 */
    int64_t N;
    void* Y;             /* [M, N] device, row pitch ldy; bf16 or fp32 as out_dtype says */
    int64_t ldy;
} resq_problem;
RESQ_API size_t hif4_resq_group_workspace_bytes(const resq_problem* problems, int count, int pattern);
RESQ_API size_t mxfp4_resq_group_workspace_bytes(const resq_problem* problems, int count, int pattern);
RESQ_API int hif4_resq_linear_group(const resq_problem* problems, int count, int pattern, int out_dtype,
                           void* workspace, size_t ws_bytes, void* stream);
RESQ_API int mxfp4_resq_linear_group(const resq_problem* problems, int count, int pattern, int out_dtype,
                            void* workspace, size_t ws_bytes, void* stream);

/* ---- the backward products of the layer, in 4 bit (training side) ---------------------------------------------------
 * The paper's training policy runs its forward and backward passes in 4 bit (Sections 1 and 3) and writes out the
 * forward product only, Eq. (1).  This library's reading: Eq. (1)'s operator Q on both operands of each backward
 * product, with the quantization blocks along that product's contraction axis, no residual term:
 *     dX^ [M, K] = Q(dY) Q(W^T)^T        dY [M, N], blocks along N;  W^T [K, N] packed once by *_pack_weight_transposed
 *     dW^ [N, K] = Q(dY^T) Q(X^T)^T      dY^T [N, M], X^T [K, M], blocks along M (M a multiple of 64 / 32)
 * Each is the layer call (*_resq_linear with RESQ_S_NONE) on transposed operands; the transposes are bf16 copies in the
 * workspace.  Argument rules, output types and error behaviour as *_resq_linear.
 *   *_pack_weight_transposed: W_bf16 [N, K] (ldw) -> wt_codes [K, N/2], wt_meta [K, N/64] (wt_scale [K, N/32]);
 *       N a multiple of the block size; workspace of resq_transposed_workspace_bytes(N, K) bytes.
 *   *_dgrad_linear: dY_bf16 [M, N] (lddy), the transposed pack, dX [M, K] (lddx); workspace *_dgrad_workspace_bytes.
 *   *_wgrad_linear: dY_bf16 [M, N] (lddy), X_bf16 [M, K] (ldx), dW [N, K] (lddw); workspace *_wgrad_workspace_bytes. */
RESQ_API size_t resq_transposed_workspace_bytes(int64_t N, int64_t K);
RESQ_API int hif4_pack_weight_transposed(const void* W_bf16, int64_t N, int64_t K, int64_t ldw, void* wt_codes, void* wt_meta,
                                void* workspace, size_t ws_bytes, void* stream);
RESQ_API int mxfp4_pack_weight_transposed(const void* W_bf16, int64_t N, int64_t K, int64_t ldw, void* wt_codes, void* wt_scale,
                                 void* workspace, size_t ws_bytes, void* stream);
RESQ_API size_t hif4_dgrad_workspace_bytes(int64_t M, int64_t N, int64_t K);
RESQ_API size_t mxfp4_dgrad_workspace_bytes(int64_t M, int64_t N, int64_t K);
RESQ_API int hif4_dgrad_linear(const void* dY_bf16, int64_t M, int64_t N, int64_t lddy, const void* wt_codes, const void* wt_meta,
                      int64_t K, void* dX, int out_dtype, int64_t lddx, void* workspace, size_t ws_bytes, void* stream);
RESQ_API int mxfp4_dgrad_linear(const void* dY_bf16, int64_t M, int64_t N, int64_t lddy, const void* wt_codes, const void* wt_scale,
                       int64_t K, void* dX, int out_dtype, int64_t lddx, void* workspace, size_t ws_bytes, void* stream);
RESQ_API size_t hif4_wgrad_workspace_bytes(int64_t M, int64_t N, int64_t K);
RESQ_API size_t mxfp4_wgrad_workspace_bytes(int64_t M, int64_t N, int64_t K);
RESQ_API int hif4_wgrad_linear(const void* dY_bf16, const void* X_bf16, int64_t M, int64_t N, int64_t K, int64_t lddy, int64_t ldx,
                      void* dW, int out_dtype, int64_t lddw, void* workspace, size_t ws_bytes, void* stream);
RESQ_API int mxfp4_wgrad_linear(const void* dY_bf16, const void* X_bf16, int64_t M, int64_t N, int64_t K, int64_t lddy, int64_t ldx,
                       void* dW, int out_dtype, int64_t lddw, void* workspace, size_t ws_bytes, void* stream);

/* Weight-only ablation of Table 1 ("W4A16"): Y = X deq(Q(W))^T, the bf16 activations are used as they are
 * (no activation quantizer, no residual term); weights as produced by *_pack_weight.  Same argument rules,
 * output types and error behaviour as *_resq_linear; workspace of resq_w4a16_workspace_bytes(M, N, K) bytes
 * (status word, arrival counters, fp32 partial tiles of a K split), owned by the caller. */
RESQ_API size_t resq_w4a16_workspace_bytes(int64_t M, int64_t N, int64_t K);
RESQ_API int hif4_w4a16_linear(const void* X_bf16, int64_t M, int64_t K, int64_t ldx,
                      const void* w_codes, const void* w_meta, int64_t N,
                      void* Y, int out_dtype, int64_t ldy,
                      void* workspace, size_t ws_bytes, void* stream);
RESQ_API int mxfp4_w4a16_linear(const void* X_bf16, int64_t M, int64_t K, int64_t ldx,
                       const void* w_codes, const void* w_scale, int64_t N,
                       void* Y, int out_dtype, int64_t ldy,
                       void* workspace, size_t ws_bytes, void* stream);

/* Weight-and-8-bit-activation ablation of Table 1 ("W4A8"): Y = deq(Q8(X)) deq(Q(W))^T.  The paper names the
 * ablation but not the 8-bit format; this library's reading is MXFP8 with E4M3 elements as the OCP microscaling
 * specification defines it: blocks of 32 along K, one E8M0 scale 2^(floor(log2 amax) - 8) per block (all-zero
 * block: scale code 0), elements rounded to the nearest E4M3 value (ties to even, subnormals below 2^-6) and
 * saturated at +-448; used with both weight formats.  K % 32 == 0 (K % 64 == 0 with HiF4 weights).  No residual
 * term.  Decoded activations below 2^-126 in magnitude lose bits (the GEMM operand is bf16).  Same argument
 * rules, output types and error behaviour as *_resq_linear; workspace of resq_w4a8_workspace_bytes(M, N, K). */
RESQ_API size_t resq_w4a8_workspace_bytes(int64_t M, int64_t N, int64_t K);
RESQ_API int hif4_w4a8_linear(const void* X_bf16, int64_t M, int64_t K, int64_t ldx,
                     const void* w_codes, const void* w_meta, int64_t N,
                     void* Y, int out_dtype, int64_t ldy,
                     void* workspace, size_t ws_bytes, void* stream);
RESQ_API int mxfp4_w4a8_linear(const void* X_bf16, int64_t M, int64_t K, int64_t ldx,
                      const void* w_codes, const void* w_scale, int64_t N,
                      void* Y, int out_dtype, int64_t ldy,
                      void* workspace, size_t ws_bytes, void* stream);

/* Down projection with its producer fused into the quantizer pass: the input is GU_bf16 = [gate | up], [M, 2K]
 * device (row pitch ldgu >= 2K elements, ldgu % 8 == 0, 16-byte aligned base), the layer's activations are
 * X = bf16(SiLU(gate) * up), formed on the fly and never written to memory; everything after that is
 * *_resq_linear on X (Eq. (5)).  The rounding of X to bf16 decides 4-bit codes, so SiLU is evaluated by a fixed
 * fp32 procedure (every operation rounded to nearest even, no fused multiply-add): t = g * (-log2 e) clamped to
 * [-126, 126], n = rint(t), f = t - n, p = 2^f by the degree-6 Taylor polynomial of exp(f ln 2) in Horner form,
 * e = p * 2^n, s = g / (1 + e), X = bf16(s * u).  All selections but RESQ_S_ROW50 (RESQ_ERR_PATTERN).  Workspace,
 * output and errors as *_resq_linear with the same (M, N, K, pattern). */
RESQ_API int hif4_swiglu_resq_linear(const void* GU_bf16, int64_t M, int64_t K, int64_t ldgu,
                            const void* w_codes, const void* w_meta, int64_t N,
                            int pattern, void* Y, int out_dtype, int64_t ldy,
                            void* workspace, size_t ws_bytes, void* stream);
RESQ_API int mxfp4_swiglu_resq_linear(const void* GU_bf16, int64_t M, int64_t K, int64_t ldgu,
                             const void* w_codes, const void* w_scale, int64_t N,
                             int pattern, void* Y, int out_dtype, int64_t ldy,
                             void* workspace, size_t ws_bytes, void* stream);

/* Projection with its RMSNorm producer fused into the quantizer pass (qkv / gate_up inputs): H_bf16 [M, K] device
 * (row pitch ldh), gamma_bf16 [K] device (16-byte aligned), the layer's activations are
 * X[m,k] = bf16((H[m,k] * r[m]) * gamma[k]), r[m] = 1 / sqrt(sum_k H[m,k]^2 / K + eps), formed on the fly and
 * never written to memory; everything after that is *_resq_linear on X.  Fixed evaluation: the sum of squares is
 * the exact sum rounded once to fp32 (realised by a fixed-order fp64 sum of the exact squares), every later
 * operation is correctly rounded fp32 (division, square root, division, two multiplies), no fused multiply-add.
 * A small row kernel computes r (kept in the workspace) before the quantizer kernel.  All selections but
 * RESQ_S_ROW50.  Workspace, output and errors as *_resq_linear with the same (M, N, K, pattern). */
RESQ_API int hif4_rmsnorm_resq_linear(const void* H_bf16, int64_t M, int64_t K, int64_t ldh,
                             const void* gamma_bf16, float eps,
                             const void* w_codes, const void* w_meta, int64_t N,
                             int pattern, void* Y, int out_dtype, int64_t ldy,
                             void* workspace, size_t ws_bytes, void* stream);
RESQ_API int mxfp4_rmsnorm_resq_linear(const void* H_bf16, int64_t M, int64_t K, int64_t ldh,
                              const void* gamma_bf16, float eps,
                              const void* w_codes, const void* w_scale, int64_t N,
                              int pattern, void* Y, int out_dtype, int64_t ldy,
                              void* workspace, size_t ws_bytes, void* stream);

/* Rotation baseline (the randomized Hadamard transform the paper compares against, Section 5.1): per block of 64
 * channels, x' = bf16((1/8) H64 (s * x)) with H64 the Sylvester Hadamard matrix and s in {+1, -1}^64 given by
 * `signs` (bit j set: channel j of every block is negated); H64 / 8 is orthogonal, so rotating X and W alike leaves
 * X W^T unchanged in exact arithmetic.  Fixed evaluation: in-place fast transform in fp32, strides 1, 2, 4, 8, 16,
 * 32, each stage (a, b) -> (a + b, a - b) with a the lower channel, every operation rounded to nearest even, the
 * scale exact.  K % 64 == 0 (both formats).  *_rht_pack_weight rotates and packs W (same outputs as
 * *_pack_weight); *_rht_resq_linear rotates X in the quantizer pass (never stored) and then is *_resq_linear
 * against weights packed with the same `signs`; all selections but RESQ_S_ROW50; pattern RESQ_S_NONE is the plain
 * rotation baseline.  Workspace, outputs and errors as *_pack_weight / *_resq_linear. */
RESQ_API int hif4_rht_pack_weight(const void* W_bf16, int64_t N, int64_t K, int64_t ldw, unsigned long long signs,
                         void* w_codes, void* w_meta, void* stream);
RESQ_API int mxfp4_rht_pack_weight(const void* W_bf16, int64_t N, int64_t K, int64_t ldw, unsigned long long signs,
                          void* w_codes, void* w_scale, void* stream);
RESQ_API int hif4_rht_resq_linear(const void* X_bf16, int64_t M, int64_t K, int64_t ldx, unsigned long long signs,
                         const void* w_codes, const void* w_meta, int64_t N,
                         int pattern, void* Y, int out_dtype, int64_t ldy,
                         void* workspace, size_t ws_bytes, void* stream);
RESQ_API int mxfp4_rht_resq_linear(const void* X_bf16, int64_t M, int64_t K, int64_t ldx, unsigned long long signs,
                          const void* w_codes, const void* w_scale, int64_t N,
                          int pattern, void* Y, int out_dtype, int64_t ldy,
                          void* workspace, size_t ws_bytes, void* stream);

/* Activation-only ablation of Table 1 ("W16A4"): Y = (deq Q(X) + S(deq Q(dX))) W^T with the weights in plain
 * bf16 (W_bf16: [N, K] device, row pitch ldw elements, ldw >= K, ldw % 8 == 0, 16-byte aligned base); the
 * activations go through the same quantizer, residual and selection as *_resq_linear (pattern RESQ_S_NONE gives
 * the table's plain Q(X) W^T).  Same argument rules, output types, error behaviour and workspace
 * (*_resq_workspace_bytes(M, N, K, pattern)) as *_resq_linear. */
RESQ_API int hif4_w16a4_linear(const void* X_bf16, int64_t M, int64_t K, int64_t ldx,
                      const void* W_bf16, int64_t N, int64_t ldw,
                      int pattern, void* Y, int out_dtype, int64_t ldy,
                      void* workspace, size_t ws_bytes, void* stream);
RESQ_API int mxfp4_w16a4_linear(const void* X_bf16, int64_t M, int64_t K, int64_t ldx,
                       const void* W_bf16, int64_t N, int64_t ldw,
                       int pattern, void* Y, int out_dtype, int64_t ldy,
                       void* workspace, size_t ws_bytes, void* stream);

/* ---- status --------------------------------------------------------------------------------------
 * resq_check synchronizes `stream` and returns the device status word kept at the start of
 * `workspace` (RESQ_OK, or RESQ_ERR_TIMEOUT if a bounded wait expired in the last call that used it). */
RESQ_API int resq_check(void* workspace, void* stream);
RESQ_API const char* resq_last_error(void);

/* ---- diagnostics (no counterpart in the paper) -----------------------------------------------------
 * resq_kernel_launches: number of kernels this library has launched in the process so far.
 * resq_profile_enable(1): from now on every kernel launch is bracketed by a pair of CUDA events on its
 * stream (this perturbs timing slightly; leave it off when measuring whole-call time).
 * resq_profile_read: synchronizes on the recorded events, adds the device time (ms) and the number of
 * launches per kernel kind into the two arrays of 4 entries (0 = quantizer/residual/mask pass,
 * 1 = top-k select and mask apply, 2 = GEMM, 3 = split-K reduce; either array may be NULL) and
 * clears the records.
 * resq_debug_expire_next_wait(1): test hook for the RESQ_ERR_TIMEOUT path.  The next decode-sized GEMM launch of
 * the process (K-streamed schedule: M > 128 and few output tiles) waits at its end for one partial tile more than
 * its CTAs can deliver, with a poll limit of about a millisecond: the bounded wait runs out, the kernel records
 * RESQ_ERR_TIMEOUT in the status word, leaves through its normal exit (tensor memory freed, no output for the
 * tiles it was summing) and the context stays usable; resq_check then returns RESQ_ERR_TIMEOUT and the next call
 * on the same workspace is an ordinary one.  Nothing faults or hangs.  (0 withdraws an unconsumed request.) */
RESQ_API int64_t resq_kernel_launches(void);
RESQ_API int resq_debug_expire_next_wait(int on);
RESQ_API int resq_profile_enable(int on);
RESQ_API int resq_profile_read(double* ms_by_kind, int64_t* launches_by_kind);

#ifdef __cplusplus
}
#endif
#endif /* RESQ_H_ */
