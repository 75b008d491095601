// C ABI of the ResQ library: argument checks, workspace carving, kernel sequencing.
// The contract of every entry point is stated in include/resq.h.
#include "common.cuh"
#include <algorithm>

#include <atomic>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <map>
#include <mutex>
#include <tuple>
#include <utility>
#include <vector>

namespace resq {

static thread_local char g_last_error[512] = "";

void set_last_error(const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_last_error, sizeof(g_last_error), fmt, ap);
    va_end(ap);
}

int cuda_fail(cudaError_t e, const char* what) {
    if (e == cudaSuccess) return RESQ_OK;
    set_last_error("%s: %s", what, cudaGetErrorString(e));
    return RESQ_ERR_CUDA;
}

// ---- diagnostics: launch counter and optional per-kernel event timing ---------------------------
namespace {
std::atomic<long long> g_launches{0};
std::atomic<int> g_profile{0};
struct ProfRec {
    int kind;
    cudaEvent_t start, stop;
};
std::mutex g_prof_mu;
std::vector<ProfRec*> g_prof;
}  // namespace

bool debug_overrides() {
    static const bool on = [] {
        const char* v = getenv("RESQ_DEBUG");
        return v && *v && *v != '0';
    }();
    return on;
}
int env_int(const char* name, int dflt) {
    if (!debug_overrides()) return dflt;
    const char* v = getenv(name);
    return v && *v ? atoi(v) : dflt;
}
bool env_is_zero(const char* name) {
    if (!debug_overrides()) return false;
    const char* v = getenv(name);
    return v && *v == '0';
}

int device_sm_count() {
    constexpr int kMaxDev = 64;
    static std::mutex mu;
    static int sms[kMaxDev] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDev) return 148;
    std::lock_guard<std::mutex> lk(mu);
    if (sms[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
        sms[dev] = n;
    }
    return sms[dev];
}

namespace {
std::mutex g_dev_mu;
std::map<std::pair<int, const void*>, int> g_smem_opt_in;                    // (device, function) -> bytes set
std::map<std::tuple<int, const void*, size_t>, int> g_max_clusters;         // (device, function, smem) -> clusters
}  // namespace

int ensure_dynamic_smem(const void* func, int bytes, const char* what) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e, "cudaGetDevice");
    std::lock_guard<std::mutex> lk(g_dev_mu);
    int& have = g_smem_opt_in[std::make_pair(dev, func)];
    if (have >= bytes) return RESQ_OK;
    e = cudaFuncSetAttribute(func, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e != cudaSuccess) return cuda_fail(e, what);
    have = bytes;
    return RESQ_OK;
}

int max_active_clusters(const void* func, const cudaLaunchConfig_t* cfg, int* out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e, "cudaGetDevice");
    std::lock_guard<std::mutex> lk(g_dev_mu);
    const auto key = std::make_tuple(dev, func, cfg->dynamicSmemBytes);
    auto it = g_max_clusters.find(key);
    if (it == g_max_clusters.end()) {
        int n = 0;
        e = cudaOccupancyMaxActiveClusters(&n, func, cfg);
        if (e != cudaSuccess) return cuda_fail(e, "cudaOccupancyMaxActiveClusters");
        it = g_max_clusters.emplace(key, n).first;
    }
    *out = it->second;
    return RESQ_OK;
}

bool pdl_enabled() {
    static const int on = env_int("RESQ_PDL", 1);
    // event records between the kernels (profiling) would serialize them anyway
    return on != 0 && !g_profile.load(std::memory_order_relaxed);
}

LaunchScope::LaunchScope(int kind, cudaStream_t stream) : kind_(kind), stream_(stream), rec_(nullptr) {
    g_launches.fetch_add(1, std::memory_order_relaxed);
    if (!g_profile.load(std::memory_order_relaxed)) return;
    ProfRec* r = new ProfRec{kind, nullptr, nullptr};
    if (cudaEventCreate(&r->start) != cudaSuccess || cudaEventCreate(&r->stop) != cudaSuccess) {
        delete r;
        return;
    }
    cudaEventRecord(r->start, stream);
    rec_ = r;
}
LaunchScope::~LaunchScope() {
    if (!rec_) return;
    ProfRec* r = static_cast<ProfRec*>(rec_);
    cudaEventRecord(r->stop, stream_);
    std::lock_guard<std::mutex> lk(g_prof_mu);
    g_prof.push_back(r);
}

// A pattern argument is a base pattern, optionally combined with RESQ_KEEP_QUARTERS(q): splits it in place.
int split_pattern(int* pattern, int* quarters, int* per_strip) {
    const int q = (*pattern >> 8) & 0xF;
    const int strip = (*pattern >> 12) & 1;
    if (*pattern < 0 || (*pattern >> 13) != 0 || q > 3) {
        set_last_error("unknown pattern %d", *pattern);
        return RESQ_ERR_PATTERN;
    }
    *quarters = q == 0 ? 2 : q;
    *per_strip = strip;
    *pattern &= 0xFF;
    if (q != 0 && (*pattern == RESQ_S_NONE || *pattern == RESQ_S_DENSE)) {
        set_last_error("RESQ_KEEP_QUARTERS applies to the selecting patterns only");
        return RESQ_ERR_PATTERN;
    }
    if (strip && *pattern != RESQ_S_BLOCK32x64_50) {
        set_last_error("RESQ_BLOCK_PER_STRIP applies to RESQ_S_BLOCK32x64_50 only");
        return RESQ_ERR_PATTERN;
    }
    return RESQ_OK;
}
int check_pattern(int pattern, int64_t M) {
    if (pattern < RESQ_S_NONE || pattern > RESQ_S_BLOCK32x64_50) {
        set_last_error("unknown pattern %d", pattern);
        return RESQ_ERR_PATTERN;
    }
    if (pattern == RESQ_S_BLOCK32x64_50 && M % kBlkRows != 0) {
        set_last_error("the 32x64 block pattern needs M %% 32 == 0 (M=%lld)", (long long)M);
        return RESQ_ERR_SHAPE;
    }
    return RESQ_OK;
}

int check_packed_outputs(const void* x_codes, const void* x_side, const void* r_codes, const void* r_side) {
    const void* ptrs[4] = {x_codes, x_side, r_codes, r_side};
    const char* names[4] = {"x_codes", "x_meta / x_scale", "r_codes", "r_meta / r_scale"};
    for (int i = 0; i < 4; ++i)
        if (ptrs[i] && (reinterpret_cast<uintptr_t>(ptrs[i]) & 3u) != 0) {
            set_last_error("%s must be 4-byte aligned (%p)", names[i], ptrs[i]);
            return RESQ_ERR_ALIGN;
        }
    return RESQ_OK;
}

namespace {

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline int block_of(int fmt) { return fmt == kHiF4 ? kHif4Block : kMxBlock; }

int check_matrix(const void* p, int64_t rows, int64_t K, int64_t ld, int fmt, const char* name) {
    if (!p) {
        set_last_error("%s is NULL", name);
        return RESQ_ERR_NULL;
    }
    if (rows <= 0 || K <= 0 || K % block_of(fmt) != 0) {
        set_last_error("%s: rows=%lld K=%lld (K must be a positive multiple of %d)", name, (long long)rows, (long long)K,
                       block_of(fmt));
        return RESQ_ERR_SHAPE;
    }
    if (!aligned16(p) || ld < K || ld % 8 != 0) {
        set_last_error("%s: needs a 16-byte aligned base and ld >= K, ld %% 8 == 0 (ld=%lld)", name, (long long)ld);
        return RESQ_ERR_ALIGN;
    }
    return RESQ_OK;
}

int base_pattern(int pattern) { return pattern < 0 ? pattern : pattern & 0xFF; }

int check_workspace(const void* ws, size_t have, size_t need) {
    if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255u) != 0 || have < need) {
        set_last_error("workspace: need %zu bytes, 256-byte aligned (have %zu at %p)", need, have, ws);
        return RESQ_ERR_WORKSPACE;
    }
    return RESQ_OK;
}

int quantize_only(int fmt, const void* X, int64_t rows, int64_t K, int64_t ld, void* codes, void* side, void* stream,
                  const char* name, bool rht = false, unsigned long long rht_signs = 0) {
    int rc = check_matrix(X, rows, K, ld, fmt, name);
    if (rc) return rc;
    if (!codes || !side) {
        set_last_error("%s: output pointer is NULL", name);
        return RESQ_ERR_NULL;
    }
    rc = check_packed_outputs(codes, side, nullptr, nullptr);
    if (rc) return rc;
    QuantArgs a;
    memset(&a, 0, sizeof(a));
    a.X = static_cast<const __nv_bfloat16*>(X);
    a.M = rows;
    a.K = K;
    a.ldx = ld;
    a.pattern = RESQ_S_NONE;
    a.x_codes = static_cast<uint8_t*>(codes);
    a.x_side = side;
    if (rht) {
        if (K % 64 != 0) {
            set_last_error("%s: the Hadamard pre-transform needs K %% 64 == 0 (K=%lld)", name, (long long)K);
            return RESQ_ERR_SHAPE;
        }
        a.rht = 1;
        a.rht_signs = rht_signs;
    }
    return launch_quantize(fmt, a, static_cast<cudaStream_t>(stream));
}

int dequantize(int fmt, const void* codes, const void* side, int64_t rows, int64_t K, float* out, void* stream) {
    if (!codes || !side || !out) {
        set_last_error("dequantize: NULL pointer");
        return RESQ_ERR_NULL;
    }
    if (rows <= 0 || K <= 0 || K % block_of(fmt) != 0) {
        set_last_error("dequantize: bad shape");
        return RESQ_ERR_SHAPE;
    }
    return launch_dequantize(fmt, static_cast<const uint8_t*>(codes), side, rows, K, out, static_cast<cudaStream_t>(stream));
}

// carve [header | scores | flags] from the front of a workspace
void carve_quant_scratch(uint8_t* ws, int64_t M, int64_t K, int pattern, QuantArgs& a, size_t& used) {
    a.status = reinterpret_cast<DeviceStatus*>(ws);
    used = kWsHeader;
    size_t n = 0;
    if (pattern == RESQ_S_CHAN50) n = (size_t)K;
    if (pattern == RESQ_S_BLOCK32x64_50) n = (size_t)(M / kBlkRows) * (size_t)(K / kBlkCols);
    if (n) {
        a.scores = reinterpret_cast<double*>(ws + used);
        used += align_up(n * sizeof(double), 256);
        a.keep_flags = ws + used;
        used += align_up(n, 256);
        if ((int64_t)n > kSelGridMin) {
            a.sel_hist = reinterpret_cast<uint32_t*>(ws + used);
            used += kSelGridScratch;
        }
    }
}

int residual_mask(int fmt, const void* X, int64_t M, int64_t K, int64_t ldx, int pattern, void* x_codes, void* x_side,
                  void* r_codes, void* r_side, void* mask_bits, void* workspace, size_t ws_bytes, void* stream) {
    int rc = check_matrix(X, M, K, ldx, fmt, "X");
    if (rc) return rc;
    int quarters = 2, per_strip = 0;
    rc = split_pattern(&pattern, &quarters, &per_strip);
    if (rc) return rc;
    rc = check_pattern(pattern, M);
    if (rc) return rc;
    rc = check_packed_outputs(x_codes, x_side, r_codes, r_side);
    if (rc) return rc;
    rc = check_workspace(workspace, ws_bytes, resq_residual_mask_workspace_bytes(M, K, pattern));
    if (rc) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemsetAsync(workspace, 0, kWsHeader, st);
    if (e != cudaSuccess) return cuda_fail(e, "cudaMemsetAsync(status)");
    QuantArgs a;
    memset(&a, 0, sizeof(a));
    a.X = static_cast<const __nv_bfloat16*>(X);
    a.M = M;
    a.K = K;
    a.ldx = ldx;
    a.pattern = pattern;
    a.keep_quarters = quarters;
    a.per_strip = per_strip;
    a.x_codes = static_cast<uint8_t*>(x_codes);
    a.x_side = x_side;
    if (pattern != RESQ_S_NONE) {
        a.r_codes = static_cast<uint8_t*>(r_codes);
        a.r_side = r_side;
        a.mask_bits = static_cast<uint8_t*>(mask_bits);
    }
    size_t used = 0;
    carve_quant_scratch(static_cast<uint8_t*>(workspace), M, K, pattern, a, used);
    return launch_quantize(fmt, a, st);
}

// Residual operand region: the bf16 image of S(deq Q(dX)), or (2:4 on the sparse MMA) the compressed image [M, K/2]
// followed by the index metadata; sized for either.
size_t sparse24_meta_bytes(int64_t M, int64_t K) { return (size_t)sparse24_rows128(M) * (size_t)sparse24_ka(K) * 2048; }
size_t residual_region_bytes(int64_t M, int64_t K, int pattern) {
    if (pattern == RESQ_S_NONE) return 0;
    size_t b = (size_t)M * (size_t)K * 2;
    if (pattern == RESQ_S_2_4) b = std::max(b, align_up((size_t)M * (size_t)K, 256) + sparse24_meta_bytes(M, K));
    return align_up(b, 256);
}

size_t linear_workspace_bytes(int fmt, int64_t M, int64_t N, int64_t K, int pattern) {
    if (M <= 0 || N <= 0 || K <= 0) return 0;
    size_t b = kWsHeader + kWsFlags + quant_scratch_bytes(M, K, pattern);
    b += align_up((size_t)M * (size_t)K * 2, 256);                            // bf16 image of deq Q(X)
    b += residual_region_bytes(M, K, pattern);
    b += align_up(gemm_hif4_scratch_bytes(M, N, K), 256);                     // fp32 partial tiles of a K split
    b += align_up((size_t)M * sizeof(float), 256);                            // row scales of the fused RMSNorm producer
    return b;
}

// w_bf16 != null: activation-only quantization (Table 1, "W16A4"): plain bf16 weights [N, K] with row pitch ldw
// instead of the packed ones.
int linear(int fmt, const void* X, int64_t M, int64_t K, int64_t ldx, const void* w_codes, const void* w_side, int64_t N,
           int pattern, void* Y, int out_dtype, int64_t ldy, void* workspace, size_t ws_bytes, void* stream,
           const void* w_bf16 = nullptr, int64_t ldw = 0, bool swiglu = false, const void* gamma = nullptr, float eps = 0.0f,
           bool rht = false, unsigned long long rht_signs = 0) {
    int rc = check_matrix(X, M, K, ldx, fmt, "X");
    if (rc) return rc;
    int quarters = 2, per_strip = 0;
    rc = split_pattern(&pattern, &quarters, &per_strip);
    if (rc) return rc;
    if (swiglu && ldx < 2 * K) {  // X is [gate | up]: 2K columns
        set_last_error("swiglu: the input needs 2K columns per row (ldx=%lld, K=%lld)", (long long)ldx, (long long)K);
        return RESQ_ERR_SHAPE;
    }
    if (rht && K % 64 != 0) {
        set_last_error("the Hadamard pre-transform needs K %% 64 == 0 (K=%lld)", (long long)K);
        return RESQ_ERR_SHAPE;
    }
    if ((swiglu || gamma || rht) && pattern == RESQ_S_ROW50) {
        set_last_error("the fused producers do not support the row-wise selection");
        return RESQ_ERR_PATTERN;
    }
    if (gamma && (!aligned16(gamma) || !(eps >= 0.0f))) {
        set_last_error("rmsnorm: gamma needs a 16-byte aligned base and eps must be >= 0");
        return RESQ_ERR_ALIGN;
    }
    rc = check_pattern(pattern, M);
    if (rc) return rc;
    if (w_bf16) {
        if (!Y) {
            set_last_error("linear: NULL output pointer");
            return RESQ_ERR_NULL;
        }
        if (!aligned16(w_bf16) || ldw < K || ldw % 8 != 0) {
            set_last_error("linear: bf16 weights need a 16-byte aligned base, ldw >= K and 16-byte aligned rows");
            return RESQ_ERR_ALIGN;
        }
        w_codes = w_side = w_bf16;  // (only to pass the checks on the packed operands below)
    }
    if (!w_codes || !w_side || !Y) {
        set_last_error("linear: NULL weight or output pointer");
        return RESQ_ERR_NULL;
    }
    if (N <= 0) {
        set_last_error("linear: N=%lld", (long long)N);
        return RESQ_ERR_SHAPE;
    }
    if (out_dtype != RESQ_OUT_BF16 && out_dtype != RESQ_OUT_F32) {
        set_last_error("unknown output type %d", out_dtype);
        return RESQ_ERR_PATTERN;
    }
    if (!aligned16(Y) || !aligned16(w_codes) || !aligned16(w_side) || ldy < N ||
        ldy % (out_dtype == RESQ_OUT_BF16 ? 8 : 4) != 0) {
        set_last_error("linear: Y / weights need 16-byte aligned bases, ldy >= N and 16-byte aligned rows");
        return RESQ_ERR_ALIGN;
    }
    rc = check_workspace(workspace, ws_bytes, linear_workspace_bytes(fmt, M, N, K, pattern));
    if (rc) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    QuantArgs a;
    memset(&a, 0, sizeof(a));
    a.X = static_cast<const __nv_bfloat16*>(X);
    if (swiglu) a.X_up = a.X + K;
    a.M = M;
    a.K = K;
    a.ldx = ldx;
    a.pattern = pattern;
    a.keep_quarters = quarters;
    a.per_strip = per_strip;
    size_t used = 0;
    carve_quant_scratch(ws + kWsFlags, M, K, pattern, a, used);
    a.status = reinterpret_cast<DeviceStatus*>(ws);
    a.clear_words = reinterpret_cast<uint32_t*>(ws);  // cleared by the quantizer kernel: no separate memset node
    a.n_clear_words = (int)((kWsHeader + kWsFlags) / 4);
    used += kWsFlags;
    if (rht) {
        a.rht = 1;
        a.rht_signs = rht_signs;
    }
    // MXFP4 where it pays: the GEMM runs on the block-scaled FP4 pipe and takes packed codes and scales (they
    // fit into the space of the bf16 images; the selection zeroes dropped codes); otherwise exact bf16 images.
    const bool native = !w_bf16 && !swiglu && !gamma && !rht && fmt == kMXFP4 && gemm_mxfp4_native_supported(M, N, K, pattern != RESQ_S_NONE);
    uint8_t* region_a = ws + used;
    used += align_up((size_t)M * (size_t)K * 2, 256);
    uint8_t* region_r = nullptr;
    if (pattern != RESQ_S_NONE) {
        region_r = ws + used;
        used += residual_region_bytes(M, K, pattern);
    }
    if (gamma) {  // row scales of the fused RMSNorm producer: last region, behind the fp32 partial tiles
        a.gamma = static_cast<const __nv_bfloat16*>(gamma);
        a.eps = eps;
        a.row_scale = reinterpret_cast<float*>(ws + used + align_up(gemm_hif4_scratch_bytes(M, N, K), 256));
    }
    // 2:4 on the CTA-pair kernel: the residual goes to the structured-sparse MMA in compressed form
    const bool sparse24 = !w_bf16 && !swiglu && !gamma && !rht && !native && pattern == RESQ_S_2_4 && quarters == 2 &&
                          gemm_sparse24_supported(M, N, K);
    const size_t codes_bytes = align_up((size_t)M * (size_t)K / 2, 256);
    if (native) {
        a.x_codes = region_a;
        a.x_side = region_a + codes_bytes;
        if (region_r) {
            a.r_codes = region_r;
            a.r_side = region_r + codes_bytes;
            a.mask_r_codes = 1;
        }
    } else if (sparse24) {
        a.a_bf16 = reinterpret_cast<__nv_bfloat16*>(region_a);
        a.r_comp = reinterpret_cast<__nv_bfloat16*>(region_r);
        a.r_meta = region_r + align_up((size_t)M * (size_t)K, 256);
        a.meta_rows128 = sparse24_rows128(M);
        a.meta_ka = sparse24_ka(K);
    } else {
        a.a_bf16 = reinterpret_cast<__nv_bfloat16*>(region_a);
        a.r_bf16 = reinterpret_cast<__nv_bfloat16*>(region_r);
    }
    // block-wise selection on the CTA-pair kernel: the GEMM reads the keep flags, the image stays unmasked
    const bool block_lists = !native && pattern == RESQ_S_BLOCK32x64_50 && a.r_bf16 && gemm_block_lists_supported(M, N, K);
    a.skip_image_mask = block_lists ? 1 : 0;
    rc = launch_quantize(fmt, a, st);
    if (rc) return rc;
    if (native) {
        Mxfp4NativeArgs n;
        memset(&n, 0, sizeof(n));
        n.a_codes = a.x_codes;
        n.a_scale = static_cast<const uint8_t*>(a.x_side);
        n.r_codes = a.r_codes;
        n.r_scale = static_cast<const uint8_t*>(a.r_side);
        n.w_codes = static_cast<const uint8_t*>(w_codes);
        n.w_scale = static_cast<const uint8_t*>(w_side);
        n.M = M;
        n.N = N;
        n.K = K;
        n.Y = Y;
        n.out_dtype = out_dtype;
        n.ldy = ldy;
        n.partial_bytes = gemm_hif4_scratch_bytes(M, N, K);
        n.partials = n.partial_bytes ? reinterpret_cast<float*>(ws + used) : nullptr;
        n.status = a.status;
        return launch_gemm_mxfp4_native(n, st);
    }
    GemmArgs g;
    memset(&g, 0, sizeof(g));
    g.fmt = fmt;
    g.a_bf16 = a.a_bf16;
    g.r_bf16 = a.r_bf16;
    g.r_comp = a.r_comp;
    g.r_meta = a.r_meta;
    g.meta_rows128 = a.meta_rows128;
    g.meta_ka = a.meta_ka;
    g.blk_flags = block_lists ? a.keep_flags : nullptr;
    g.w_codes = static_cast<const uint8_t*>(w_codes);
    g.w_side = w_side;
    g.w_bf16 = static_cast<const __nv_bfloat16*>(w_bf16);
    g.ldw = ldw;
    g.M = M;
    g.N = N;
    g.K = K;
    g.Y = Y;
    g.out_dtype = out_dtype;
    g.ldy = ldy;
    g.partial_bytes = gemm_hif4_scratch_bytes(M, N, K);
    g.splitk_partials = g.partial_bytes ? reinterpret_cast<float*>(ws + used) : nullptr;
    g.splits = (int)(g.partial_bytes / ((size_t)M * (size_t)N * 4));
    g.sk_flags = reinterpret_cast<unsigned int*>(ws + kWsHeader);
    g.status = a.status;
    return launch_gemm_hif4(g, st);
}

// ---- a group of independent projections in one quantizer launch and one GEMM launch ---------------------------
// Workspace: [header | counters | per problem: image of deq Q(X), residual operand | fp32 partial-tile slots].
size_t group_workspace_bytes(const resq_problem* pr, int count, int pattern) {
    if (!pr || count < 1 || count > kMaxQuantGroup) return 0;
    size_t b = kWsHeader + kWsFlags;
    for (int i = 0; i < count; ++i) {
        if (pr[i].M <= 0 || pr[i].N <= 0 || pr[i].K <= 0) return 0;
        b += align_up((size_t)pr[i].M * (size_t)pr[i].K * 2, 256) + residual_region_bytes(pr[i].M, pr[i].K, pattern);
    }
    return b + align_up(gemm_pair_streamk_scratch_bytes(), 256);
}

int linear_group(int fmt, const resq_problem* pr, int count, int pattern, int out_dtype, void* workspace, size_t ws_bytes,
                 void* stream) {
    if (!pr) {
        set_last_error("linear_group: problems is NULL");
        return RESQ_ERR_NULL;
    }
    if (count < 1 || count > kMaxQuantGroup) {
        set_last_error("linear_group: a group holds 1 to %d problems (got %d)", kMaxQuantGroup, count);
        return RESQ_ERR_SHAPE;
    }
    int quarters = 2, per_strip = 0;
    int rc = split_pattern(&pattern, &quarters, &per_strip);
    if (rc) return rc;
    if (pattern != RESQ_S_NONE && pattern != RESQ_S_DENSE && pattern != RESQ_S_2_4) {
        set_last_error("linear_group takes the selections that are local to a token row (none, dense, n:4); the row-wise, "
                       "channel-wise and block-wise selections run through *_resq_linear");
        return RESQ_ERR_PATTERN;
    }
    if (out_dtype != RESQ_OUT_BF16 && out_dtype != RESQ_OUT_F32) {
        set_last_error("unknown output type %d", out_dtype);
        return RESQ_ERR_PATTERN;
    }
    for (int i = 0; i < count; ++i) {
        rc = check_matrix(pr[i].X_bf16, pr[i].M, pr[i].K, pr[i].ldx, fmt, "X");
        if (rc) return rc;
        if (!pr[i].w_codes || !pr[i].w_side || !pr[i].Y) {
            set_last_error("linear_group: NULL weight or output pointer in problem %d", i);
            return RESQ_ERR_NULL;
        }
        if (pr[i].N <= 0) {
            set_last_error("linear_group: N=%lld in problem %d", (long long)pr[i].N, i);
            return RESQ_ERR_SHAPE;
        }
        if (!aligned16(pr[i].Y) || !aligned16(pr[i].w_codes) || !aligned16(pr[i].w_side) || pr[i].ldy < pr[i].N ||
            pr[i].ldy % (out_dtype == RESQ_OUT_BF16 ? 8 : 4) != 0) {
            set_last_error("linear_group: Y / weights need 16-byte aligned bases, ldy >= N and 16-byte aligned rows (problem %d)", i);
            return RESQ_ERR_ALIGN;
        }
    }
    rc = check_workspace(workspace, ws_bytes, group_workspace_bytes(pr, count, pattern));
    if (rc) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    QuantArgs qa[kMaxQuantGroup];
    GemmArgs ga[kMaxQuantGroup];
    size_t used = kWsHeader + kWsFlags;
    // (the residual operand of a group is the dense masked image: the compressed 2:4 form pays from a few thousand token
    // rows on, which is not what groups are for)
    for (int i = 0; i < count; ++i) {
        QuantArgs& a = qa[i];
        memset(&a, 0, sizeof(a));
        a.X = static_cast<const __nv_bfloat16*>(pr[i].X_bf16);
        a.M = pr[i].M;
        a.K = pr[i].K;
        a.ldx = pr[i].ldx;
        a.pattern = pattern;
        a.keep_quarters = quarters;
        a.status = reinterpret_cast<DeviceStatus*>(ws);
        if (i == 0) {  // cleared by the quantizer kernel: no separate memset node
            a.clear_words = reinterpret_cast<uint32_t*>(ws);
            a.n_clear_words = (int)((kWsHeader + kWsFlags) / 4);
        }
        a.a_bf16 = reinterpret_cast<__nv_bfloat16*>(ws + used);
        used += align_up((size_t)a.M * (size_t)a.K * 2, 256);
        if (pattern != RESQ_S_NONE) {
            uint8_t* region_r = ws + used;
            used += residual_region_bytes(a.M, a.K, pattern);
            a.r_bf16 = reinterpret_cast<__nv_bfloat16*>(region_r);
        }
    }
    for (int i = 0; i < count; ++i) {
        GemmArgs& g = ga[i];
        memset(&g, 0, sizeof(g));
        g.fmt = fmt;
        g.a_bf16 = qa[i].a_bf16;
        g.r_bf16 = qa[i].r_bf16;
        g.r_comp = qa[i].r_comp;
        g.r_meta = qa[i].r_meta;
        g.meta_rows128 = qa[i].meta_rows128;
        g.meta_ka = qa[i].meta_ka;
        g.w_codes = static_cast<const uint8_t*>(pr[i].w_codes);
        g.w_side = pr[i].w_side;
        g.M = pr[i].M;
        g.N = pr[i].N;
        g.K = pr[i].K;
        g.Y = pr[i].Y;
        g.out_dtype = out_dtype;
        g.ldy = pr[i].ldy;
        g.partial_bytes = gemm_pair_streamk_scratch_bytes();
        g.splitk_partials = reinterpret_cast<float*>(ws + used);
        g.sk_flags = reinterpret_cast<unsigned int*>(ws + kWsHeader);
        g.status = reinterpret_cast<DeviceStatus*>(ws);
    }
    rc = launch_quantize_group(fmt, qa, count, st);
    if (rc) return rc;
    if (gemm_decode_supported(ga, count)) return launch_gemm_decode(ga, count, st);
    return launch_gemm_pair_group(ga, count, st);
}

// ---- backward products of the layer (training side) ---------------------------------------------------------------
// Both are Eq. (1) on transposed operands: the quantization blocks run along the product's own contraction axis.
size_t transposed_bytes(int64_t rows, int64_t cols) { return align_up((size_t)rows * (size_t)cols * 2, 256); }

int pack_weight_transposed(int fmt, const void* W, int64_t N, int64_t K, int64_t ldw, void* wt_codes, void* wt_side, void* workspace,
                           size_t ws_bytes, void* stream) {
    // W [N, K] -> Q(W^T): K rows of N values, blocks along N
    if (!W || !wt_codes || !wt_side) {
        set_last_error("pack_weight_transposed: NULL pointer");
        return RESQ_ERR_NULL;
    }
    if (N <= 0 || K <= 0 || N % block_of(fmt) != 0) {
        set_last_error("pack_weight_transposed: N=%lld K=%lld (N must be a positive multiple of %d)", (long long)N, (long long)K,
                       block_of(fmt));
        return RESQ_ERR_SHAPE;
    }
    if (!aligned16(W) || ldw < K || ldw % 8 != 0 || N % 8 != 0) {
        set_last_error("pack_weight_transposed: W needs a 16-byte aligned base, ldw >= K, ldw %% 8 == 0");
        return RESQ_ERR_ALIGN;
    }
    int rc = check_packed_outputs(wt_codes, wt_side, nullptr, nullptr);
    if (rc) return rc;
    rc = check_workspace(workspace, ws_bytes, transposed_bytes(K, N));
    if (rc) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    __nv_bfloat16* wt = static_cast<__nv_bfloat16*>(workspace);
    rc = launch_transpose_bf16(static_cast<const __nv_bfloat16*>(W), N, K, ldw, wt, N, st);
    if (rc) return rc;
    return quantize_only(fmt, wt, K, N, N, wt_codes, wt_side, stream, "W^T");
}

size_t wgrad_workspace_bytes(int fmt, int64_t M, int64_t N, int64_t K) {
    if (M <= 0 || N <= 0 || K <= 0) return 0;
    const size_t side = fmt == kHiF4 ? (size_t)K * (size_t)(M / kHif4Block) * 4 : (size_t)K * (size_t)(M / kMxBlock);
    return linear_workspace_bytes(fmt, N, K, M, RESQ_S_NONE) + transposed_bytes(N, M) + transposed_bytes(K, M) +
           align_up((size_t)K * (size_t)M / 2, 256) + align_up(side, 256);
}

int wgrad_linear(int fmt, const void* dY, const void* X, int64_t M, int64_t N, int64_t K, int64_t lddy, int64_t ldx, void* dW,
                 int out_dtype, int64_t lddw, void* workspace, size_t ws_bytes, void* stream) {
    if (!dY || !X || !dW) {
        set_last_error("wgrad_linear: NULL pointer");
        return RESQ_ERR_NULL;
    }
    if (M <= 0 || N <= 0 || K <= 0 || M % block_of(fmt) != 0) {
        set_last_error("wgrad_linear: M=%lld N=%lld K=%lld (the contraction runs over M: a positive multiple of %d)", (long long)M,
                       (long long)N, (long long)K, block_of(fmt));
        return RESQ_ERR_SHAPE;
    }
    if (!aligned16(dY) || !aligned16(X) || lddy < N || ldx < K || lddy % 8 != 0 || ldx % 8 != 0 || M % 8 != 0) {
        set_last_error("wgrad_linear: dY / X need 16-byte aligned bases and row pitches that are multiples of 8 and cover the rows");
        return RESQ_ERR_ALIGN;
    }
    int rc = check_workspace(workspace, ws_bytes, wgrad_workspace_bytes(fmt, M, N, K));
    if (rc) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    size_t used = linear_workspace_bytes(fmt, N, K, M, RESQ_S_NONE);
    __nv_bfloat16* gt = reinterpret_cast<__nv_bfloat16*>(ws + used);   // dY^T [N, M]
    used += transposed_bytes(N, M);
    __nv_bfloat16* xt = reinterpret_cast<__nv_bfloat16*>(ws + used);   // X^T [K, M]
    used += transposed_bytes(K, M);
    uint8_t* xt_codes = ws + used;
    used += align_up((size_t)K * (size_t)M / 2, 256);
    void* xt_side = ws + used;
    rc = launch_transpose_bf16(static_cast<const __nv_bfloat16*>(dY), M, N, lddy, gt, M, st);
    if (rc) return rc;
    rc = launch_transpose_bf16(static_cast<const __nv_bfloat16*>(X), M, K, ldx, xt, M, st);
    if (rc) return rc;
    rc = quantize_only(fmt, xt, K, M, M, xt_codes, xt_side, stream, "X^T");
    if (rc) return rc;
    // dW^ [N, K] = Q(dY^T) Q(X^T)^T: the layer call with dY^T as its activation and Q(X^T) as its packed operand
    return linear(fmt, gt, N, M, M, xt_codes, xt_side, K, RESQ_S_NONE, dW, out_dtype, lddw, workspace, ws_bytes, stream);
}

// Weight-only variant (Table 1, "W4A16"): Y = X deq(Q(W))^T with the bf16 activations used as they are.
// Workspace: [header | counters | fp32 partial tiles].
size_t w4a16_workspace_bytes(int64_t M, int64_t N, int64_t K) {
    if (M <= 0 || N <= 0 || K <= 0) return 0;
    return kWsHeader + kWsFlags + align_up(gemm_hif4_scratch_bytes(M, N, K), 256);
}

int w4a16_linear(int fmt, const void* X, int64_t M, int64_t K, int64_t ldx, const void* w_codes, const void* w_side, int64_t N,
                 void* Y, int out_dtype, int64_t ldy, void* workspace, size_t ws_bytes, void* stream) {
    int rc = check_matrix(X, M, K, ldx, fmt, "X");
    if (rc) return rc;
    if (!w_codes || !w_side || !Y) {
        set_last_error("w4a16_linear: NULL weight or output pointer");
        return RESQ_ERR_NULL;
    }
    if (N <= 0) {
        set_last_error("w4a16_linear: N=%lld", (long long)N);
        return RESQ_ERR_SHAPE;
    }
    if (out_dtype != RESQ_OUT_BF16 && out_dtype != RESQ_OUT_F32) {
        set_last_error("unknown output type %d", out_dtype);
        return RESQ_ERR_PATTERN;
    }
    if (!aligned16(Y) || !aligned16(w_codes) || !aligned16(w_side) || ldy < N ||
        ldy % (out_dtype == RESQ_OUT_BF16 ? 8 : 4) != 0) {
        set_last_error("w4a16_linear: Y / weights need 16-byte aligned bases, ldy >= N and 16-byte aligned rows");
        return RESQ_ERR_ALIGN;
    }
    rc = check_workspace(workspace, ws_bytes, w4a16_workspace_bytes(M, N, K));
    if (rc) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemsetAsync(workspace, 0, kWsHeader + kWsFlags, st);  // no quantizer kernel to clear it
    if (e != cudaSuccess) return cuda_fail(e, "cudaMemsetAsync(status)");
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    GemmArgs g;
    memset(&g, 0, sizeof(g));
    g.fmt = fmt;
    g.a_bf16 = static_cast<const __nv_bfloat16*>(X);
    g.r_bf16 = nullptr;
    g.lda = ldx;
    g.w_codes = static_cast<const uint8_t*>(w_codes);
    g.w_side = w_side;
    g.M = M;
    g.N = N;
    g.K = K;
    g.Y = Y;
    g.out_dtype = out_dtype;
    g.ldy = ldy;
    g.partial_bytes = gemm_hif4_scratch_bytes(M, N, K);
    g.splitk_partials = g.partial_bytes ? reinterpret_cast<float*>(ws + kWsHeader + kWsFlags) : nullptr;
    g.splits = (int)(g.partial_bytes / ((size_t)M * (size_t)N * 4));
    g.sk_flags = reinterpret_cast<unsigned int*>(ws + kWsHeader);
    g.status = reinterpret_cast<DeviceStatus*>(ws);
    return launch_gemm_hif4(g, st);
}

// "W4A8" (Table 1): 8-bit activations (MXFP8-E4M3, see include/resq.h) against the packed 4-bit weights.
// Workspace: [header | counters | bf16 image of the decoded activations | fp32 partial tiles].
size_t w4a8_workspace_bytes(int64_t M, int64_t N, int64_t K) {
    if (M <= 0 || N <= 0 || K <= 0) return 0;
    return kWsHeader + kWsFlags + align_up((size_t)M * (size_t)K * 2, 256) + align_up(gemm_hif4_scratch_bytes(M, N, K), 256);
}

int w4a8_linear(int fmt, const void* X, int64_t M, int64_t K, int64_t ldx, const void* w_codes, const void* w_side, int64_t N,
                void* Y, int out_dtype, int64_t ldy, void* workspace, size_t ws_bytes, void* stream) {
    int rc = check_matrix(X, M, K, ldx, fmt, "X");
    if (rc) return rc;
    if (K % 32 != 0) {
        set_last_error("w4a8_linear: K must be a multiple of 32 (K=%lld)", (long long)K);
        return RESQ_ERR_SHAPE;
    }
    if (!w_codes || !w_side || !Y) {
        set_last_error("w4a8_linear: NULL weight or output pointer");
        return RESQ_ERR_NULL;
    }
    if (N <= 0) {
        set_last_error("w4a8_linear: N=%lld", (long long)N);
        return RESQ_ERR_SHAPE;
    }
    if (out_dtype != RESQ_OUT_BF16 && out_dtype != RESQ_OUT_F32) {
        set_last_error("unknown output type %d", out_dtype);
        return RESQ_ERR_PATTERN;
    }
    if (!aligned16(Y) || !aligned16(w_codes) || !aligned16(w_side) || ldy < N ||
        ldy % (out_dtype == RESQ_OUT_BF16 ? 8 : 4) != 0) {
        set_last_error("w4a8_linear: Y / weights need 16-byte aligned bases, ldy >= N and 16-byte aligned rows");
        return RESQ_ERR_ALIGN;
    }
    rc = check_workspace(workspace, ws_bytes, w4a8_workspace_bytes(M, N, K));
    if (rc) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    __nv_bfloat16* img = reinterpret_cast<__nv_bfloat16*>(ws + kWsHeader + kWsFlags);
    rc = launch_quantize_mxfp8_image(static_cast<const __nv_bfloat16*>(X), M, K, ldx, img, reinterpret_cast<uint32_t*>(ws),
                                     (int)((kWsHeader + kWsFlags) / 4), st);
    if (rc) return rc;
    GemmArgs g;
    memset(&g, 0, sizeof(g));
    g.fmt = fmt;
    g.a_bf16 = img;
    g.w_codes = static_cast<const uint8_t*>(w_codes);
    g.w_side = w_side;
    g.M = M;
    g.N = N;
    g.K = K;
    g.Y = Y;
    g.out_dtype = out_dtype;
    g.ldy = ldy;
    g.partial_bytes = gemm_hif4_scratch_bytes(M, N, K);
    g.splitk_partials = g.partial_bytes ? reinterpret_cast<float*>(ws + kWsHeader + kWsFlags + align_up((size_t)M * (size_t)K * 2, 256))
                                        : nullptr;
    g.splits = (int)(g.partial_bytes / ((size_t)M * (size_t)N * 4));
    g.sk_flags = reinterpret_cast<unsigned int*>(ws + kWsHeader);
    g.status = reinterpret_cast<DeviceStatus*>(ws);
    return launch_gemm_hif4(g, st);
}

}  // namespace
}  // namespace resq

using namespace resq;

extern "C" {

size_t hif4_codes_bytes(int64_t rows, int64_t K) { return rows > 0 && K > 0 ? (size_t)rows * (size_t)K / 2 : 0; }
size_t hif4_meta_bytes(int64_t rows, int64_t K) { return rows > 0 && K > 0 ? (size_t)rows * (size_t)(K / kHif4Block) * 4 : 0; }
size_t mxfp4_codes_bytes(int64_t rows, int64_t K) { return rows > 0 && K > 0 ? (size_t)rows * (size_t)K / 2 : 0; }
size_t mxfp4_scale_bytes(int64_t rows, int64_t K) { return rows > 0 && K > 0 ? (size_t)rows * (size_t)(K / kMxBlock) : 0; }
size_t resq_mask_bytes(int64_t M, int64_t K) { return M > 0 && K > 0 ? (size_t)M * (size_t)K / 8 : 0; }

size_t resq_residual_mask_workspace_bytes(int64_t M, int64_t K, int pattern) {
    if (M <= 0 || K <= 0) return kWsHeader;
    return kWsHeader + quant_scratch_bytes(M, K, base_pattern(pattern));
}
size_t hif4_resq_workspace_bytes(int64_t M, int64_t N, int64_t K, int pattern) {
    return linear_workspace_bytes(kHiF4, M, N, K, base_pattern(pattern));
}
size_t mxfp4_resq_workspace_bytes(int64_t M, int64_t N, int64_t K, int pattern) {
    return linear_workspace_bytes(kMXFP4, M, N, K, base_pattern(pattern));
}

int hif4_pack_weight(const void* W, int64_t N, int64_t K, int64_t ldw, void* w_codes, void* w_meta, void* stream) {
    return quantize_only(kHiF4, W, N, K, ldw, w_codes, w_meta, stream, "W");
}
int mxfp4_pack_weight(const void* W, int64_t N, int64_t K, int64_t ldw, void* w_codes, void* w_scale, void* stream) {
    return quantize_only(kMXFP4, W, N, K, ldw, w_codes, w_scale, stream, "W");
}
int hif4_quantize_act(const void* X, int64_t M, int64_t K, int64_t ldx, void* x_codes, void* x_meta, void* stream) {
    return quantize_only(kHiF4, X, M, K, ldx, x_codes, x_meta, stream, "X");
}
int mxfp4_quantize_act(const void* X, int64_t M, int64_t K, int64_t ldx, void* x_codes, void* x_scale, void* stream) {
    return quantize_only(kMXFP4, X, M, K, ldx, x_codes, x_scale, stream, "X");
}
int hif4_dequantize(const void* codes, const void* meta, int64_t rows, int64_t K, float* out, void* stream) {
    return dequantize(kHiF4, codes, meta, rows, K, out, stream);
}
int mxfp4_dequantize(const void* codes, const void* scale, int64_t rows, int64_t K, float* out, void* stream) {
    return dequantize(kMXFP4, codes, scale, rows, K, out, stream);
}

int resq_residual_mask(const void* X, int64_t M, int64_t K, int64_t ldx, int pattern, void* x_codes, void* x_meta,
                       void* r_codes, void* r_meta, void* mask_bits, void* workspace, size_t ws_bytes, void* stream) {
    return residual_mask(kHiF4, X, M, K, ldx, pattern, x_codes, x_meta, r_codes, r_meta, mask_bits, workspace, ws_bytes,
                         stream);
}
int mxfp4_residual_mask(const void* X, int64_t M, int64_t K, int64_t ldx, int pattern, void* x_codes, void* x_scale,
                        void* r_codes, void* r_scale, void* mask_bits, void* workspace, size_t ws_bytes, void* stream) {
    return residual_mask(kMXFP4, X, M, K, ldx, pattern, x_codes, x_scale, r_codes, r_scale, mask_bits, workspace,
                         ws_bytes, stream);
}

int hif4_swiglu_resq_linear(const void* GU, int64_t M, int64_t K, int64_t ldgu, const void* w_codes, const void* w_meta,
                            int64_t N, int pattern, void* Y, int out_dtype, int64_t ldy, void* workspace, size_t ws_bytes,
                            void* stream) {
    return linear(kHiF4, GU, M, K, ldgu, w_codes, w_meta, N, pattern, Y, out_dtype, ldy, workspace, ws_bytes, stream, nullptr, 0,
                  true);
}
int mxfp4_swiglu_resq_linear(const void* GU, int64_t M, int64_t K, int64_t ldgu, const void* w_codes, const void* w_scale,
                             int64_t N, int pattern, void* Y, int out_dtype, int64_t ldy, void* workspace, size_t ws_bytes,
                             void* stream) {
    return linear(kMXFP4, GU, M, K, ldgu, w_codes, w_scale, N, pattern, Y, out_dtype, ldy, workspace, ws_bytes, stream, nullptr,
                  0, true);
}

int hif4_rht_pack_weight(const void* W, int64_t N, int64_t K, int64_t ldw, unsigned long long signs, void* w_codes, void* w_meta,
                         void* stream) {
    return quantize_only(kHiF4, W, N, K, ldw, w_codes, w_meta, stream, "W", true, signs);
}
int mxfp4_rht_pack_weight(const void* W, int64_t N, int64_t K, int64_t ldw, unsigned long long signs, void* w_codes, void* w_scale,
                          void* stream) {
    return quantize_only(kMXFP4, W, N, K, ldw, w_codes, w_scale, stream, "W", true, signs);
}
int hif4_rht_resq_linear(const void* X, int64_t M, int64_t K, int64_t ldx, unsigned long long signs, const void* w_codes,
                         const void* w_meta, int64_t N, int pattern, void* Y, int out_dtype, int64_t ldy, void* workspace,
                         size_t ws_bytes, void* stream) {
    return linear(kHiF4, X, M, K, ldx, w_codes, w_meta, N, pattern, Y, out_dtype, ldy, workspace, ws_bytes, stream, nullptr, 0,
                  false, nullptr, 0.0f, true, signs);
}
int mxfp4_rht_resq_linear(const void* X, int64_t M, int64_t K, int64_t ldx, unsigned long long signs, const void* w_codes,
                          const void* w_scale, int64_t N, int pattern, void* Y, int out_dtype, int64_t ldy, void* workspace,
                          size_t ws_bytes, void* stream) {
    return linear(kMXFP4, X, M, K, ldx, w_codes, w_scale, N, pattern, Y, out_dtype, ldy, workspace, ws_bytes, stream, nullptr, 0,
                  false, nullptr, 0.0f, true, signs);
}

int hif4_rmsnorm_resq_linear(const void* H, int64_t M, int64_t K, int64_t ldh, const void* gamma, float eps, const void* w_codes,
                             const void* w_meta, int64_t N, int pattern, void* Y, int out_dtype, int64_t ldy, void* workspace,
                             size_t ws_bytes, void* stream) {
    if (!gamma) {
        set_last_error("rmsnorm_resq_linear: NULL gamma");
        return RESQ_ERR_NULL;
    }
    return linear(kHiF4, H, M, K, ldh, w_codes, w_meta, N, pattern, Y, out_dtype, ldy, workspace, ws_bytes, stream, nullptr, 0,
                  false, gamma, eps);
}
int mxfp4_rmsnorm_resq_linear(const void* H, int64_t M, int64_t K, int64_t ldh, const void* gamma, float eps, const void* w_codes,
                              const void* w_scale, int64_t N, int pattern, void* Y, int out_dtype, int64_t ldy, void* workspace,
                              size_t ws_bytes, void* stream) {
    if (!gamma) {
        set_last_error("rmsnorm_resq_linear: NULL gamma");
        return RESQ_ERR_NULL;
    }
    return linear(kMXFP4, H, M, K, ldh, w_codes, w_scale, N, pattern, Y, out_dtype, ldy, workspace, ws_bytes, stream, nullptr, 0,
                  false, gamma, eps);
}

int hif4_w16a4_linear(const void* X, int64_t M, int64_t K, int64_t ldx, const void* W, int64_t N, int64_t ldw, int pattern,
                      void* Y, int out_dtype, int64_t ldy, void* workspace, size_t ws_bytes, void* stream) {
    if (!W) {
        set_last_error("w16a4_linear: NULL weight pointer");
        return RESQ_ERR_NULL;
    }
    return linear(kHiF4, X, M, K, ldx, nullptr, nullptr, N, pattern, Y, out_dtype, ldy, workspace, ws_bytes, stream, W, ldw);
}
int mxfp4_w16a4_linear(const void* X, int64_t M, int64_t K, int64_t ldx, const void* W, int64_t N, int64_t ldw, int pattern,
                       void* Y, int out_dtype, int64_t ldy, void* workspace, size_t ws_bytes, void* stream) {
    if (!W) {
        set_last_error("w16a4_linear: NULL weight pointer");
        return RESQ_ERR_NULL;
    }
    return linear(kMXFP4, X, M, K, ldx, nullptr, nullptr, N, pattern, Y, out_dtype, ldy, workspace, ws_bytes, stream, W, ldw);
}

size_t resq_w4a8_workspace_bytes(int64_t M, int64_t N, int64_t K) { return w4a8_workspace_bytes(M, N, K); }
int hif4_w4a8_linear(const void* X, int64_t M, int64_t K, int64_t ldx, const void* w_codes, const void* w_meta, int64_t N, void* Y,
                     int out_dtype, int64_t ldy, void* workspace, size_t ws_bytes, void* stream) {
    return w4a8_linear(kHiF4, X, M, K, ldx, w_codes, w_meta, N, Y, out_dtype, ldy, workspace, ws_bytes, stream);
}
int mxfp4_w4a8_linear(const void* X, int64_t M, int64_t K, int64_t ldx, const void* w_codes, const void* w_scale, int64_t N, void* Y,
                      int out_dtype, int64_t ldy, void* workspace, size_t ws_bytes, void* stream) {
    return w4a8_linear(kMXFP4, X, M, K, ldx, w_codes, w_scale, N, Y, out_dtype, ldy, workspace, ws_bytes, stream);
}

size_t resq_w4a16_workspace_bytes(int64_t M, int64_t N, int64_t K) { return w4a16_workspace_bytes(M, N, K); }
int hif4_w4a16_linear(const void* X, int64_t M, int64_t K, int64_t ldx, const void* w_codes, const void* w_meta, int64_t N,
                      void* Y, int out_dtype, int64_t ldy, void* workspace, size_t ws_bytes, void* stream) {
    return w4a16_linear(kHiF4, X, M, K, ldx, w_codes, w_meta, N, Y, out_dtype, ldy, workspace, ws_bytes, stream);
}
int mxfp4_w4a16_linear(const void* X, int64_t M, int64_t K, int64_t ldx, const void* w_codes, const void* w_scale, int64_t N,
                       void* Y, int out_dtype, int64_t ldy, void* workspace, size_t ws_bytes, void* stream) {
    return w4a16_linear(kMXFP4, X, M, K, ldx, w_codes, w_scale, N, Y, out_dtype, ldy, workspace, ws_bytes, stream);
}

int hif4_resq_linear(const void* X, int64_t M, int64_t K, int64_t ldx, const void* w_codes, const void* w_meta, int64_t N,
                     int pattern, void* Y, int out_dtype, int64_t ldy, void* workspace, size_t ws_bytes, void* stream) {
    return linear(kHiF4, X, M, K, ldx, w_codes, w_meta, N, pattern, Y, out_dtype, ldy, workspace, ws_bytes, stream);
}
int mxfp4_resq_linear(const void* X, int64_t M, int64_t K, int64_t ldx, const void* w_codes, const void* w_scale,
                      int64_t N, int pattern, void* Y, int out_dtype, int64_t ldy, void* workspace, size_t ws_bytes,
                      void* stream) {
    return linear(kMXFP4, X, M, K, ldx, w_codes, w_scale, N, pattern, Y, out_dtype, ldy, workspace, ws_bytes, stream);
}

size_t hif4_resq_group_workspace_bytes(const resq_problem* problems, int count, int pattern) {
    return group_workspace_bytes(problems, count, base_pattern(pattern));
}
size_t mxfp4_resq_group_workspace_bytes(const resq_problem* problems, int count, int pattern) {
    return group_workspace_bytes(problems, count, base_pattern(pattern));
}
int hif4_resq_linear_group(const resq_problem* problems, int count, int pattern, int out_dtype, void* workspace, size_t ws_bytes,
                           void* stream) {
    return linear_group(kHiF4, problems, count, pattern, out_dtype, workspace, ws_bytes, stream);
}
int mxfp4_resq_linear_group(const resq_problem* problems, int count, int pattern, int out_dtype, void* workspace, size_t ws_bytes,
                            void* stream) {
    return linear_group(kMXFP4, problems, count, pattern, out_dtype, workspace, ws_bytes, stream);
}

size_t resq_transposed_workspace_bytes(int64_t N, int64_t K) { return N > 0 && K > 0 ? transposed_bytes(K, N) : 0; }
int hif4_pack_weight_transposed(const void* W, int64_t N, int64_t K, int64_t ldw, void* wt_codes, void* wt_meta, void* workspace,
                                size_t ws_bytes, void* stream) {
    return pack_weight_transposed(kHiF4, W, N, K, ldw, wt_codes, wt_meta, workspace, ws_bytes, stream);
}
int mxfp4_pack_weight_transposed(const void* W, int64_t N, int64_t K, int64_t ldw, void* wt_codes, void* wt_scale, void* workspace,
                                 size_t ws_bytes, void* stream) {
    return pack_weight_transposed(kMXFP4, W, N, K, ldw, wt_codes, wt_scale, workspace, ws_bytes, stream);
}
size_t hif4_dgrad_workspace_bytes(int64_t M, int64_t N, int64_t K) { return linear_workspace_bytes(kHiF4, M, K, N, RESQ_S_NONE); }
size_t mxfp4_dgrad_workspace_bytes(int64_t M, int64_t N, int64_t K) { return linear_workspace_bytes(kMXFP4, M, K, N, RESQ_S_NONE); }
int hif4_dgrad_linear(const void* dY, int64_t M, int64_t N, int64_t lddy, const void* wt_codes, const void* wt_meta, int64_t K, void* dX,
                      int out_dtype, int64_t lddx, void* workspace, size_t ws_bytes, void* stream) {
    return linear(kHiF4, dY, M, N, lddy, wt_codes, wt_meta, K, RESQ_S_NONE, dX, out_dtype, lddx, workspace, ws_bytes, stream);
}
int mxfp4_dgrad_linear(const void* dY, int64_t M, int64_t N, int64_t lddy, const void* wt_codes, const void* wt_scale, int64_t K, void* dX,
                       int out_dtype, int64_t lddx, void* workspace, size_t ws_bytes, void* stream) {
    return linear(kMXFP4, dY, M, N, lddy, wt_codes, wt_scale, K, RESQ_S_NONE, dX, out_dtype, lddx, workspace, ws_bytes, stream);
}
size_t hif4_wgrad_workspace_bytes(int64_t M, int64_t N, int64_t K) { return wgrad_workspace_bytes(kHiF4, M, N, K); }
size_t mxfp4_wgrad_workspace_bytes(int64_t M, int64_t N, int64_t K) { return wgrad_workspace_bytes(kMXFP4, M, N, K); }
int hif4_wgrad_linear(const void* dY, const void* X, int64_t M, int64_t N, int64_t K, int64_t lddy, int64_t ldx, void* dW, int out_dtype,
                      int64_t lddw, void* workspace, size_t ws_bytes, void* stream) {
    return wgrad_linear(kHiF4, dY, X, M, N, K, lddy, ldx, dW, out_dtype, lddw, workspace, ws_bytes, stream);
}
int mxfp4_wgrad_linear(const void* dY, const void* X, int64_t M, int64_t N, int64_t K, int64_t lddy, int64_t ldx, void* dW, int out_dtype,
                       int64_t lddw, void* workspace, size_t ws_bytes, void* stream) {
    return wgrad_linear(kMXFP4, dY, X, M, N, K, lddy, ldx, dW, out_dtype, lddw, workspace, ws_bytes, stream);
}

int resq_check(void* workspace, void* stream) {
    if (!workspace) {
        set_last_error("resq_check: workspace is NULL");
        return RESQ_ERR_NULL;
    }
    cudaError_t e = cudaStreamSynchronize(static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(e, "cudaStreamSynchronize");
    DeviceStatus st;
    e = cudaMemcpy(&st, workspace, sizeof(st), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return cuda_fail(e, "cudaMemcpy(status)");
    if (st.code != RESQ_OK) set_last_error("device status %d (wait %d gave up in block %d)", st.code, st.where, st.block);
    return st.code;
}

const char* resq_last_error(void) { return g_last_error; }

int resq_debug_expire_next_wait(int on) {
    debug_expire_next_wait(on);
    return RESQ_OK;
}

int64_t resq_kernel_launches(void) { return (int64_t)g_launches.load(); }

int resq_profile_enable(int on) {
    g_profile.store(on ? 1 : 0);
    return RESQ_OK;
}

int resq_profile_read(double* ms_by_kind, int64_t* launches_by_kind) {
    std::vector<ProfRec*> recs;
    {
        std::lock_guard<std::mutex> lk(g_prof_mu);
        recs.swap(g_prof);
    }
    for (int k = 0; k < kNumKinds; ++k) {
        if (ms_by_kind) ms_by_kind[k] = 0.0;
        if (launches_by_kind) launches_by_kind[k] = 0;
    }
    int rc = RESQ_OK;
    for (ProfRec* r : recs) {
        float ms = 0.0f;
        cudaError_t e = cudaEventSynchronize(r->stop);
        if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, r->start, r->stop);
        if (e != cudaSuccess) rc = cuda_fail(e, "profile event");
        else {
            if (ms_by_kind) ms_by_kind[r->kind] += (double)ms;
            if (launches_by_kind) launches_by_kind[r->kind] += 1;
        }
        cudaEventDestroy(r->start);
        cudaEventDestroy(r->stop);
        delete r;
    }
    return rc;
}

}  // extern "C"
