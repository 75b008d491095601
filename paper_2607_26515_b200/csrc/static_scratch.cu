// resq_residual_mask_static: the residual / mask pass for callers that cannot allocate device memory.
//
// Some hosts of this library have no way to hand it a workspace: an inference server that gave the whole
// device to its own memory pool at start-up (a later cudaMalloc would fail or fragment the pool), a plugin
// that is called from inside a serving loop where any allocation would synchronise the device, or a thin
// foreign-function caller that owns nothing but its input and output buffers.  For them the scratch of the
// channel-wise and block-wise selections (fp64 scores and keep flags) lives in a fixed array that is part of
// the library image itself.  Every GPU that loads the library holds these bytes until the process exits.
#include "common.cuh"

#include <cstring>
#include <mutex>

namespace resq {
namespace {

constexpr size_t kStaticMaxScores = RESQ_STATIC_SCRATCH_MAX_SCORES;
// layout: [256-byte header | scores: kStaticMaxScores doubles | keep flags: kStaticMaxScores bytes]
constexpr size_t kStaticBytes = kWsHeader + kStaticMaxScores * sizeof(double) + kStaticMaxScores;

static __device__ __align__(256) unsigned char g_static_scratch[kStaticBytes];

// In host code `g_static_scratch` is only a stand-in for the symbol, never a device address: the address
// has to be asked for, once per device, with that device current.
constexpr int kMaxDevices = 64;
std::mutex g_mu;
unsigned char* g_dev_ptr[kMaxDevices] = {nullptr};

int static_scratch_for_current_device(unsigned char** out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e, "cudaGetDevice");
    if (dev < 0 || dev >= kMaxDevices) {
        set_last_error("device ordinal %d is outside the supported range 0..%d", dev, kMaxDevices - 1);
        return RESQ_ERR_CUDA;
    }
    std::lock_guard<std::mutex> lk(g_mu);
    if (!g_dev_ptr[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess) return cuda_fail(e, "cudaGetSymbolAddress(static scratch)");
        g_dev_ptr[dev] = static_cast<unsigned char*>(p);
    }
    *out = g_dev_ptr[dev];
    return RESQ_OK;
}

}  // namespace
}  // namespace resq

using namespace resq;

extern "C" int resq_residual_mask_static(const void* X, int64_t M, int64_t K, int64_t ldx, int pattern, void* x_codes,
                                         void* x_meta, void* r_codes, void* r_meta, void* mask_bits, void* stream) {
    if (!X) {
        set_last_error("X is NULL");
        return RESQ_ERR_NULL;
    }
    if (M <= 0 || K <= 0 || K % kHif4Block != 0) {
        set_last_error("X: M=%lld K=%lld (K must be a positive multiple of %d)", (long long)M, (long long)K, kHif4Block);
        return RESQ_ERR_SHAPE;
    }
    if ((reinterpret_cast<uintptr_t>(X) & 15u) != 0 || ldx < K || ldx % 8 != 0) {
        set_last_error("X: needs a 16-byte aligned base and ld >= K, ld %% 8 == 0 (ld=%lld)", (long long)ldx);
        return RESQ_ERR_ALIGN;
    }
    // the same pattern rules as resq_residual_mask: RESQ_KEEP_QUARTERS and RESQ_BLOCK_PER_STRIP are honoured
    int quarters = 2, per_strip = 0;
    int rc = split_pattern(&pattern, &quarters, &per_strip);
    if (rc) return rc;
    rc = check_pattern(pattern, M);
    if (rc) return rc;
    rc = check_packed_outputs(x_codes, x_meta, r_codes, r_meta);
    if (rc) return rc;
    size_t nscores = 0;
    if (pattern == RESQ_S_CHAN50) nscores = (size_t)K;
    if (pattern == RESQ_S_BLOCK32x64_50) nscores = (size_t)(M / kBlkRows) * (size_t)(K / kBlkCols);
    if (nscores > kStaticMaxScores) {
        set_last_error("resq_residual_mask_static: this selection needs %zu scores but the built-in scratch holds %zu "
                       "(RESQ_STATIC_SCRATCH_MAX_SCORES); use resq_residual_mask with a caller workspace",
                       nscores, kStaticMaxScores);
        return RESQ_ERR_WORKSPACE;
    }
    unsigned char* scratch = nullptr;
    rc = static_scratch_for_current_device(&scratch);
    if (rc) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // the array keeps whatever the previous call left: the status header is cleared here, the scores are
    // cleared by the launcher before they are accumulated, the flags are fully rewritten by the select kernel
    cudaError_t e = cudaMemsetAsync(scratch, 0, kWsHeader, st);
    if (e != cudaSuccess) return cuda_fail(e, "cudaMemsetAsync(static scratch header)");
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
    a.x_side = x_meta;
    if (pattern != RESQ_S_NONE) {
        a.r_codes = static_cast<uint8_t*>(r_codes);
        a.r_side = r_meta;
        a.mask_bits = static_cast<uint8_t*>(mask_bits);
    }
    a.status = reinterpret_cast<DeviceStatus*>(scratch);
    if (nscores) {
        a.scores = reinterpret_cast<double*>(scratch + kWsHeader);
        a.keep_flags = scratch + kWsHeader + kStaticMaxScores * sizeof(double);
    }
    return launch_quantize(kHiF4, a, st);
}
