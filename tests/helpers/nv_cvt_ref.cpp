// Test-only helper: exposes NVIDIA's host-callable conversion routines from the CUDA
// toolkit headers so that the oracle's E2M1 / E8M0 tables and rounding can be pinned to a
// library routine.  Contains no arithmetic of its own.
#include <cuda_fp4.h>
#include <cuda_fp8.h>
#include <cuda_fp16.h>
#include <cstring>
#include <cstdint>

extern "C" int nv_float_to_e2m1(float x) {
    return (int)__nv_cvt_float_to_fp4(x, __NV_E2M1, cudaRoundNearest);
}

extern "C" float nv_e2m1_to_float(int code) {
    __half_raw h = __nv_cvt_fp4_to_halfraw((__nv_fp4_storage_t)code, __NV_E2M1);
    // widen the IEEE half bit pattern by hand (no device intrinsics on the host)
    uint32_t s = (h.x >> 15) & 1u, e = (h.x >> 10) & 31u, m = h.x & 1023u;
    float v;
    if (e == 0) v = (float)m / 1024.0f / 16384.0f;            // subnormal: m * 2^-24
    else { uint32_t bits = (s << 31) | ((e + 112u) << 23) | (m << 13); std::memcpy(&v, &bits, 4); return v; }
    return s ? -v : v;
}

extern "C" float nv_e8m0_to_float(int code) {
    __nv_bfloat16_raw b = __nv_cvt_e8m0_to_bf16raw((__nv_fp8_storage_t)code);
    uint32_t bits = ((uint32_t)b.x) << 16;
    float v; std::memcpy(&v, &bits, 4); return v;
}
