"""CPU oracle for the Rollout-ResQ FP4 linear layer -- TEST INFRASTRUCTURE ONLY.

A thin ctypes wrapper over ``resq_oracle.c`` (plain scalar C, fp64).  Only the
tests, the smoke check and the benchmark's cpu-baseline leg may import this
package; the CUDA library never does, and shares no code with it.

The C file states which passage of the paper each function follows and which
choices are readings of this project (the paper fixes the HiF4 field widths but
not the group sizes, bias, scale rule or packing: those are "parity unpinned").
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Dict, Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "resq_oracle.c")
_LIB = os.path.join(_HERE, "libresq_oracle.so")

S_NONE, S_DENSE, S_2_4, S_ROW50, S_CHAN50, S_BLOCK = 0, 1, 2, 3, 4, 5


def keep_quarters(pattern: int, q: int) -> int:
    """Sparsity sweep: the pattern with q/4 of the entries kept instead of one half (q = 1, 2, 3)."""
    return pattern | (q << 8)


def per_strip(pattern: int) -> int:
    """The 32x64 block pattern with the selection taken inside every strip of 32 token rows (each strip keeps
    floor(nbc q / 4) of its K/64 blocks) instead of over the whole tensor: the load-balanced alternative."""
    return pattern | (1 << 12)


_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain -O2, OpenMP over rows)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared",
                               "-ffp-contract=off", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        i64, dbl, vp, ci = ctypes.c_int64, ctypes.c_double, ctypes.c_void_p, ctypes.c_int
        for name in ("oracle_hif4_e6m2_value", "oracle_hif4_s1p2_value", "oracle_e2m1_value", "oracle_e8m0_value"):
            getattr(L, name).restype = dbl
            getattr(L, name).argtypes = [ci]
        L.oracle_hif4_encode.argtypes = [vp, i64, i64, vp, vp]
        L.oracle_hif4_decode.argtypes = [vp, vp, i64, i64, vp]
        L.oracle_mxfp4_encode.argtypes = [vp, i64, i64, vp, vp]
        L.oracle_mxfp4_decode.argtypes = [vp, vp, i64, i64, vp]
        L.oracle_residual.argtypes = [vp, vp, i64, vp]
        L.oracle_residual.restype = i64
        L.oracle_mask.argtypes = [vp, i64, i64, ci, vp, vp, vp]
        L.oracle_apply_mask.argtypes = [vp, vp, i64, i64, vp]
        L.oracle_apply_mask.restype = None
        L.oracle_matmul.argtypes = [vp, vp, vp, i64, i64, i64, vp, vp]
        L.oracle_matmul.restype = None
        _lib = L
    return _lib


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _f32(x: np.ndarray) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float32)
    assert x.ndim == 2
    return x


# ------------------------------------------------------------------ formats

def e6m2_value(s: int) -> float:
    return float(lib().oracle_hif4_e6m2_value(int(s)))


def s1p2_value(code: int) -> float:
    return float(lib().oracle_hif4_s1p2_value(int(code)))


def e2m1_value(code: int) -> float:
    return float(lib().oracle_e2m1_value(int(code)))


def e8m0_value(code: int) -> float:
    return float(lib().oracle_e8m0_value(int(code)))


def hif4_encode(x: np.ndarray):
    """x float32 [rows,K] -> (codes uint8 [rows,K/2], meta uint32 [rows,K/64])."""
    x = _f32(x)
    rows, K = x.shape
    codes = np.empty((rows, K // 2), dtype=np.uint8)
    meta = np.empty((rows, K // 64), dtype=np.uint32)
    rc = lib().oracle_hif4_encode(_p(x), rows, K, _p(codes), _p(meta))
    if rc:
        raise ValueError("HiF4 needs K % 64 == 0")
    return codes, meta


def hif4_decode(codes: np.ndarray, meta: np.ndarray) -> np.ndarray:
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    meta = np.ascontiguousarray(meta, dtype=np.uint32)
    rows, K = codes.shape[0], codes.shape[1] * 2
    out = np.empty((rows, K), dtype=np.float64)
    rc = lib().oracle_hif4_decode(_p(codes), _p(meta), rows, K, _p(out))
    if rc:
        raise ValueError("HiF4 needs K % 64 == 0")
    return out


def mxfp4_encode(x: np.ndarray):
    """x float32 [rows,K] -> (codes uint8 [rows,K/2], scale uint8 [rows,K/32])."""
    x = _f32(x)
    rows, K = x.shape
    codes = np.empty((rows, K // 2), dtype=np.uint8)
    scale = np.empty((rows, K // 32), dtype=np.uint8)
    rc = lib().oracle_mxfp4_encode(_p(x), rows, K, _p(codes), _p(scale))
    if rc:
        raise ValueError("MXFP4 needs K % 32 == 0")
    return codes, scale


def mxfp4_decode(codes: np.ndarray, scale: np.ndarray) -> np.ndarray:
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    scale = np.ascontiguousarray(scale, dtype=np.uint8)
    rows, K = codes.shape[0], codes.shape[1] * 2
    out = np.empty((rows, K), dtype=np.float64)
    rc = lib().oracle_mxfp4_decode(_p(codes), _p(scale), rows, K, _p(out))
    if rc:
        raise ValueError("MXFP4 needs K % 32 == 0")
    return out


def encode(fmt: str, x: np.ndarray):
    return hif4_encode(x) if fmt == "hif4" else mxfp4_encode(x)


def decode(fmt: str, codes: np.ndarray, side: np.ndarray) -> np.ndarray:
    return hif4_decode(codes, side) if fmt == "hif4" else mxfp4_decode(codes, side)


# ------------------------------------------------------------------ residual, masks, product

def residual(x: np.ndarray, deq: np.ndarray) -> np.ndarray:
    """Eq. (3): x - deq(Q(x)), returned as float32; raises if any difference is not fp32-exact."""
    x = _f32(x)
    deq = np.ascontiguousarray(deq, dtype=np.float64)
    dx = np.empty_like(x)
    bad = lib().oracle_residual(_p(x), _p(deq), x.size, _p(dx))
    if bad:
        raise ArithmeticError(f"{bad} residual elements are not exact in fp32")
    return dx


def mask(v: np.ndarray, pattern: int, want_scores: bool = False):
    """Selection S on the decoded quantized residual v [M,K] -> (mask_bits uint8 [M,K/8], info dict)."""
    v = np.ascontiguousarray(v, dtype=np.float64)
    M, K = v.shape
    bits = np.empty((M, K // 8), dtype=np.uint8)
    info = np.zeros(2, dtype=np.float64)
    scores = None
    if want_scores and (pattern & 0xFF) == S_CHAN50:
        scores = np.zeros(K, dtype=np.float64)
    if want_scores and (pattern & 0xFF) == S_BLOCK:
        scores = np.zeros((M // 32) * (K // 64), dtype=np.float64)
    rc = lib().oracle_mask(_p(v), M, K, int(pattern), _p(bits), _p(info), _p(scores))
    if rc == -1:
        raise ValueError("shape not valid for this pattern")
    if rc == -2:
        raise ValueError("unknown pattern")
    return bits, {"exact": bool(info[0]), "margin": float(info[1]), "scores": scores}


def apply_mask(r: np.ndarray, bits: np.ndarray) -> np.ndarray:
    r = np.ascontiguousarray(r, dtype=np.float64)
    bits = np.ascontiguousarray(bits, dtype=np.uint8)
    out = np.empty_like(r)
    lib().oracle_apply_mask(_p(r), _p(bits), r.shape[0], r.shape[1], _p(out))
    return out


def matmul(a: np.ndarray, r: Optional[np.ndarray], w: np.ndarray, want_abs: bool = True):
    """Eq. (5) on decoded operands: a@w.T + r@w.T in fp64 -> (y [M,N], abs_sum [M,N] or None)."""
    a = np.ascontiguousarray(a, dtype=np.float64)
    w = np.ascontiguousarray(w, dtype=np.float64)
    if r is not None:
        r = np.ascontiguousarray(r, dtype=np.float64)
    M, K = a.shape
    N = w.shape[0]
    assert w.shape[1] == K
    y = np.empty((M, N), dtype=np.float64)
    ab = np.empty((M, N), dtype=np.float64) if want_abs else None
    lib().oracle_matmul(_p(a), _p(r), _p(w), M, N, K, _p(y), _p(ab))
    return y, ab


def quantize_residual_mask(x_f32: np.ndarray, pattern: int, fmt: str = "hif4") -> Dict[str, np.ndarray]:
    """Steps Q(X), Eq. (3), Q(dX), S(.) in the paper's order."""
    x_f32 = _f32(x_f32)
    x_codes, x_side = encode(fmt, x_f32)
    a = decode(fmt, x_codes, x_side)
    out = {"x_codes": x_codes, "x_side": x_side, "a": a}
    if pattern == S_NONE:
        return out
    dx = residual(x_f32, a)
    r_codes, r_side = encode(fmt, dx)
    r = decode(fmt, r_codes, r_side)
    bits, info = mask(r, pattern)
    out.update({"dx": dx, "r_codes": r_codes, "r_side": r_side, "r": r, "mask": bits,
                "mask_info": info, "r_masked": apply_mask(r, bits)})
    return out


def resq_linear(x_f32: np.ndarray, w_f32: np.ndarray, pattern: int, fmt: str = "hif4",
                want_abs: bool = True) -> Dict[str, np.ndarray]:
    """The whole path: pack W, quantize X, residual, mask, two-term product."""
    out = quantize_residual_mask(x_f32, pattern, fmt)
    w_codes, w_side = encode(fmt, _f32(w_f32))
    w = decode(fmt, w_codes, w_side)
    y, ab = matmul(out["a"], out.get("r_masked"), w, want_abs)
    out.update({"w_codes": w_codes, "w_side": w_side, "w": w, "y": y, "abs_sum": ab})
    return out


def w16a4_linear(x_f32: np.ndarray, w_f32: np.ndarray, pattern: int = S_NONE, fmt: str = "hif4",
                 want_abs: bool = True) -> Dict[str, np.ndarray]:
    """Activation-only ablation (Table 1, W16A4): the activations go through Q, Eq. (3) and S as in Eq. (5); the
    weights are used as given (bf16 values): Y = (deq Q(X) + S(deq Q(dX))) W^T."""
    out = quantize_residual_mask(x_f32, pattern, fmt)
    y, ab = matmul(out["a"], out.get("r_masked"), np.asarray(w_f32, dtype=np.float64), want_abs)
    out.update({"y": y, "abs_sum": ab})
    return out


def w4a16_linear(x_f32: np.ndarray, w_f32: np.ndarray, fmt: str = "hif4", want_abs: bool = True) -> Dict[str, np.ndarray]:
    """Weight-only ablation (Table 1, W4A16): Y = X deq(Q(W))^T, activations as given (bf16 values)."""
    w_codes, w_side = encode(fmt, _f32(w_f32))
    w = decode(fmt, w_codes, w_side)
    y, ab = matmul(np.asarray(x_f32, dtype=np.float64), None, w, want_abs)
    return {"w_codes": w_codes, "w_side": w_side, "w": w, "y": y, "abs_sum": ab}


# ---- fused producer of the down projection: x = SiLU(gate) * up, rounded to bf16, then the path above ---------
# The paper applies the method to the linear layers of every transformer block; the input of the down projection is
# SiLU(g) * u of the gate / up projection outputs.  Its rounding to bf16 decides 4-bit codes, so the evaluation is
# fixed here operation by operation in fp32 (every operation rounded to nearest even, no fused multiply-add), the
# precision the fused kernel works in:
#   t = g * (-log2 e), clamped to [-126, 126];  n = rint(t);  f = t - n;
#   p = 2^f by the degree-6 Taylor polynomial of exp(f ln 2) in Horner form;  e = p * 2^n  (= exp(-g));
#   s = g / (1 + e);   x = bf16(s * u).
_LOG2E_NEG = np.float32(-1.4426950408889634)
_EXP2_COEF = [np.float32(c) for c in (1.0, 0.6931471805599453, 0.2402265069591007, 0.05550410866482158,
                                       0.009618129107628477, 0.0013333558146428443, 0.00015403530393381608)]


def silu32(g: np.ndarray) -> np.ndarray:
    """SiLU(g) = g / (1 + exp(-g)) by the fixed fp32 procedure above (relative error about 2e-7)."""
    g = np.asarray(g, dtype=np.float32)
    t = np.multiply(g, _LOG2E_NEG, dtype=np.float32)
    t = np.minimum(np.maximum(t, np.float32(-126.0)), np.float32(126.0))
    n = np.rint(t).astype(np.float32)
    f = np.subtract(t, n, dtype=np.float32)
    p = np.full_like(f, _EXP2_COEF[6])
    for c in reversed(_EXP2_COEF[:6]):
        p = np.add(np.multiply(p, f, dtype=np.float32), c, dtype=np.float32)
    scale = ((n.astype(np.int32) + 127) << 23).astype(np.uint32).view(np.float32)  # 2^n, exact
    e = np.multiply(p, scale, dtype=np.float32)
    d = np.add(np.float32(1.0), e, dtype=np.float32)
    return np.divide(g, d, dtype=np.float32)


def _bf16_rne(x: np.ndarray) -> np.ndarray:
    b = np.asarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    b = (b + 0x7FFF + ((b >> 16) & 1)) & 0xFFFF0000
    return b.astype(np.uint32).view(np.float32)


def swiglu_bf16(g: np.ndarray, u: np.ndarray) -> np.ndarray:
    """x = bf16(SiLU(g) * u) for bf16-valued g, u (finite)."""
    s = silu32(g)
    return _bf16_rne(np.multiply(s, np.asarray(u, dtype=np.float32), dtype=np.float32))


def swiglu_resq_linear(gu_f32: np.ndarray, w_f32: np.ndarray, pattern: int, fmt: str = "hif4",
                       want_abs: bool = True) -> Dict[str, np.ndarray]:
    """Down projection with its producer: gu = [gate | up] ([M, 2K]); Eq. (5) on x = bf16(SiLU(gate) * up)."""
    gu = np.asarray(gu_f32, dtype=np.float32)
    K = gu.shape[1] // 2
    x = swiglu_bf16(gu[:, :K], gu[:, K:])
    out = resq_linear(x, w_f32, pattern, fmt, want_abs)
    out["x"] = x
    return out


# ---- fused producer of the qkv / gate_up projections: x = RMSNorm(h) * gamma, rounded to bf16 -------------------
# Fixed evaluation (fp32, every operation rounded to nearest even): ss = the exact sum of squares of the row (the
# squares of bf16 values are exact; the sum is taken exactly and rounded once to fp32), ms = ss / K, v = ms + eps,
# r = 1 / sqrt(v) as a correctly rounded square root followed by a correctly rounded division, and
# x[k] = bf16((h[k] * r) * gamma[k]).
def rmsnorm_row_scale(h: np.ndarray, eps: float) -> np.ndarray:
    import math
    h = np.asarray(h, dtype=np.float32)
    K = h.shape[1]
    ss = np.array([math.fsum((float(v) * float(v) for v in row)) for row in h], dtype=np.float64).astype(np.float32)
    ms = np.divide(ss, np.float32(K), dtype=np.float32)
    v = np.add(ms, np.float32(eps), dtype=np.float32)
    return np.divide(np.float32(1.0), np.sqrt(v, dtype=np.float32), dtype=np.float32)


def rmsnorm_bf16(h: np.ndarray, gamma: np.ndarray, eps: float) -> np.ndarray:
    """x = bf16((h * r_row) * gamma) for bf16-valued h [M, K] and gamma [K]."""
    h = np.asarray(h, dtype=np.float32)
    r = rmsnorm_row_scale(h, eps)
    t = np.multiply(h, r[:, None], dtype=np.float32)
    return _bf16_rne(np.multiply(t, np.asarray(gamma, dtype=np.float32)[None, :], dtype=np.float32))


def rmsnorm_resq_linear(h_f32: np.ndarray, gamma_f32: np.ndarray, eps: float, w_f32: np.ndarray, pattern: int,
                        fmt: str = "hif4", want_abs: bool = True) -> Dict[str, np.ndarray]:
    """Projection with its RMSNorm producer: Eq. (5) on x = bf16(RMSNorm(h) * gamma)."""
    x = rmsnorm_bf16(h_f32, gamma_f32, eps)
    out = resq_linear(x, w_f32, pattern, fmt, want_abs)
    out["x"] = x
    return out


# ---- randomized Hadamard pre-transform (the rotation baseline the paper compares against) ----------------------
# Per block of 64 channels: x' = bf16( (1/8) * H64 (s * x) ), s in {+1, -1}^64 given by the bits of `signs` (bit j
# set = channel j of every block negated), H64 the Sylvester Hadamard matrix.  Evaluated as the in-place fast
# transform in fp32: six stages with strides 1, 2, 4, 8, 16, 32, each replacing a pair (a, b) = (v[j], v[j + stride])
# by (a + b, a - b), every operation rounded to nearest even; the scale 1/8 is exact.  H64 / 8 is orthogonal, so
# rotating X and W alike leaves X W^T unchanged in exact arithmetic.
def rht64_bf16(x: np.ndarray, signs: int) -> np.ndarray:
    x = np.asarray(x, dtype=np.float32)
    M, K = x.shape
    assert K % 64 == 0
    s = np.array([-1.0 if (signs >> j) & 1 else 1.0 for j in range(64)], dtype=np.float32)
    v = np.multiply(x.reshape(M, K // 64, 64), s, dtype=np.float32)
    stride = 1
    while stride < 64:
        v = v.reshape(M, K // 64, 64 // (2 * stride), 2, stride)
        a, b = v[:, :, :, 0, :], v[:, :, :, 1, :]
        v = np.stack([np.add(a, b, dtype=np.float32), np.subtract(a, b, dtype=np.float32)], axis=3)
        stride *= 2
    v = np.multiply(v.reshape(M, K), np.float32(0.125), dtype=np.float32)
    return _bf16_rne(v)


def rht_resq_linear(x_f32: np.ndarray, w_f32: np.ndarray, signs: int, pattern: int, fmt: str = "hif4",
                    want_abs: bool = True) -> Dict[str, np.ndarray]:
    """Rotation baseline: Eq. (5) on the rotated activations and the rotated weights."""
    x = rht64_bf16(x_f32, signs)
    w = rht64_bf16(w_f32, signs)
    out = resq_linear(x, w, pattern, fmt, want_abs)
    out["x"] = x
    out["w_rot"] = w
    return out


# ---- 8-bit activations for the "W4A8" ablation of Table 1 -----------------------------------------------------
# The paper names the ablation but not the 8-bit format.  Reading of this project: MXFP8 with E4M3 elements as the
# OCP microscaling specification defines it -- blocks of 32 along K, one E8M0 power-of-two scale
# 2^(floor(log2 amax) - 8) per block (8 = exponent of the largest E4M3 value, 448 = 1.75 * 2^8; all-zero block:
# scale code 0), elements rounded to the nearest E4M3 value (4 exponent bits, bias 7, 3 mantissa bits, subnormals
# below 2^-6, ties to even) and saturated at +-448.  Used for both weight formats.
def e4m3_value(code: int) -> float:
    s = -1.0 if code & 0x80 else 1.0
    e, m = (code >> 3) & 15, code & 7
    if e == 15 and m == 7:
        return float("nan")
    return s * (m / 8.0 * 2.0 ** -6 if e == 0 else (1.0 + m / 8.0) * 2.0 ** (e - 7))


def mxfp8_e4m3_quantize(x: np.ndarray):
    """x float32 [rows, K] -> (codes uint8 [rows, K], scale uint8 [rows, K/32], decoded float64 [rows, K])."""
    x = np.asarray(x, dtype=np.float64)
    rows, K = x.shape
    if K % 32:
        raise ValueError("MXFP8 needs K % 32 == 0")
    xb = x.reshape(rows, K // 32, 32)
    amax = np.abs(xb).max(axis=2)
    e = np.full(amax.shape, -127, dtype=np.int64)
    nz = amax > 0
    # floor(log2 amax) through frexp (exact at powers of two)
    _, ex = np.frexp(amax[nz])
    e[nz] = np.clip(ex.astype(np.int64) - 1 - 8, -127, 127)
    t = np.abs(xb) / np.exp2(e.astype(np.float64))[:, :, None]            # exact scaling
    # spacing of the E4M3 grid at t: 2^-9 below 2^-6, else 2^(floor(log2 t) - 3)
    _, tex = np.frexp(np.maximum(t, 2.0 ** -6))
    step = np.exp2((tex - 1 - 3).astype(np.float64))
    q = np.minimum(np.rint(t / step) * step, 448.0)                        # rint: ties to even; exact quotient
    deq = np.copysign(q, xb) * np.exp2(e.astype(np.float64))[:, :, None]
    # codes (for the table pins): sign | exponent field | mantissa
    _, qex = np.frexp(np.maximum(q, 2.0 ** -7))
    ef = np.where(q < 2.0 ** -6, 0, qex - 1 + 7)
    mf = np.where(q < 2.0 ** -6, np.rint(q * 2.0 ** 9), np.rint((q / np.exp2((qex - 1).astype(np.float64)) - 1.0) * 8))
    codes = ((np.signbit(xb).astype(np.int64) << 7) | (ef.astype(np.int64) << 3) | mf.astype(np.int64)).astype(np.uint8)
    return codes.reshape(rows, K), (e + 127).astype(np.uint8), deq.reshape(rows, K)


def w4a8_linear(x_f32: np.ndarray, w_f32: np.ndarray, fmt: str = "hif4", want_abs: bool = True) -> Dict[str, np.ndarray]:
    """Table 1, W4A8: Y = deq(Q8(X)) deq(Q4(W))^T with MXFP8-E4M3 activations and 4-bit weights."""
    codes, scale, a = mxfp8_e4m3_quantize(x_f32)
    w_codes, w_side = encode(fmt, _f32(w_f32))
    w = decode(fmt, w_codes, w_side)
    y, ab = matmul(a, None, w, want_abs)
    return {"a_codes": codes, "a_scale": scale, "a": a, "w": w, "y": y, "abs_sum": ab}


# ---- training-side GEMMs of the same layer (the backward pass of Y = X W^T) -----------------------------------------
# The paper states that the forward and the backward passes of the training policy run in 4 bit (Sections 1 and 3)
# and writes out the forward product only (Eq. (1)).  Reading taken here: Eq. (1)'s operator Q is applied to both
# operands of each backward product, with the quantization blocks along that product's contraction axis (as in the
# forward product, where they run along d):
#     dX = dY W        (contraction over n):  dX^ = Q(dY) Q(W^T)^T,   Q along n on the rows of dY [m, n] and of W^T [d, n]
#     dW = dY^T X      (contraction over m):  dW^ = Q(dY^T) Q(X^T)^T, Q along m on the rows of dY^T [n, m] and of X^T [d, m]
# No residual term: Rollout-ResQ corrects the rollout policy's activations only (Section 4).

def dgrad_linear(dy_f32: np.ndarray, w_f32: np.ndarray, fmt: str = "hif4", want_abs: bool = True) -> Dict[str, np.ndarray]:
    """dX^ [m, d] = Q(dY) Q(W^T)^T for dY [m, n], W [n, d]."""
    dy = _f32(dy_f32)
    wt = np.ascontiguousarray(_f32(w_f32).T)
    g_codes, g_side = encode(fmt, dy)
    wt_codes, wt_side = encode(fmt, wt)
    g = decode(fmt, g_codes, g_side)
    wtd = decode(fmt, wt_codes, wt_side)
    y, ab = matmul(g, None, wtd, want_abs)
    return {"g": g, "wt": wtd, "wt_codes": wt_codes, "wt_side": wt_side, "y": y, "abs_sum": ab}


def wgrad_linear(dy_f32: np.ndarray, x_f32: np.ndarray, fmt: str = "hif4", want_abs: bool = True) -> Dict[str, np.ndarray]:
    """dW^ [n, d] = Q(dY^T) Q(X^T)^T for dY [m, n], X [m, d]."""
    gt = np.ascontiguousarray(_f32(dy_f32).T)
    xt = np.ascontiguousarray(_f32(x_f32).T)
    gt_codes, gt_side = encode(fmt, gt)
    xt_codes, xt_side = encode(fmt, xt)
    gtd = decode(fmt, gt_codes, gt_side)
    xtd = decode(fmt, xt_codes, xt_side)
    y, ab = matmul(gtd, None, xtd, want_abs)
    return {"gt": gtd, "xt": xtd, "y": y, "abs_sum": ab}
