"""Thin ctypes binding of the C ABI in include/resq.h (argument marshalling only).

PyTorch supplies device memory (`tensor.data_ptr()`) and the stream; every step of the path
runs in the CUDA library.  There is no CPU fallback: if the library is missing or a call fails,
this module raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libresq.so")

S_NONE, S_DENSE, S_2_4, S_ROW50, S_CHAN50, S_BLOCK = 0, 1, 2, 3, 4, 5
OUT_BF16, OUT_F32 = 0, 1
PATTERN_NAMES = {S_NONE: "none", S_DENSE: "dense", S_2_4: "2:4", S_ROW50: "row50", S_CHAN50: "chan50",
                 S_BLOCK: "block32x64"}
STATUS_NAMES = {0: "OK", 1: "ERR_NULL", 2: "ERR_SHAPE", 3: "ERR_ALIGN", 4: "ERR_WORKSPACE", 5: "ERR_PATTERN",
                6: "ERR_CUDA", 7: "ERR_TIMEOUT"}

# every symbol include/resq.h declares: (name, restype, argtypes)
_i64, _vp, _ci, _sz = ctypes.c_int64, ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
SYMBOLS = {
    "hif4_codes_bytes": (_sz, [_i64, _i64]),
    "hif4_meta_bytes": (_sz, [_i64, _i64]),
    "mxfp4_codes_bytes": (_sz, [_i64, _i64]),
    "mxfp4_scale_bytes": (_sz, [_i64, _i64]),
    "resq_mask_bytes": (_sz, [_i64, _i64]),
    "resq_residual_mask_workspace_bytes": (_sz, [_i64, _i64, _ci]),
    "hif4_resq_workspace_bytes": (_sz, [_i64, _i64, _i64, _ci]),
    "mxfp4_resq_workspace_bytes": (_sz, [_i64, _i64, _i64, _ci]),
    "hif4_pack_weight": (_ci, [_vp, _i64, _i64, _i64, _vp, _vp, _vp]),
    "mxfp4_pack_weight": (_ci, [_vp, _i64, _i64, _i64, _vp, _vp, _vp]),
    "hif4_quantize_act": (_ci, [_vp, _i64, _i64, _i64, _vp, _vp, _vp]),
    "mxfp4_quantize_act": (_ci, [_vp, _i64, _i64, _i64, _vp, _vp, _vp]),
    "hif4_dequantize": (_ci, [_vp, _vp, _i64, _i64, _vp, _vp]),
    "mxfp4_dequantize": (_ci, [_vp, _vp, _i64, _i64, _vp, _vp]),
    "resq_residual_mask": (_ci, [_vp, _i64, _i64, _i64, _ci, _vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp]),
    "mxfp4_residual_mask": (_ci, [_vp, _i64, _i64, _i64, _ci, _vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp]),
    "resq_residual_mask_static": (_ci, [_vp, _i64, _i64, _i64, _ci, _vp, _vp, _vp, _vp, _vp, _vp]),
    "hif4_resq_linear": (_ci, [_vp, _i64, _i64, _i64, _vp, _vp, _i64, _ci, _vp, _ci, _i64, _vp, _sz, _vp]),
    "mxfp4_resq_linear": (_ci, [_vp, _i64, _i64, _i64, _vp, _vp, _i64, _ci, _vp, _ci, _i64, _vp, _sz, _vp]),
    "hif4_resq_group_workspace_bytes": (_sz, [_vp, _ci, _ci]),
    "mxfp4_resq_group_workspace_bytes": (_sz, [_vp, _ci, _ci]),
    "hif4_resq_linear_group": (_ci, [_vp, _ci, _ci, _ci, _vp, _sz, _vp]),
    "mxfp4_resq_linear_group": (_ci, [_vp, _ci, _ci, _ci, _vp, _sz, _vp]),
    "resq_transposed_workspace_bytes": (_sz, [_i64, _i64]),
    "hif4_pack_weight_transposed": (_ci, [_vp, _i64, _i64, _i64, _vp, _vp, _vp, _sz, _vp]),
    "mxfp4_pack_weight_transposed": (_ci, [_vp, _i64, _i64, _i64, _vp, _vp, _vp, _sz, _vp]),
    "hif4_dgrad_workspace_bytes": (_sz, [_i64, _i64, _i64]),
    "mxfp4_dgrad_workspace_bytes": (_sz, [_i64, _i64, _i64]),
    "hif4_dgrad_linear": (_ci, [_vp, _i64, _i64, _i64, _vp, _vp, _i64, _vp, _ci, _i64, _vp, _sz, _vp]),
    "mxfp4_dgrad_linear": (_ci, [_vp, _i64, _i64, _i64, _vp, _vp, _i64, _vp, _ci, _i64, _vp, _sz, _vp]),
    "hif4_wgrad_workspace_bytes": (_sz, [_i64, _i64, _i64]),
    "mxfp4_wgrad_workspace_bytes": (_sz, [_i64, _i64, _i64]),
    "hif4_wgrad_linear": (_ci, [_vp, _vp, _i64, _i64, _i64, _i64, _i64, _vp, _ci, _i64, _vp, _sz, _vp]),
    "mxfp4_wgrad_linear": (_ci, [_vp, _vp, _i64, _i64, _i64, _i64, _i64, _vp, _ci, _i64, _vp, _sz, _vp]),
    "resq_w4a16_workspace_bytes": (_sz, [_i64, _i64, _i64]),
    "resq_w4a8_workspace_bytes": (_sz, [_i64, _i64, _i64]),
    "hif4_w4a8_linear": (_ci, [_vp, _i64, _i64, _i64, _vp, _vp, _i64, _vp, _ci, _i64, _vp, _sz, _vp]),
    "mxfp4_w4a8_linear": (_ci, [_vp, _i64, _i64, _i64, _vp, _vp, _i64, _vp, _ci, _i64, _vp, _sz, _vp]),
    "hif4_w4a16_linear": (_ci, [_vp, _i64, _i64, _i64, _vp, _vp, _i64, _vp, _ci, _i64, _vp, _sz, _vp]),
    "mxfp4_w4a16_linear": (_ci, [_vp, _i64, _i64, _i64, _vp, _vp, _i64, _vp, _ci, _i64, _vp, _sz, _vp]),
    "hif4_swiglu_resq_linear": (_ci, [_vp, _i64, _i64, _i64, _vp, _vp, _i64, _ci, _vp, _ci, _i64, _vp, _sz, _vp]),
    "mxfp4_swiglu_resq_linear": (_ci, [_vp, _i64, _i64, _i64, _vp, _vp, _i64, _ci, _vp, _ci, _i64, _vp, _sz, _vp]),
    "hif4_rmsnorm_resq_linear": (_ci, [_vp, _i64, _i64, _i64, _vp, ctypes.c_float, _vp, _vp, _i64, _ci, _vp, _ci, _i64, _vp, _sz, _vp]),
    "mxfp4_rmsnorm_resq_linear": (_ci, [_vp, _i64, _i64, _i64, _vp, ctypes.c_float, _vp, _vp, _i64, _ci, _vp, _ci, _i64, _vp, _sz, _vp]),
    "hif4_rht_pack_weight": (_ci, [_vp, _i64, _i64, _i64, ctypes.c_ulonglong, _vp, _vp, _vp]),
    "mxfp4_rht_pack_weight": (_ci, [_vp, _i64, _i64, _i64, ctypes.c_ulonglong, _vp, _vp, _vp]),
    "hif4_rht_resq_linear": (_ci, [_vp, _i64, _i64, _i64, ctypes.c_ulonglong, _vp, _vp, _i64, _ci, _vp, _ci, _i64, _vp, _sz, _vp]),
    "mxfp4_rht_resq_linear": (_ci, [_vp, _i64, _i64, _i64, ctypes.c_ulonglong, _vp, _vp, _i64, _ci, _vp, _ci, _i64, _vp, _sz, _vp]),
    "hif4_w16a4_linear": (_ci, [_vp, _i64, _i64, _i64, _vp, _i64, _i64, _ci, _vp, _ci, _i64, _vp, _sz, _vp]),
    "mxfp4_w16a4_linear": (_ci, [_vp, _i64, _i64, _i64, _vp, _i64, _i64, _ci, _vp, _ci, _i64, _vp, _sz, _vp]),
    "resq_check": (_ci, [_vp, _vp]),
    "resq_last_error": (ctypes.c_char_p, []),
    "resq_kernel_launches": (_i64, []),
    "resq_debug_expire_next_wait": (_ci, [_ci]),
    "resq_profile_enable": (_ci, [_ci]),
    "resq_profile_read": (_ci, [_vp, _vp]),
}

_lib: Optional[ctypes.CDLL] = None


class ResqError(RuntimeError):
    def __init__(self, status: int, msg: str):
        super().__init__(f"resq: {STATUS_NAMES.get(status, status)}: {msg}")
        self.status = status


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2607_26515_b200.build` "
                               "(there is no fallback path)")
        L = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in SYMBOLS.items():
            fn = getattr(L, name)
            fn.restype = res
            fn.argtypes = args
        _lib = L
    return _lib


def last_error() -> str:
    return lib().resq_last_error().decode()


def _check(status: int) -> None:
    if status != 0:
        raise ResqError(status, last_error())


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else t.data_ptr()


def _side(fmt: str, rows: int, K: int, device) -> torch.Tensor:
    if fmt == "hif4":
        return torch.empty((rows, K // 64), dtype=torch.int32, device=device)
    return torch.empty((rows, K // 32), dtype=torch.uint8, device=device)


def _fn(fmt: str, hif4_name: str, mx_name: str):
    if fmt not in ("hif4", "mxfp4"):
        raise ValueError(f"unknown format {fmt!r}")
    return getattr(lib(), hif4_name if fmt == "hif4" else mx_name)


def _require_bf16_matrix(x: torch.Tensor, name: str) -> None:
    if x.dtype != torch.bfloat16 or x.dim() != 2 or not x.is_cuda or x.stride(1) != 1:
        raise ValueError(f"{name} must be a 2-D CUDA bf16 tensor with unit inner stride")


# ------------------------------------------------------------------ size queries

def residual_mask_workspace_bytes(M: int, K: int, pattern: int) -> int:
    return int(lib().resq_residual_mask_workspace_bytes(M, K, pattern))


def resq_workspace_bytes(M: int, N: int, K: int, pattern: int, fmt: str = "hif4") -> int:
    return int(_fn(fmt, "hif4_resq_workspace_bytes", "mxfp4_resq_workspace_bytes")(M, N, K, pattern))


def alloc_workspace(nbytes: int, device="cuda") -> torch.Tensor:
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)


# ------------------------------------------------------------------ calls

def keep_quarters(pattern: int, q: int) -> int:
    """RESQ_KEEP_QUARTERS: the pattern with q/4 of the entries kept instead of one half (q = 1, 2, 3)."""
    return pattern | (q << 8)


def per_strip(pattern: int) -> int:
    """RESQ_BLOCK_PER_STRIP: the 32x64 block pattern with the selection taken inside every strip of 32 token rows."""
    return pattern | (1 << 12)


def pack_weight(W: torch.Tensor, fmt: str = "hif4", stream=None) -> Tuple[torch.Tensor, torch.Tensor]:
    """*_pack_weight: W bf16 [N,K] -> (codes u8 [N,K/2], meta i32 [N,K/64] | scale u8 [N,K/32])."""
    _require_bf16_matrix(W, "W")
    N, K = W.shape
    codes = torch.empty((N, K // 2), dtype=torch.uint8, device=W.device)
    side = _side(fmt, N, K, W.device)
    _check(_fn(fmt, "hif4_pack_weight", "mxfp4_pack_weight")(W.data_ptr(), N, K, W.stride(0), codes.data_ptr(),
                                                              side.data_ptr(), _stream(stream)))
    return codes, side


def rht_pack_weight(W: torch.Tensor, signs: int, fmt: str = "hif4", stream=None) -> Tuple[torch.Tensor, torch.Tensor]:
    """*_rht_pack_weight: rotate every block of 64 channels by the randomized Hadamard transform, then pack."""
    _require_bf16_matrix(W, "W")
    N, K = W.shape
    codes = torch.empty((N, K // 2), dtype=torch.uint8, device=W.device)
    side = _side(fmt, N, K, W.device)
    _check(_fn(fmt, "hif4_rht_pack_weight", "mxfp4_rht_pack_weight")(W.data_ptr(), N, K, W.stride(0), signs & (2 ** 64 - 1),
                                                                      codes.data_ptr(), side.data_ptr(), _stream(stream)))
    return codes, side


def rht_resq_linear(X: torch.Tensor, signs: int, w_codes: torch.Tensor, w_side: torch.Tensor, pattern: int = S_NONE,
                    fmt: str = "hif4", out_dtype: torch.dtype = torch.bfloat16, Y: Optional[torch.Tensor] = None,
                    workspace: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """*_rht_resq_linear: Eq. (5) on the rotated activations against weights packed by rht_pack_weight."""
    _require_bf16_matrix(X, "X")
    M, K = X.shape
    N = w_codes.shape[0]
    if Y is None:
        ld = (N + 7) // 8 * 8
        Y = torch.empty((M, ld), dtype=out_dtype, device=X.device)[:, :N]
    if Y.dtype not in (torch.bfloat16, torch.float32):
        raise ValueError("Y must be bf16 or fp32")
    if workspace is None:
        workspace = alloc_workspace(resq_workspace_bytes(M, N, K, pattern, fmt), X.device)
    _check(_fn(fmt, "hif4_rht_resq_linear", "mxfp4_rht_resq_linear")(
        X.data_ptr(), M, K, X.stride(0), signs & (2 ** 64 - 1), w_codes.data_ptr(), w_side.data_ptr(), N, pattern,
        Y.data_ptr(), OUT_BF16 if Y.dtype == torch.bfloat16 else OUT_F32, Y.stride(0), workspace.data_ptr(),
        workspace.numel(), _stream(stream)))
    return Y


def quantize_act(X: torch.Tensor, fmt: str = "hif4", stream=None) -> Tuple[torch.Tensor, torch.Tensor]:
    """*_quantize_act: X bf16 [M,K] -> (codes, meta | scale)."""
    _require_bf16_matrix(X, "X")
    M, K = X.shape
    codes = torch.empty((M, K // 2), dtype=torch.uint8, device=X.device)
    side = _side(fmt, M, K, X.device)
    _check(_fn(fmt, "hif4_quantize_act", "mxfp4_quantize_act")(X.data_ptr(), M, K, X.stride(0), codes.data_ptr(),
                                                                side.data_ptr(), _stream(stream)))
    return codes, side


def dequantize(codes: torch.Tensor, side: torch.Tensor, fmt: str = "hif4", stream=None) -> torch.Tensor:
    rows, K = codes.shape[0], codes.shape[1] * 2
    out = torch.empty((rows, K), dtype=torch.float32, device=codes.device)
    _check(_fn(fmt, "hif4_dequantize", "mxfp4_dequantize")(codes.data_ptr(), side.data_ptr(), rows, K, out.data_ptr(),
                                                            _stream(stream)))
    return out


def residual_mask(X: torch.Tensor, pattern: int, fmt: str = "hif4", workspace: Optional[torch.Tensor] = None,
                  stream=None):
    """resq_residual_mask / mxfp4_residual_mask -> dict(x_codes, x_side, r_codes, r_side, mask)."""
    _require_bf16_matrix(X, "X")
    M, K = X.shape
    dev = X.device
    out = {"x_codes": torch.empty((M, K // 2), dtype=torch.uint8, device=dev), "x_side": _side(fmt, M, K, dev),
           "r_codes": None, "r_side": None, "mask": None}
    if pattern != S_NONE:
        out["r_codes"] = torch.empty((M, K // 2), dtype=torch.uint8, device=dev)
        out["r_side"] = _side(fmt, M, K, dev)
        out["mask"] = torch.empty((M, K // 8), dtype=torch.uint8, device=dev)
    if workspace is None:
        workspace = alloc_workspace(residual_mask_workspace_bytes(M, K, pattern), dev)
    _check(_fn(fmt, "resq_residual_mask", "mxfp4_residual_mask")(
        X.data_ptr(), M, K, X.stride(0), pattern, _ptr(out["x_codes"]), _ptr(out["x_side"]), _ptr(out["r_codes"]),
        _ptr(out["r_side"]), _ptr(out["mask"]), workspace.data_ptr(), workspace.numel(), _stream(stream)))
    return out


STATIC_SCRATCH_MAX_SCORES = 32768


def residual_mask_static(X: torch.Tensor, pattern: int, stream=None):
    """resq_residual_mask_static: the HiF4 residual / mask pass without a caller workspace, for callers that
    cannot allocate device memory; its selection scratch is a fixed array inside the library (at most
    STATIC_SCRATCH_MAX_SCORES channel or block scores).  Calls that overlap on the GPU race on that array."""
    _require_bf16_matrix(X, "X")
    M, K = X.shape
    dev = X.device
    out = {"x_codes": torch.empty((M, K // 2), dtype=torch.uint8, device=dev), "x_side": _side("hif4", M, K, dev),
           "r_codes": None, "r_side": None, "mask": None}
    if pattern != S_NONE:
        out["r_codes"] = torch.empty((M, K // 2), dtype=torch.uint8, device=dev)
        out["r_side"] = _side("hif4", M, K, dev)
        out["mask"] = torch.empty((M, K // 8), dtype=torch.uint8, device=dev)
    _check(lib().resq_residual_mask_static(
        X.data_ptr(), M, K, X.stride(0), pattern, _ptr(out["x_codes"]), _ptr(out["x_side"]), _ptr(out["r_codes"]),
        _ptr(out["r_side"]), _ptr(out["mask"]), _stream(stream)))
    return out


def resq_linear(X: torch.Tensor, w_codes: torch.Tensor, w_side: torch.Tensor, pattern: int, fmt: str = "hif4",
                out_dtype: torch.dtype = torch.bfloat16, Y: Optional[torch.Tensor] = None,
                workspace: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """*_resq_linear: Y = Q(X) Q(W)^T + S(Q(X - deq Q(X))) Q(W)^T  (Eq. (5))."""
    _require_bf16_matrix(X, "X")
    M, K = X.shape
    N = w_codes.shape[0]
    if Y is None:
        ld = (N + 7) // 8 * 8  # rows of Y start on 16-byte boundaries
        Y = torch.empty((M, ld), dtype=out_dtype, device=X.device)[:, :N]
    if Y.dtype not in (torch.bfloat16, torch.float32):
        raise ValueError("Y must be bf16 or fp32")
    if workspace is None:
        workspace = alloc_workspace(resq_workspace_bytes(M, N, K, pattern, fmt), X.device)
    _check(_fn(fmt, "hif4_resq_linear", "mxfp4_resq_linear")(
        X.data_ptr(), M, K, X.stride(0), w_codes.data_ptr(), w_side.data_ptr(), N, pattern, Y.data_ptr(),
        OUT_BF16 if Y.dtype == torch.bfloat16 else OUT_F32, Y.stride(0), workspace.data_ptr(), workspace.numel(),
        _stream(stream)))
    return Y


class _Problem(ctypes.Structure):
    """struct resq_problem of include/resq.h."""
    _fields_ = [("X_bf16", _vp), ("M", _i64), ("K", _i64), ("ldx", _i64), ("w_codes", _vp), ("w_side", _vp), ("N", _i64),
                ("Y", _vp), ("ldy", _i64)]


MAX_GROUP = 8


def _problem_array(problems, out_dtype):
    """problems: sequence of (X, w_codes, w_side) or (X, w_codes, w_side, Y) -> (ctypes array, list of Y)."""
    arr = (_Problem * len(problems))()
    ys = []
    for i, pr in enumerate(problems):
        X, wc, ws = pr[0], pr[1], pr[2]
        _require_bf16_matrix(X, "X")
        M, K = X.shape
        N = wc.shape[0]
        Y = pr[3] if len(pr) > 3 and pr[3] is not None else torch.empty((M, (N + 7) // 8 * 8), dtype=out_dtype, device=X.device)[:, :N]
        if Y.dtype != out_dtype:
            raise ValueError("every Y of a group has the group's output type")
        ys.append(Y)
        arr[i] = _Problem(X.data_ptr(), M, K, X.stride(0), wc.data_ptr(), ws.data_ptr(), N, Y.data_ptr(), Y.stride(0))
    return arr, ys


def resq_group_workspace_bytes(problems, pattern: int, fmt: str = "hif4", out_dtype: torch.dtype = torch.bfloat16) -> int:
    arr, _ = _problem_array(problems, out_dtype)
    return int(_fn(fmt, "hif4_resq_group_workspace_bytes", "mxfp4_resq_group_workspace_bytes")(
        ctypes.cast(arr, _vp), len(problems), pattern))


def resq_linear_group(problems, pattern: int, fmt: str = "hif4", out_dtype: torch.dtype = torch.bfloat16,
                      workspace: Optional[torch.Tensor] = None, stream=None):
    """*_resq_linear_group: up to MAX_GROUP independent projections of Eq. (5) in one quantizer launch and one GEMM
    launch.  problems: sequence of (X, w_codes, w_side[, Y]); returns the list of outputs."""
    if out_dtype not in (torch.bfloat16, torch.float32):
        raise ValueError("Y must be bf16 or fp32")
    arr, ys = _problem_array(problems, out_dtype)
    fn_b = _fn(fmt, "hif4_resq_group_workspace_bytes", "mxfp4_resq_group_workspace_bytes")
    if workspace is None:
        workspace = alloc_workspace(int(fn_b(ctypes.cast(arr, _vp), len(problems), pattern)), problems[0][0].device)
    _check(_fn(fmt, "hif4_resq_linear_group", "mxfp4_resq_linear_group")(
        ctypes.cast(arr, _vp), len(problems), pattern, OUT_BF16 if out_dtype == torch.bfloat16 else OUT_F32,
        workspace.data_ptr(), workspace.numel(), _stream(stream)))
    return ys


def _out(rows: int, cols: int, dtype: torch.dtype, device) -> torch.Tensor:
    """An output matrix whose rows start on 16-byte boundaries."""
    return torch.empty((rows, (cols + 7) // 8 * 8), dtype=dtype, device=device)[:, :cols]


def pack_weight_transposed(W: torch.Tensor, fmt: str = "hif4", stream=None) -> Tuple[torch.Tensor, torch.Tensor]:
    """*_pack_weight_transposed: W bf16 [N,K] -> Q(W^T) as (codes [K,N/2], meta [K,N/64] | scale [K,N/32]), for dgrad."""
    _require_bf16_matrix(W, "W")
    N, K = W.shape
    codes = torch.empty((K, N // 2), dtype=torch.uint8, device=W.device)
    side = _side(fmt, K, N, W.device)
    work = alloc_workspace(int(lib().resq_transposed_workspace_bytes(N, K)), W.device)
    _check(_fn(fmt, "hif4_pack_weight_transposed", "mxfp4_pack_weight_transposed")(
        W.data_ptr(), N, K, W.stride(0), codes.data_ptr(), side.data_ptr(), work.data_ptr(), work.numel(), _stream(stream)))
    return codes, side


def dgrad_linear(dY: torch.Tensor, wt_codes: torch.Tensor, wt_side: torch.Tensor, fmt: str = "hif4",
                 out_dtype: torch.dtype = torch.bfloat16, workspace: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """*_dgrad_linear: dX^ [M,K] = Q(dY) Q(W^T)^T with the transposed pack of the weight."""
    _require_bf16_matrix(dY, "dY")
    M, N = dY.shape
    K = wt_codes.shape[0]
    dX = _out(M, K, out_dtype, dY.device)
    if workspace is None:
        workspace = alloc_workspace(int(_fn(fmt, "hif4_dgrad_workspace_bytes", "mxfp4_dgrad_workspace_bytes")(M, N, K)), dY.device)
    _check(_fn(fmt, "hif4_dgrad_linear", "mxfp4_dgrad_linear")(
        dY.data_ptr(), M, N, dY.stride(0), wt_codes.data_ptr(), wt_side.data_ptr(), K, dX.data_ptr(),
        OUT_BF16 if out_dtype == torch.bfloat16 else OUT_F32, dX.stride(0), workspace.data_ptr(), workspace.numel(), _stream(stream)))
    return dX


def wgrad_linear(dY: torch.Tensor, X: torch.Tensor, fmt: str = "hif4", out_dtype: torch.dtype = torch.bfloat16,
                 workspace: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """*_wgrad_linear: dW^ [N,K] = Q(dY^T) Q(X^T)^T."""
    _require_bf16_matrix(dY, "dY")
    _require_bf16_matrix(X, "X")
    M, N = dY.shape
    K = X.shape[1]
    if X.shape[0] != M:
        raise ValueError("dY and X must have the same number of token rows")
    dW = _out(N, K, out_dtype, dY.device)
    if workspace is None:
        workspace = alloc_workspace(int(_fn(fmt, "hif4_wgrad_workspace_bytes", "mxfp4_wgrad_workspace_bytes")(M, N, K)), dY.device)
    _check(_fn(fmt, "hif4_wgrad_linear", "mxfp4_wgrad_linear")(
        dY.data_ptr(), X.data_ptr(), M, N, K, dY.stride(0), X.stride(0), dW.data_ptr(),
        OUT_BF16 if out_dtype == torch.bfloat16 else OUT_F32, dW.stride(0), workspace.data_ptr(), workspace.numel(), _stream(stream)))
    return dW


def w4a16_linear(X: torch.Tensor, w_codes: torch.Tensor, w_side: torch.Tensor, fmt: str = "hif4",
                 out_dtype: torch.dtype = torch.bfloat16, Y: Optional[torch.Tensor] = None,
                 workspace: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """*_w4a16_linear: Y = X deq(Q(W))^T, activations kept in bf16 (Table 1, W4A16)."""
    _require_bf16_matrix(X, "X")
    M, K = X.shape
    N = w_codes.shape[0]
    if Y is None:
        ld = (N + 7) // 8 * 8
        Y = torch.empty((M, ld), dtype=out_dtype, device=X.device)[:, :N]
    if Y.dtype not in (torch.bfloat16, torch.float32):
        raise ValueError("Y must be bf16 or fp32")
    if workspace is None:
        workspace = alloc_workspace(int(lib().resq_w4a16_workspace_bytes(M, N, K)), X.device)
    _check(_fn(fmt, "hif4_w4a16_linear", "mxfp4_w4a16_linear")(
        X.data_ptr(), M, K, X.stride(0), w_codes.data_ptr(), w_side.data_ptr(), N, Y.data_ptr(),
        OUT_BF16 if Y.dtype == torch.bfloat16 else OUT_F32, Y.stride(0), workspace.data_ptr(), workspace.numel(),
        _stream(stream)))
    return Y


def swiglu_resq_linear(GU: torch.Tensor, w_codes: torch.Tensor, w_side: torch.Tensor, pattern: int, fmt: str = "hif4",
                       out_dtype: torch.dtype = torch.bfloat16, Y: Optional[torch.Tensor] = None,
                       workspace: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """*_swiglu_resq_linear: Eq. (5) on X = bf16(SiLU(gate) * up) with GU = [gate | up], X never stored."""
    _require_bf16_matrix(GU, "GU")
    M, K2 = GU.shape
    K = K2 // 2
    N = w_codes.shape[0]
    if K2 % 2 or w_codes.shape[1] * 2 != K:
        raise ValueError("GU must be [M, 2K] for weights packed as [N, K/2]")
    if Y is None:
        ld = (N + 7) // 8 * 8
        Y = torch.empty((M, ld), dtype=out_dtype, device=GU.device)[:, :N]
    if Y.dtype not in (torch.bfloat16, torch.float32):
        raise ValueError("Y must be bf16 or fp32")
    if workspace is None:
        workspace = alloc_workspace(resq_workspace_bytes(M, N, K, pattern, fmt), GU.device)
    _check(_fn(fmt, "hif4_swiglu_resq_linear", "mxfp4_swiglu_resq_linear")(
        GU.data_ptr(), M, K, GU.stride(0), w_codes.data_ptr(), w_side.data_ptr(), N, pattern, Y.data_ptr(),
        OUT_BF16 if Y.dtype == torch.bfloat16 else OUT_F32, Y.stride(0), workspace.data_ptr(), workspace.numel(),
        _stream(stream)))
    return Y


def rmsnorm_resq_linear(H: torch.Tensor, gamma: torch.Tensor, eps: float, w_codes: torch.Tensor, w_side: torch.Tensor,
                        pattern: int, fmt: str = "hif4", out_dtype: torch.dtype = torch.bfloat16,
                        Y: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """*_rmsnorm_resq_linear: Eq. (5) on X = bf16(RMSNorm(H) * gamma), X never stored."""
    _require_bf16_matrix(H, "H")
    M, K = H.shape
    N = w_codes.shape[0]
    if gamma.dtype != torch.bfloat16 or gamma.numel() != K or not gamma.is_contiguous():
        raise ValueError("gamma must be a contiguous bf16 vector of K elements")
    if Y is None:
        ld = (N + 7) // 8 * 8
        Y = torch.empty((M, ld), dtype=out_dtype, device=H.device)[:, :N]
    if Y.dtype not in (torch.bfloat16, torch.float32):
        raise ValueError("Y must be bf16 or fp32")
    if workspace is None:
        workspace = alloc_workspace(resq_workspace_bytes(M, N, K, pattern, fmt), H.device)
    _check(_fn(fmt, "hif4_rmsnorm_resq_linear", "mxfp4_rmsnorm_resq_linear")(
        H.data_ptr(), M, K, H.stride(0), gamma.data_ptr(), float(eps), w_codes.data_ptr(), w_side.data_ptr(), N, pattern,
        Y.data_ptr(), OUT_BF16 if Y.dtype == torch.bfloat16 else OUT_F32, Y.stride(0), workspace.data_ptr(),
        workspace.numel(), _stream(stream)))
    return Y


def w4a8_linear(X: torch.Tensor, w_codes: torch.Tensor, w_side: torch.Tensor, fmt: str = "hif4",
                out_dtype: torch.dtype = torch.bfloat16, Y: Optional[torch.Tensor] = None,
                workspace: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """*_w4a8_linear: Y = deq(MXFP8-E4M3(X)) deq(Q(W))^T (Table 1, W4A8; the 8-bit format is this library's reading)."""
    _require_bf16_matrix(X, "X")
    M, K = X.shape
    N = w_codes.shape[0]
    if Y is None:
        ld = (N + 7) // 8 * 8
        Y = torch.empty((M, ld), dtype=out_dtype, device=X.device)[:, :N]
    if Y.dtype not in (torch.bfloat16, torch.float32):
        raise ValueError("Y must be bf16 or fp32")
    if workspace is None:
        workspace = alloc_workspace(int(lib().resq_w4a8_workspace_bytes(M, N, K)), X.device)
    _check(_fn(fmt, "hif4_w4a8_linear", "mxfp4_w4a8_linear")(
        X.data_ptr(), M, K, X.stride(0), w_codes.data_ptr(), w_side.data_ptr(), N, Y.data_ptr(),
        OUT_BF16 if Y.dtype == torch.bfloat16 else OUT_F32, Y.stride(0), workspace.data_ptr(), workspace.numel(),
        _stream(stream)))
    return Y


def w16a4_linear(X: torch.Tensor, W: torch.Tensor, pattern: int = S_NONE, fmt: str = "hif4",
                 out_dtype: torch.dtype = torch.bfloat16, Y: Optional[torch.Tensor] = None,
                 workspace: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """*_w16a4_linear: Y = (deq Q(X) + S(deq Q(dX))) W^T with plain bf16 weights (Table 1, W16A4)."""
    _require_bf16_matrix(X, "X")
    _require_bf16_matrix(W, "W")
    M, K = X.shape
    N = W.shape[0]
    if W.shape[1] != K:
        raise ValueError("W must be [N, K]")
    if Y is None:
        ld = (N + 7) // 8 * 8
        Y = torch.empty((M, ld), dtype=out_dtype, device=X.device)[:, :N]
    if Y.dtype not in (torch.bfloat16, torch.float32):
        raise ValueError("Y must be bf16 or fp32")
    if workspace is None:
        workspace = alloc_workspace(resq_workspace_bytes(M, N, K, pattern, fmt), X.device)
    _check(_fn(fmt, "hif4_w16a4_linear", "mxfp4_w16a4_linear")(
        X.data_ptr(), M, K, X.stride(0), W.data_ptr(), N, W.stride(0), pattern, Y.data_ptr(),
        OUT_BF16 if Y.dtype == torch.bfloat16 else OUT_F32, Y.stride(0), workspace.data_ptr(), workspace.numel(),
        _stream(stream)))
    return Y


def check(workspace: torch.Tensor, stream=None) -> int:
    """resq_check: synchronize and return the device status word."""
    return int(lib().resq_check(workspace.data_ptr(), _stream(stream)))


# ------------------------------------------------------------------ diagnostics

KERNEL_KINDS = ("quantize", "select", "gemm", "splitk_reduce")


def kernel_launches() -> int:
    """resq_kernel_launches: kernels launched by the library in this process so far."""
    return int(lib().resq_kernel_launches())


def debug_expire_next_wait(on: bool = True) -> None:
    """resq_debug_expire_next_wait: the next decode-sized GEMM launch lets its bounded wait run out (test hook)."""
    _check(lib().resq_debug_expire_next_wait(1 if on else 0))


def profile_enable(on: bool) -> None:
    _check(lib().resq_profile_enable(1 if on else 0))


def profile_read():
    """resq_profile_read -> {kind: (device ms, launches)} since the last read."""
    ms = (ctypes.c_double * 4)()
    n = (ctypes.c_int64 * 4)()
    _check(lib().resq_profile_read(ctypes.cast(ms, ctypes.c_void_p), ctypes.cast(n, ctypes.c_void_p)))
    return {k: (float(ms[i]), int(n[i])) for i, k in enumerate(KERNEL_KINDS)}
