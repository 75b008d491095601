"""CPU-side checks of the boundary: the C-ABI library loads, exports every symbol include/resq.h
declares, answers its size queries, and rejects bad arguments on the host (no device work)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2607_26515_b200 import build
    path = build.build()
    return ctypes.CDLL(path)


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "resq.h")).read()
    return sorted(set(re.findall(r"RESQ_API\s+[\w\s\*]+?\b(\w+)\s*\(", text)))


def test_header_declares_the_expected_entry_points():
    names = declared_symbols()
    for must in ("hif4_pack_weight", "hif4_quantize_act", "resq_residual_mask", "hif4_resq_linear",
                 "mxfp4_pack_weight", "mxfp4_quantize_act", "mxfp4_residual_mask", "mxfp4_resq_linear"):
        assert must in names


def test_library_exports_every_declared_symbol(lib):
    for name in declared_symbols():
        assert hasattr(lib, name), name


def test_binding_table_matches_header():
    from paper_2607_26515_b200 import binding
    assert sorted(binding.SYMBOLS) == declared_symbols()


def test_size_queries(lib):
    i64, sz = ctypes.c_int64, ctypes.c_size_t
    for f in ("hif4_codes_bytes", "hif4_meta_bytes", "mxfp4_codes_bytes", "mxfp4_scale_bytes", "resq_mask_bytes"):
        getattr(lib, f).restype = sz
        getattr(lib, f).argtypes = [i64, i64]
    assert lib.hif4_codes_bytes(256, 2048) == 256 * 2048 // 2
    assert lib.hif4_meta_bytes(256, 2048) == 256 * 32 * 4
    assert lib.mxfp4_scale_bytes(256, 2048) == 256 * 64
    assert lib.resq_mask_bytes(256, 2048) == 256 * 256
    # 4.5 bits per HiF4 value, 4.25 per MXFP4 value
    assert (lib.hif4_codes_bytes(64, 2048) + lib.hif4_meta_bytes(64, 2048)) * 8 == int(4.5 * 64 * 2048)
    assert (lib.mxfp4_codes_bytes(64, 2048) + lib.mxfp4_scale_bytes(64, 2048)) * 8 == int(4.25 * 64 * 2048)
    lib.resq_residual_mask_workspace_bytes.restype = sz
    lib.resq_residual_mask_workspace_bytes.argtypes = [i64, i64, ctypes.c_int]
    assert lib.resq_residual_mask_workspace_bytes(256, 2048, 2) == 256
    assert lib.resq_residual_mask_workspace_bytes(256, 2048, 4) >= 256 + 2048 * 8 + 2048
    assert lib.resq_residual_mask_workspace_bytes(256, 2048, 5) >= 256 + 8 * 32 * 9
    lib.hif4_resq_workspace_bytes.restype = sz
    lib.hif4_resq_workspace_bytes.argtypes = [i64, i64, i64, ctypes.c_int]
    assert lib.hif4_resq_workspace_bytes(256, 2560, 2048, 0) >= 256 * 2048 * 2
    assert lib.hif4_resq_workspace_bytes(256, 2560, 2048, 2) >= 2 * 256 * 2048 * 2


def test_host_side_argument_errors_need_no_device(lib):
    vp, i64, ci, sz = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_size_t
    lib.hif4_quantize_act.argtypes = [vp, i64, i64, i64, vp, vp, vp]
    lib.resq_last_error.restype = ctypes.c_char_p
    assert lib.hif4_quantize_act(None, 4, 64, 64, None, None, None) == 1          # ERR_NULL
    fake = ctypes.c_void_p(0x1000)
    assert lib.hif4_quantize_act(fake, 4, 96, 96, fake, fake, None) == 2           # K % 64
    assert b"multiple of 64" in lib.resq_last_error()
    assert lib.hif4_quantize_act(ctypes.c_void_p(0x1004), 4, 64, 64, fake, fake, None) == 3   # alignment
    assert lib.hif4_quantize_act(fake, 4, 64, 60, fake, fake, None) == 3           # ld < K
    lib.resq_residual_mask.argtypes = [vp, i64, i64, i64, ci, vp, vp, vp, vp, vp, vp, sz, vp]
    assert lib.resq_residual_mask(fake, 40, 64, 64, 5, fake, fake, fake, fake, fake, fake, 1 << 20, None) == 2
    assert lib.resq_residual_mask(fake, 32, 64, 64, 9, fake, fake, fake, fake, fake, fake, 1 << 20, None) == 5
    assert lib.resq_residual_mask(fake, 32, 64, 64, 4, fake, fake, fake, fake, fake, None, 0, None) == 4
    # pattern modifiers: kept share in quarters (bits 8..11: 1..3, selecting patterns only), per-strip flag
    # (bit 12: block pattern only), nothing above
    for bad in (2 | (4 << 8), 0 | (1 << 8), 1 | (3 << 8), 2 | (1 << 12), 3 | (1 << 12), 4 | (1 << 12), 5 | (1 << 13), -1):
        assert lib.resq_residual_mask(fake, 32, 64, 64, bad, fake, fake, fake, fake, fake, fake, 1 << 20, None) == 5, bad
    assert lib.resq_residual_mask(fake, 40, 64, 64, 5 | (1 << 12), fake, fake, fake, fake, fake, fake, 1 << 20, None) == 2
    # packed outputs are written with 32-bit / 16-bit stores: codes, metadata and scales must be 4-byte aligned
    # (a sub-buffer at an odd offset is refused on the host, not found by a misaligned-address fault)
    odd, half = ctypes.c_void_p(0x1001), ctypes.c_void_p(0x1002)
    assert lib.hif4_quantize_act(fake, 4, 64, 64, odd, fake, None) == 3
    assert lib.hif4_quantize_act(fake, 4, 64, 64, fake, half, None) == 3
    assert b"4-byte aligned" in lib.resq_last_error()
    lib.mxfp4_pack_weight.argtypes = [vp, i64, i64, i64, vp, vp, vp]
    assert lib.mxfp4_pack_weight(fake, 4, 64, 64, fake, odd, None) == 3
    for slot in range(4):    # x_codes, x_meta, r_codes, r_meta in turn
        outs = [fake] * 4
        outs[slot] = half
        assert lib.resq_residual_mask(fake, 32, 64, 64, 2, *outs, fake, fake, 1 << 20, None) == 3, slot
    lib.mxfp4_residual_mask.argtypes = lib.resq_residual_mask.argtypes
    assert lib.mxfp4_residual_mask(fake, 32, 64, 64, 2, fake, odd, fake, fake, fake, fake, 1 << 20, None) == 3
    lib.resq_residual_mask_static.argtypes = [vp, i64, i64, i64, ci, vp, vp, vp, vp, vp, vp]
    assert lib.resq_residual_mask_static(fake, 32, 64, 64, 2, fake, fake, half, fake, fake, None) == 3
    # the allocation-free variant takes the same pattern modifiers and refuses the same combinations
    for bad in (2 | (4 << 8), 0 | (1 << 8), 2 | (1 << 12), 5 | (1 << 13), -1, 9):
        assert lib.resq_residual_mask_static(fake, 32, 64, 64, bad, fake, fake, fake, fake, fake, None) == 5, bad
    assert lib.resq_residual_mask_static(fake, 40, 64, 64, 5 | (1 << 12), fake, fake, fake, fake, fake, None) == 2
    # its size limit (32768 scores) is checked on the host: one block column too many
    assert lib.resq_residual_mask_static(fake, 32, 32768 + 64, 32768 + 64, 4, fake, fake, fake, fake, fake, None) == 4
    assert b"32768" in lib.resq_last_error()
    lib.hif4_resq_linear.argtypes = [vp, i64, i64, i64, vp, vp, i64, ci, vp, ci, i64, vp, sz, vp]
    assert lib.hif4_resq_linear(fake, 32, 64, 64, fake, fake, 0, 0, fake, 0, 64, fake, 1 << 20, None) == 2
    assert lib.hif4_resq_linear(fake, 32, 64, 64, fake, fake, 64, 0, fake, 7, 64, fake, 1 << 20, None) == 5
    assert lib.hif4_resq_linear(fake, 32, 64, 64, fake, fake, 64, 0, fake, 0, 64, fake, 16, None) == 4


def test_cost_model_matches_the_papers_overhead_analysis():
    # Section 5.4: dense FP16 GEMM 2mdn; the 2:4 residual GEMM touches half the entries (mdn flops);
    # FP4 at 4x FP16 throughput gives 1/2 mdn + 1/4 mdn for S_2:4 and 1/2 + 1/2 for Dense.
    import bench
    m, d, n = 256, 2048, 2560
    base = bench.layer_flops(m, n, d, 0)
    assert base == 2 * m * d * n
    assert bench.layer_flops(m, n, d, 2) - base == m * d * n
    assert bench.layer_flops(m, n, d, 1) - base == 2 * m * d * n
    fp4 = lambda f: f / 4.0
    assert fp4(base) == 0.5 * m * d * n
    assert fp4(bench.layer_flops(m, n, d, 2)) == 0.75 * m * d * n
    assert 2 * m * d * n / fp4(bench.layer_flops(m, n, d, 2)) == pytest.approx(8 / 3)
    assert 2 * m * d * n / fp4(bench.layer_flops(m, n, d, 1)) == 2.0
