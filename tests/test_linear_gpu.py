"""Parity of hif4_resq_linear (Eq. (5)) with the CPU oracle, through the C ABI.

Tolerance (fp32 accumulation on the GPU vs fp64 in the oracle; products are exact on both sides):
    |y - y_ref| <= 2e-3 * |y_ref| + 1e-5 * sum_k |(a + r)[m,k] * w[n,k]|
The second term is the cancellation floor: fp32 accumulation of K exact products errs by about
sqrt(K) * 2^-24 of that sum.  bf16 output adds one rounding (2^-9 relative)."""
import numpy as np
import pytest
import torch

import oracle
from workloads import CONFIGS, bf16_bits_to_f32, f32_to_bf16_bits, make_layer

pytestmark = pytest.mark.gpu


def rq():
    import paper_2607_26515_b200 as m
    return m


def to_dev(bits):
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def synth_xw(seed, M, K, N, n_out=4, w_std=0.02):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((M, K)).astype(np.float32)
    x[:, rng.choice(K, n_out, replace=False)] *= 50.0
    w = (rng.standard_normal((N, K)) * w_std).astype(np.float32)
    return f32_to_bf16_bits(x), f32_to_bf16_bits(w)


def check_close(y, ref, abs_sum, bf16_out=False):
    y = np.asarray(y, dtype=np.float64)
    tol = 2e-3 * np.abs(ref) + 1e-5 * abs_sum
    if bf16_out:
        tol = tol + 2.0 ** -8 * np.abs(ref)
    err = np.abs(y - ref)
    bad = err > tol
    assert not bad.any(), (f"{bad.sum()} of {bad.size} outside tolerance; worst ratio "
                           f"{(err / np.maximum(tol, 1e-300)).max():.3g} at {np.unravel_index(np.argmax(err / np.maximum(tol, 1e-300)), err.shape)}")


def run_case(xb, wb, pattern, fmt="hif4", out_dtype=torch.float32):
    m = rq()
    want = oracle.resq_linear(bf16_bits_to_f32(xb), bf16_bits_to_f32(wb), pattern, fmt)
    wc, ws = m.pack_weight(to_dev(wb), fmt)
    M, K = xb.shape
    N = wb.shape[0]
    wsz = m.resq_workspace_bytes(M, N, K, pattern, fmt)
    work = m.alloc_workspace(wsz)
    y = m.resq_linear(to_dev(xb), wc, ws, pattern, fmt, out_dtype=out_dtype, workspace=work)
    assert m.check(work) == 0, m.last_error()
    check_close(y.float().cpu().numpy(), want["y"], want["abs_sum"], bf16_out=out_dtype == torch.bfloat16)
    return y


ALL = [oracle.S_NONE, oracle.S_DENSE, oracle.S_2_4, oracle.S_ROW50, oracle.S_CHAN50, oracle.S_BLOCK]


@pytest.mark.parametrize("pattern", ALL)
def test_linear_one_tile(pattern):
    xb, wb = synth_xw(1, 128, 256, 256)
    run_case(xb, wb, pattern)


@pytest.mark.parametrize("pattern", ALL)
@pytest.mark.parametrize("shape", [(64, 2048, 2048), (96, 192, 80), (160, 704, 328), (288, 1024, 1000), (32, 64, 16)])
def test_linear_shapes(pattern, shape):
    M, K, N = shape
    xb, wb = synth_xw(M + N + pattern, M, K, N, n_out=max(1, K // 256))
    run_case(xb, wb, pattern)


@pytest.mark.parametrize("pattern", ALL)
@pytest.mark.parametrize("shape", [(128, 256, 256), (96, 192, 80), (288, 1024, 1000), (64, 2048, 2048)])
def test_linear_mxfp4(pattern, shape):
    M, K, N = shape
    xb, wb = synth_xw(M + N + pattern + 1, M, K, N, n_out=max(1, K // 256))
    run_case(xb, wb, pattern, fmt="mxfp4")


@pytest.mark.parametrize("pattern", [oracle.S_NONE, oracle.S_2_4])
def test_linear_bf16_output(pattern):
    xb, wb = synth_xw(7, 200, 512, 520)
    run_case(xb, wb, pattern, out_dtype=torch.bfloat16)


def test_linear_config0_tiny():
    cfg = CONFIGS[0]
    xb, wb = make_layer(cfg, 0)
    run_case(xb, wb, cfg.patterns[0])
    run_case(xb, wb, cfg.patterns[0], out_dtype=torch.bfloat16)


def test_linear_deterministic():
    xb, wb = synth_xw(9, 256, 2048, 2560)
    m = rq()
    wc, ws = m.pack_weight(to_dev(wb))
    y1 = m.resq_linear(to_dev(xb), wc, ws, m.S_2_4, out_dtype=torch.float32).clone()
    y2 = m.resq_linear(to_dev(xb), wc, ws, m.S_2_4, out_dtype=torch.float32)
    assert torch.equal(y1, y2)


def test_linear_zero_input_gives_zero():
    m = rq()
    x = torch.zeros((128, 256), dtype=torch.bfloat16, device="cuda")
    _, wb = synth_xw(3, 8, 256, 64)
    wc, ws = m.pack_weight(to_dev(wb))
    for pattern in ALL:
        y = m.resq_linear(x, wc, ws, pattern, out_dtype=torch.float32)
        assert not y.any()


@pytest.mark.parametrize("fmt", ["hif4", "mxfp4"])
@pytest.mark.parametrize("shape", [(64, 256, 200), (300, 1152, 1336), (256, 2048, 2560)])
def test_w4a16_linear_parity(fmt, shape):
    """Weight-only variant: bf16 activations straight into the GEMM, strided input included."""
    m = rq()
    M, K, N = shape
    xb, wb = synth_xw(5 * M + N, M, K, N, n_out=max(1, K // 256))
    want = oracle.w4a16_linear(bf16_bits_to_f32(xb), bf16_bits_to_f32(wb), fmt)
    wc, ws = m.pack_weight(to_dev(wb), fmt)
    big = torch.zeros((M, K + 64), dtype=torch.bfloat16, device="cuda")
    big[:, :K] = to_dev(xb)
    for x in (to_dev(xb), big[:, :K]):
        y = m.w4a16_linear(x, wc, ws, fmt, out_dtype=torch.float32)
        torch.cuda.synchronize()
        check_close(y.cpu().numpy(), want["y"], want["abs_sum"])
    yb = m.w4a16_linear(to_dev(xb), wc, ws, fmt, out_dtype=torch.bfloat16)
    check_close(yb.float().cpu().numpy(), want["y"], want["abs_sum"], bf16_out=True)


@pytest.mark.parametrize("fmt", ["hif4", "mxfp4"])
@pytest.mark.parametrize("pattern", [oracle.S_NONE, oracle.S_2_4, oracle.S_BLOCK])
@pytest.mark.parametrize("shape", [(64, 256, 200), (300, 1152, 1336), (1056, 512, 1100)])
def test_w16a4_linear_parity(shape, pattern, fmt):
    """Activation-only quantization (Table 1, W16A4): quantizer + residual + selection as in the main path, GEMM
    against plain bf16 weights (TMA straight into the MMA operand ring); contiguous and strided weights."""
    m = rq()
    M, K, N = shape
    if pattern == oracle.S_BLOCK and M % 32:
        pytest.skip("block pattern needs M % 32 == 0")
    xb, wb = synth_xw(7 * M + N + pattern, M, K, N, n_out=max(1, K // 256))
    want = oracle.w16a4_linear(bf16_bits_to_f32(xb), bf16_bits_to_f32(wb), pattern, fmt)
    wbig = torch.zeros((N, K + 72), dtype=torch.bfloat16, device="cuda")
    wbig[:, :K] = to_dev(wb)
    for w in (to_dev(wb), wbig[:, :K]):
        y = m.w16a4_linear(to_dev(xb), w, pattern, fmt, out_dtype=torch.float32)
        torch.cuda.synchronize()
        check_close(y.cpu().numpy(), want["y"], want["abs_sum"])
    yb = m.w16a4_linear(to_dev(xb), to_dev(wb), pattern, fmt, out_dtype=torch.bfloat16)
    check_close(yb.float().cpu().numpy(), want["y"], want["abs_sum"], bf16_out=True)


@pytest.mark.parametrize("fmt", ["hif4", "mxfp4"])
@pytest.mark.parametrize("pattern", [oracle.S_NONE, oracle.S_2_4, oracle.S_CHAN50, oracle.S_BLOCK])
@pytest.mark.parametrize("shape", [(64, 256, 200), (320, 1152, 520)])
def test_swiglu_fused_producer(shape, pattern, fmt):
    """Down projection with SiLU(gate) * up folded into the quantizer pass: within tolerance of the oracle, and
    bit-identical to the unfused call on the oracle's bf16 activations (so the fused producer rounds every
    activation exactly as the fixed procedure says, extremes included)."""
    m = rq()
    M, K, N = shape
    rng = np.random.default_rng(1000 * M + K + pattern)
    gu = rng.standard_normal((M, 2 * K)).astype(np.float32) * 2.5
    gu[0, :16] = [0.0, -0.0, 100.0, -100.0, 88.0, -88.0, 1e-20, -1e-20, 30.0, -30.0, 0.5, -0.5, 7.0, -7.0, 3e4, -3e4]
    gu[1, K:K + 8] = [0.0, -0.0, 1e-30, -3e4, 3e4, 1.0, -1.0, 2.0 ** -126]
    gub = f32_to_bf16_bits(gu)
    _, wb = synth_xw(9 * M + N, 8, K, N, n_out=1)
    want = oracle.swiglu_resq_linear(bf16_bits_to_f32(gub), bf16_bits_to_f32(wb), pattern, fmt)
    wc, ws = m.pack_weight(to_dev(wb), fmt)
    import os
    old = os.environ.get("RESQ_MXFP4_NATIVE")
    os.environ["RESQ_MXFP4_NATIVE"] = "0"   # the unfused reference call takes the same GEMM route as the fused one
    try:
        y = m.swiglu_resq_linear(to_dev(gub), wc, ws, pattern, fmt, out_dtype=torch.float32)
        x_dev = to_dev(f32_to_bf16_bits(want["x"]))
        y_unfused = m.resq_linear(x_dev, wc, ws, pattern, fmt, out_dtype=torch.float32)
        torch.cuda.synchronize()
    finally:
        if old is None:
            os.environ.pop("RESQ_MXFP4_NATIVE", None)
        else:
            os.environ["RESQ_MXFP4_NATIVE"] = old
    check_close(y.cpu().numpy(), want["y"], want["abs_sum"])
    assert torch.equal(y, y_unfused)


@pytest.mark.parametrize("fmt", ["hif4", "mxfp4"])
@pytest.mark.parametrize("pattern", [oracle.S_NONE, oracle.S_2_4, oracle.S_BLOCK])
@pytest.mark.parametrize("shape", [(64, 256, 200), (320, 1152, 520), (40, 4160, 96)])
def test_rmsnorm_fused_producer(shape, pattern, fmt, monkeypatch):
    """Projection with RMSNorm * gamma folded into the quantizer pass: within tolerance of the oracle, and
    bit-identical to the unfused call on the oracle's bf16 activations (rows of very different magnitude, a zero
    row, an outlier channel, a strided input)."""
    m = rq()
    M, K, N = shape
    if pattern == oracle.S_BLOCK and M % 32:
        pytest.skip("block pattern needs M % 32 == 0")
    rng = np.random.default_rng(77 * M + K + pattern)
    h = rng.standard_normal((M, K)).astype(np.float32)
    h[:, 5] *= 60.0
    h[1] *= 2.0 ** 20
    h[2] *= 2.0 ** -20
    h[3] = 0.0
    hb = f32_to_bf16_bits(h)
    gb = f32_to_bf16_bits((1.0 + 0.2 * rng.standard_normal(K)).astype(np.float32))
    _, wb = synth_xw(5 * M + N, 8, K, N, n_out=1)
    eps = 1e-6
    want = oracle.rmsnorm_resq_linear(bf16_bits_to_f32(hb), bf16_bits_to_f32(gb), eps, bf16_bits_to_f32(wb), pattern, fmt)
    wc, ws = m.pack_weight(to_dev(wb), fmt)
    monkeypatch.setenv("RESQ_MXFP4_NATIVE", "0")   # the unfused reference call takes the same GEMM route as the fused one
    big = torch.zeros((M, K + 40), dtype=torch.bfloat16, device="cuda")
    big[:, :K] = to_dev(hb)
    x_dev = to_dev(f32_to_bf16_bits(want["x"]))
    y_unfused = m.resq_linear(x_dev, wc, ws, pattern, fmt, out_dtype=torch.float32)
    for hin in (to_dev(hb), big[:, :K]):
        y = m.rmsnorm_resq_linear(hin, to_dev(gb), eps, wc, ws, pattern, fmt, out_dtype=torch.float32)
        torch.cuda.synchronize()
        check_close(y.cpu().numpy(), want["y"], want["abs_sum"])
        assert torch.equal(y, y_unfused)


@pytest.mark.parametrize("fmt", ["hif4", "mxfp4"])
@pytest.mark.parametrize("pattern", [oracle.S_NONE, oracle.S_2_4, oracle.S_CHAN50])
@pytest.mark.parametrize("shape", [(64, 256, 200), (300, 1152, 520)])
def test_randomized_hadamard_baseline(shape, pattern, fmt, monkeypatch):
    """Rotation baseline: weights rotated and packed by *_rht_pack_weight are bit-identical to packing the oracle's
    rotated weights; the rotated layer is within tolerance of the oracle and bit-identical to the plain call on the
    oracle's rotated activations."""
    m = rq()
    M, K, N = shape
    signs = 0x9E3779B97F4A7C15
    xb, wb = synth_xw(13 * M + N + pattern, M, K, N, n_out=max(1, K // 256))
    want = oracle.rht_resq_linear(bf16_bits_to_f32(xb), bf16_bits_to_f32(wb), signs, pattern, fmt)
    wc, ws = m.rht_pack_weight(to_dev(wb), signs, fmt)
    wc2, ws2 = m.pack_weight(to_dev(f32_to_bf16_bits(want["w_rot"])), fmt)
    assert torch.equal(wc, wc2) and torch.equal(ws, ws2)
    assert np.array_equal(wc.cpu().numpy(), want["w_codes"])
    monkeypatch.setenv("RESQ_MXFP4_NATIVE", "0")   # the plain reference call takes the same GEMM route
    y = m.rht_resq_linear(to_dev(xb), signs, wc, ws, pattern, fmt, out_dtype=torch.float32)
    y_plain = m.resq_linear(to_dev(f32_to_bf16_bits(want["x"])), wc, ws, pattern, fmt, out_dtype=torch.float32)
    torch.cuda.synchronize()
    check_close(y.cpu().numpy(), want["y"], want["abs_sum"])
    assert torch.equal(y, y_plain)


@pytest.mark.parametrize("fmt", ["hif4", "mxfp4"])
@pytest.mark.parametrize("q", [1, 3])
@pytest.mark.parametrize("base", [oracle.S_2_4, oracle.S_ROW50, oracle.S_CHAN50, oracle.S_BLOCK])
def test_sparsity_sweep_linear(base, q, fmt):
    """The layer with 1/4 and 3/4 of the residual kept (both GEMM routes of the MXFP4 twin)."""
    m = rq()
    M, K, N = 288, 512, 600
    pattern = oracle.keep_quarters(base, q)
    xb, wb = synth_xw(3 * base + q, M, K, N, n_out=2)
    want = oracle.resq_linear(bf16_bits_to_f32(xb), bf16_bits_to_f32(wb), pattern, fmt)
    wc, ws = m.pack_weight(to_dev(wb), fmt)
    work = m.alloc_workspace(m.resq_workspace_bytes(M, N, K, pattern, fmt))
    import os
    for native in (("1", "0") if fmt == "mxfp4" else ("0",)):
        os.environ["RESQ_MXFP4_NATIVE"] = native
        try:
            y = m.resq_linear(to_dev(xb), wc, ws, pattern, fmt, out_dtype=torch.float32, workspace=work)
            assert m.check(work) == 0, m.last_error()
        finally:
            os.environ.pop("RESQ_MXFP4_NATIVE", None)
        check_close(y.cpu().numpy(), want["y"], want["abs_sum"])


@pytest.mark.parametrize("case", [(256, 1024, 22016, oracle.S_2_4), (200, 1024, 20000, oracle.S_NONE),
                                  (512, 1024, 11000, oracle.S_DENSE), (256, 1088, 37888, oracle.S_2_4)])
def test_whole_tiles_then_dealt_out_k_blocks(case, monkeypatch):
    """K-streamed schedule with more tiles than CTA pairs (opt-in): whole rounds of tiles are computed one per pair
    and written directly, only the last round's k-blocks are dealt out and summed from fp32 slots.  One round plus a
    remainder, two M tiles, a ragged last tile, and two whole rounds with no remainder."""
    m = rq()
    M, K, N, pattern = case
    monkeypatch.setenv("RESQ_GEMM_HYBRID", "1")
    if N > 30000:
        monkeypatch.setenv("RESQ_GEMM_STREAMK", "1")   # 148 tiles: two whole rounds
    xb, wb = synth_xw(M + N, M, K, N, n_out=2)
    want = oracle.resq_linear(bf16_bits_to_f32(xb), bf16_bits_to_f32(wb), pattern, "hif4")
    wc, ws = m.pack_weight(to_dev(wb), "hif4")
    work = m.alloc_workspace(m.resq_workspace_bytes(M, N, K, pattern, "hif4"))
    y = m.resq_linear(to_dev(xb), wc, ws, pattern, "hif4", out_dtype=torch.float32, workspace=work)
    assert m.check(work) == 0, m.last_error()
    check_close(y.cpu().numpy(), want["y"], want["abs_sum"])


@pytest.mark.parametrize("fmt", ["hif4", "mxfp4"])
@pytest.mark.parametrize("shape", [(288, 512, 600), (1024, 2048, 1100)])
def test_block_per_strip_linear(shape, fmt):
    """The layer with the block selection taken per strip of 32 token rows (both GEMM routes of the MXFP4 twin)."""
    m = rq()
    M, K, N = shape
    pattern = oracle.per_strip(oracle.S_BLOCK)
    xb, wb = synth_xw(7 * M + N, M, K, N, n_out=2)
    want = oracle.resq_linear(bf16_bits_to_f32(xb), bf16_bits_to_f32(wb), pattern, fmt)
    wc, ws = m.pack_weight(to_dev(wb), fmt)
    work = m.alloc_workspace(m.resq_workspace_bytes(M, N, K, pattern, fmt))
    import os
    for native in (("1", "0") if fmt == "mxfp4" else ("0",)):
        os.environ["RESQ_MXFP4_NATIVE"] = native
        try:
            y = m.resq_linear(to_dev(xb), wc, ws, pattern, fmt, out_dtype=torch.float32, workspace=work)
            assert m.check(work) == 0, m.last_error()
        finally:
            os.environ.pop("RESQ_MXFP4_NATIVE", None)
        check_close(y.cpu().numpy(), want["y"], want["abs_sum"])


@pytest.mark.parametrize("fmt", ["hif4", "mxfp4"])
@pytest.mark.parametrize("shape", [(64, 256, 200), (300, 1152, 520), (1056, 512, 1100)])
def test_w4a8_linear_parity(shape, fmt):
    """W4A8 (Table 1) with MXFP8-E4M3 activations: within tolerance of the oracle and bit-identical to the W4A16
    call on the oracle's decoded 8-bit activations (so every activation is quantized exactly as the oracle does:
    block scales, ties, saturation, zero blocks, an outlier that pushes its block into the subnormal codes)."""
    m = rq()
    M, K, N = shape
    xb, wb = synth_xw(19 * M + N, M, K, N, n_out=max(1, K // 256))
    xf = bf16_bits_to_f32(xb).copy()
    xf[0, :32] = 0.0
    xf[1, 7] *= 300.0
    xf[2, :64] = np.float32(448.0) * np.float32(2.0 ** -3)       # exactly at the largest code
    xb = f32_to_bf16_bits(xf)
    want = oracle.w4a8_linear(bf16_bits_to_f32(xb), bf16_bits_to_f32(wb), fmt)
    wc, ws = m.pack_weight(to_dev(wb), fmt)
    big = torch.zeros((M, K + 24), dtype=torch.bfloat16, device="cuda")
    big[:, :K] = to_dev(xb)
    a_dev = to_dev(f32_to_bf16_bits(want["a"].astype(np.float32)))
    y_ref = m.w4a16_linear(a_dev, wc, ws, fmt, out_dtype=torch.float32)
    for x in (to_dev(xb), big[:, :K]):
        y = m.w4a8_linear(x, wc, ws, fmt, out_dtype=torch.float32)
        torch.cuda.synchronize()
        check_close(y.cpu().numpy(), want["y"], want["abs_sum"])
        assert torch.equal(y, y_ref)
    yb = m.w4a8_linear(to_dev(xb), wc, ws, fmt, out_dtype=torch.bfloat16)
    check_close(yb.float().cpu().numpy(), want["y"], want["abs_sum"], bf16_out=True)


@pytest.mark.parametrize("fmt", ["hif4", "mxfp4"])
@pytest.mark.parametrize("q", [2, 1])
def test_channel_selection_through_the_block_quantizer(fmt, q, monkeypatch):
    """CHAN50 on an input large enough for the block-per-lane quantizer: the channel scores are then summed from the
    residual image by a kernel of their own; same result as the chunk-per-lane path, which keeps them in registers."""
    m = rq()
    M, K, N = 2432, 1152, 264
    pattern = oracle.keep_quarters(oracle.S_CHAN50, q)
    xb, wb = synth_xw(4242 + q, M, K, N, n_out=4)
    want = oracle.resq_linear(bf16_bits_to_f32(xb), bf16_bits_to_f32(wb), pattern, fmt)
    wc, ws = m.pack_weight(to_dev(wb), fmt)
    monkeypatch.setenv("RESQ_MXFP4_NATIVE", "0")
    y = m.resq_linear(to_dev(xb), wc, ws, pattern, fmt, out_dtype=torch.float32)
    monkeypatch.setenv("RESQ_CHAN_FROM_IMAGE", "0")
    y_old = m.resq_linear(to_dev(xb), wc, ws, pattern, fmt, out_dtype=torch.float32)
    torch.cuda.synchronize()
    info = want["mask_info"]
    if info["exact"] or info["margin"] > 2.0 ** -40:
        check_close(y.cpu().numpy(), want["y"], want["abs_sum"])
        assert torch.equal(y, y_old)


@pytest.mark.parametrize("fmt", ["hif4", "mxfp4"])
@pytest.mark.parametrize("pattern", [oracle.S_NONE, oracle.S_2_4])
def test_last_round_of_tiles_as_a_second_call(pattern, fmt, monkeypatch):
    """80 output tiles of 256 x 512 on 74 CTA pairs: the six tiles of the second round are the end of the last row of
    tiles and are computed by a second, decode-sized call on sub-matrices of X, W and Y (ragged in M and N)."""
    m = rq()
    M, K, N = 2560 - 40, 256, 4096 - 24
    monkeypatch.setenv("RESQ_GEMM_PAIR_TN", "512")
    monkeypatch.setenv("RESQ_GEMM_SPLITS", "1")
    monkeypatch.setenv("RESQ_MXFP4_NATIVE", "0")
    xb, wb = synth_xw(31 + pattern, M, K, N, n_out=2)
    want = oracle.resq_linear(bf16_bits_to_f32(xb), bf16_bits_to_f32(wb), pattern, fmt)
    wc, ws = m.pack_weight(to_dev(wb), fmt)
    work = m.alloc_workspace(m.resq_workspace_bytes(M, N, K, pattern, fmt))
    for cut in ("1", "0"):
        monkeypatch.setenv("RESQ_GEMM_TAIL_SPLIT", cut)
        for out_dtype in (torch.float32, torch.bfloat16):
            y = m.resq_linear(to_dev(xb), wc, ws, pattern, fmt, out_dtype=out_dtype, workspace=work)
            assert m.check(work) == 0, m.last_error()
            check_close(y.float().cpu().numpy(), want["y"], want["abs_sum"], bf16_out=out_dtype == torch.bfloat16)


def test_swiglu_rejects_row50_and_narrow_input():
    m = rq()
    gu = torch.zeros((64, 512), dtype=torch.bfloat16, device="cuda")
    w = torch.zeros((32, 256), dtype=torch.bfloat16, device="cuda")
    wc, ws = m.pack_weight(w)
    with pytest.raises(m.ResqError):
        m.swiglu_resq_linear(gu, wc, ws, m.S_ROW50)
    with pytest.raises((m.ResqError, ValueError)):
        m.swiglu_resq_linear(gu[:, :256], wc, ws, m.S_NONE)     # weights say K = 256 but only 256 columns of [gate | up]


def test_w16a4_rejects_bad_weights():
    m = rq()
    x = torch.zeros((64, 256), dtype=torch.bfloat16, device="cuda")
    w = torch.zeros((32, 260), dtype=torch.bfloat16, device="cuda")[:, :256]   # row pitch not a multiple of 8
    with pytest.raises(m.ResqError):
        m.w16a4_linear(x, w)


# ----------------------------------------------------------------------------------------------
# Every tile configuration of the GEMM on one shape that spans several tiles and ragged edges.
# RESQ_GEMM_* are the library's debugging overrides of its tile heuristic (read at every call).

TILE_CONFIGS = [
    {"RESQ_GEMM_PAIR_TN": "512", "RESQ_GEMM_SPLITS": "1"},
    {"RESQ_GEMM_PAIR_TN": "512", "RESQ_GEMM_SPLITS": "2"},
    {"RESQ_GEMM_PAIR_TN": "384", "RESQ_GEMM_SPLITS": "1"},
    {"RESQ_GEMM_PAIR_TN": "320", "RESQ_GEMM_SPLITS": "2"},
    {"RESQ_GEMM_STREAMK": "1"},
    {"RESQ_GEMM_STREAMK": "0"},
    {"RESQ_GEMM_PAIR_TN": "256", "RESQ_GEMM_SPLITS": "1"},
    {"RESQ_GEMM_PAIR_TN": "256", "RESQ_GEMM_SPLITS": "4"},
    {"RESQ_GEMM_PAIR_TN": "128", "RESQ_GEMM_SPLITS": "1"},
    {"RESQ_GEMM_PAIR": "0", "RESQ_GEMM_MT": "1", "RESQ_GEMM_BN": "64", "RESQ_GEMM_NT": "1", "RESQ_GEMM_SPLITS": "1"},
    {"RESQ_GEMM_PAIR": "0", "RESQ_GEMM_MT": "1", "RESQ_GEMM_BN": "128", "RESQ_GEMM_NT": "1", "RESQ_GEMM_SPLITS": "2"},
    {"RESQ_GEMM_PAIR": "0", "RESQ_GEMM_MT": "1", "RESQ_GEMM_BN": "256", "RESQ_GEMM_NT": "1", "RESQ_GEMM_SPLITS": "1"},
    {"RESQ_GEMM_PAIR": "0", "RESQ_GEMM_MT": "1", "RESQ_GEMM_BN": "256", "RESQ_GEMM_NT": "2", "RESQ_GEMM_SPLITS": "1"},
    {"RESQ_GEMM_PAIR": "0", "RESQ_GEMM_MT": "2", "RESQ_GEMM_BN": "256", "RESQ_GEMM_NT": "1", "RESQ_GEMM_SPLITS": "1"},
]


@pytest.fixture(scope="module")
def tile_case():
    M, K, N = 400, 1152, 1336          # 2 pair tiles in M (ragged), 18 k-blocks, N not a multiple of any tile
    xb, wb = synth_xw(77, M, K, N, n_out=5)
    want = {}
    for pattern in (oracle.S_NONE, oracle.S_2_4):
        for fmt in ("hif4", "mxfp4"):
            want[(pattern, fmt)] = oracle.resq_linear(bf16_bits_to_f32(xb), bf16_bits_to_f32(wb), pattern, fmt)
    return xb, wb, want


@pytest.mark.parametrize("cfg", TILE_CONFIGS, ids=lambda c: ",".join(f"{k[10:]}={v}" for k, v in c.items()))
@pytest.mark.parametrize("pattern", [oracle.S_NONE, oracle.S_2_4])
@pytest.mark.parametrize("fmt", ["hif4", "mxfp4"])
def test_every_tile_configuration(tile_case, cfg, pattern, fmt, monkeypatch):
    xb, wb, want = tile_case
    if pattern != oracle.S_NONE and cfg.get("RESQ_GEMM_MT") == "2":
        pytest.skip("two M tiles per CTA exist only without a residual operand")
    for k, v in cfg.items():
        monkeypatch.setenv(k, v)
    m = rq()
    M, K = xb.shape
    N = wb.shape[0]
    wc, ws = m.pack_weight(to_dev(wb), fmt)
    work = m.alloc_workspace(m.resq_workspace_bytes(M, N, K, pattern, fmt))
    y = m.resq_linear(to_dev(xb), wc, ws, pattern, fmt, out_dtype=torch.float32, workspace=work)
    assert m.check(work) == 0, m.last_error()
    w = want[(pattern, fmt)]
    check_close(y.cpu().numpy(), w["y"], w["abs_sum"])


SPARSE_CONFIGS = [
    {},
    {"RESQ_GEMM_PAIR_TN": "480", "RESQ_GEMM_SPLITS": "1"},
    {"RESQ_GEMM_PAIR_TN": "384", "RESQ_GEMM_SPLITS": "2"},
    {"RESQ_GEMM_PAIR_TN": "320", "RESQ_GEMM_SPLITS": "4"},   # K ranges that start at odd k-blocks
    {"RESQ_GEMM_PAIR_TN": "256", "RESQ_GEMM_SPLITS": "1", "RESQ_GEMM_DEEP_E": "0"},
    {"RESQ_GEMM_PAIR_TN": "128", "RESQ_GEMM_SPLITS": "1"},
    {"RESQ_GEMM_STREAMK": "1"},
]


@pytest.mark.parametrize("cfg", SPARSE_CONFIGS, ids=lambda c: ",".join(f"{k[10:]}={v}" for k, v in c.items()) or "default")
@pytest.mark.parametrize("fmt", ["hif4", "mxfp4"])
def test_two_to_four_residual_on_the_sparse_mma(tile_case, cfg, fmt, monkeypatch):
    """S_2:4 with the residual in compressed form (two kept values of every four channels + index metadata) on
    the structured-sparse tensor instruction: same result as the dense form, for every tile width that has room
    for the metadata, split K ranges and the K-streamed schedule."""
    xb, wb, want = tile_case
    monkeypatch.setenv("RESQ_SPARSE24", "1")
    monkeypatch.setenv("RESQ_MXFP4_NATIVE", "0")
    for k, v in cfg.items():
        monkeypatch.setenv(k, v)
    m = rq()
    M, K = xb.shape
    N = wb.shape[0]
    wc, ws = m.pack_weight(to_dev(wb), fmt)
    work = m.alloc_workspace(m.resq_workspace_bytes(M, N, K, oracle.S_2_4, fmt))
    y = m.resq_linear(to_dev(xb), wc, ws, oracle.S_2_4, fmt, out_dtype=torch.float32, workspace=work)
    assert m.check(work) == 0, m.last_error()
    w = want[(oracle.S_2_4, fmt)]
    check_close(y.cpu().numpy(), w["y"], w["abs_sum"])


@pytest.mark.parametrize("fmt", ["hif4", "mxfp4"])
@pytest.mark.parametrize("shape", [(2400, 192, 200), (2500, 4160, 96)])
def test_sparse_mma_with_the_block_per_lane_quantizer(shape, fmt, monkeypatch):
    """Shapes large enough for the block-per-lane quantizer kernel (which compresses in its staging buffers): an odd
    number of k-blocks (half-used metadata block), rows that are not a multiple of the 128-row metadata bands,
    and a row longer than one warp segment."""
    monkeypatch.setenv("RESQ_SPARSE24", "1")
    monkeypatch.setenv("RESQ_MXFP4_NATIVE", "0")
    m = rq()
    M, K, N = shape
    xb, wb = synth_xw(3 * M + K, M, K, N, n_out=max(1, K // 256))
    want = oracle.resq_linear(bf16_bits_to_f32(xb), bf16_bits_to_f32(wb), oracle.S_2_4, fmt)
    wc, ws = m.pack_weight(to_dev(wb), fmt)
    work = m.alloc_workspace(m.resq_workspace_bytes(M, N, K, oracle.S_2_4, fmt))
    y = m.resq_linear(to_dev(xb), wc, ws, oracle.S_2_4, fmt, out_dtype=torch.float32, workspace=work)
    assert m.check(work) == 0, m.last_error()
    check_close(y.cpu().numpy(), want["y"], want["abs_sum"])


@pytest.mark.parametrize("pattern", ALL)
@pytest.mark.parametrize("shape", [(288, 512, 600), (128, 256, 256), (992, 1024, 1300)])
def test_mxfp4_block_scaled_fp4_gemm(monkeypatch, pattern, shape):
    """MXFP4 on the block-scaled FP4 tensor pipe (packed codes + scales straight into tcgen05.mma kind::mxf4),
    forced on for these small shapes; the same call with the path switched off must agree within tolerance too."""
    m = rq()
    M, K, N = shape
    xb, wb = synth_xw(17 * M + N + pattern, M, K, N, n_out=max(1, K // 256))
    want = oracle.resq_linear(bf16_bits_to_f32(xb), bf16_bits_to_f32(wb), pattern, "mxfp4")
    wc, ws = m.pack_weight(to_dev(wb), "mxfp4")
    work = m.alloc_workspace(m.resq_workspace_bytes(M, N, K, pattern, "mxfp4"))
    for native in ("1", "0"):
        monkeypatch.setenv("RESQ_MXFP4_NATIVE", native)
        y = m.resq_linear(to_dev(xb), wc, ws, pattern, "mxfp4", out_dtype=torch.float32, workspace=work)
        assert m.check(work) == 0, m.last_error()
        check_close(y.cpu().numpy(), want["y"], want["abs_sum"])
    monkeypatch.setenv("RESQ_MXFP4_NATIVE", "1")
    yb = m.resq_linear(to_dev(xb), wc, ws, pattern, "mxfp4", out_dtype=torch.bfloat16, workspace=work)
    check_close(yb.float().cpu().numpy(), want["y"], want["abs_sum"], bf16_out=True)


@pytest.mark.parametrize("out_dtype", [torch.float32, torch.bfloat16])
def test_k_streamed_schedule_with_uneven_segments(monkeypatch, out_dtype):
    """More output tiles than CTA pairs with a short K range: two whole rounds of tiles, then the 50 k-blocks of the
    last ten tiles are dealt out to 25 pairs (two each), so those tiles are summed from two or three partial
    segments while the other pairs have nothing left to do."""
    monkeypatch.setenv("RESQ_GEMM_STREAMK", "1")
    m = rq()
    M, K, N = 300, 320, 20000 - 24     # 2 x 79 tiles of 256 x 256, 5 k-blocks each; ragged in M and N
    xb, wb = synth_xw(91, M, K, N, n_out=3)
    want = oracle.resq_linear(bf16_bits_to_f32(xb), bf16_bits_to_f32(wb), oracle.S_2_4)
    wc, ws = m.pack_weight(to_dev(wb))
    work = m.alloc_workspace(m.resq_workspace_bytes(M, N, K, oracle.S_2_4))
    ys = [m.resq_linear(to_dev(xb), wc, ws, oracle.S_2_4, out_dtype=out_dtype, workspace=work) for _ in range(2)]
    assert m.check(work) == 0, m.last_error()
    assert torch.equal(ys[0], ys[1])   # fixed summation order: identical bits on every run
    y = ys[0].float().cpu().numpy().astype(np.float64)
    check_close(y, want["y"], want["abs_sum"], bf16_out=out_dtype == torch.bfloat16)


# ----------------------------------------------------------------------------------------------
# Full benchmark sizes in the launch configuration bench.py times: the GPU computes the whole layer,
# the oracle recomputes sampled token rows (the 2:4 and per-row selections are row-local).

@pytest.mark.parametrize("cfg_idx,layer,pattern", [(1, 0, oracle.S_2_4), (1, 2, oracle.S_2_4), (1, 3, oracle.S_2_4),
                                                   (2, 1, oracle.S_ROW50), (3, 0, oracle.S_2_4)])
def test_full_size_layers_on_sampled_rows(cfg_idx, layer, pattern):
    m = rq()
    cfg = CONFIGS[cfg_idx]
    xb, wb = make_layer(cfg, layer)
    M, K = xb.shape
    N = wb.shape[0]
    wc, ws = m.pack_weight(to_dev(wb))
    work = m.alloc_workspace(m.resq_workspace_bytes(M, N, K, pattern))
    y = m.resq_linear(to_dev(xb), wc, ws, pattern, out_dtype=torch.bfloat16, workspace=work)
    assert m.check(work) == 0, m.last_error()
    rows = np.unique(np.concatenate([[0, 127, 128, M - 1], np.random.default_rng(5).integers(0, M, 12)]))
    want = oracle.resq_linear(bf16_bits_to_f32(np.ascontiguousarray(xb[rows])), bf16_bits_to_f32(wb), pattern)
    got = y[torch.from_numpy(rows).cuda()].float().cpu().numpy()
    check_close(got, want["y"], want["abs_sum"], bf16_out=True)


def test_bounded_wait_expires_and_the_context_stays_usable():
    """RESQ_ERR_TIMEOUT path: the test hook makes the decode-sized GEMM wait for a partial tile that cannot come.  The
    bounded wait gives up, the kernel records the status and exits normally (nothing faults, nothing hangs),
    resq_check reports it, and the next call on the same workspace is an ordinary, correct one."""
    m = rq()
    xb, wb = make_layer(CONFIGS[1], 1, N=512)   # M = 256, K = 2048: CTA-pair kernel, K-streamed schedule
    pattern = oracle.S_2_4
    want = oracle.resq_linear(bf16_bits_to_f32(xb), bf16_bits_to_f32(wb), pattern)
    wc, ws = m.pack_weight(to_dev(wb))
    M, K = xb.shape
    work = m.alloc_workspace(m.resq_workspace_bytes(M, 512, K, pattern))
    x = to_dev(xb)
    m.debug_expire_next_wait(True)
    m.resq_linear(x, wc, ws, pattern, out_dtype=torch.float32, workspace=work)
    assert m.check(work) == 7                     # RESQ_ERR_TIMEOUT
    assert "wait 7" in m.last_error()             # the wait for the other pairs' segments
    torch.cuda.synchronize()                      # the context is intact
    for _ in range(2):
        y = m.resq_linear(x, wc, ws, pattern, out_dtype=torch.float32, workspace=work)
        assert m.check(work) == 0, m.last_error()
        check_close(y.cpu().numpy(), want["y"], want["abs_sum"])
    # a request that no launch consumed can be withdrawn
    m.debug_expire_next_wait(True)
    m.debug_expire_next_wait(False)
    y = m.resq_linear(x, wc, ws, pattern, out_dtype=torch.float32, workspace=work)
    assert m.check(work) == 0


GROUPS = {
    # the four linears of a 3B block at decode size (gate_up narrowed for the oracle's sake): short and long K mixed
    "block": ([(256, 2048, 2560), (256, 2048, 2048), (256, 2048, 4352), (256, 11008, 2048)], oracle.S_2_4, "hif4", torch.float32),
    # different M, ragged N, fewer rows than one MMA tile
    "ragged": ([(64, 1024, 512), (300, 512, 1000), (16, 2048, 264)], oracle.S_DENSE, "hif4", torch.bfloat16),
    "single": ([(160, 704, 328)], oracle.S_NONE, "hif4", torch.float32),
    "eight": ([(32 * (i + 1), 256 * (1 + i % 3), 136 * (i + 1)) for i in range(8)], oracle.S_2_4, "mxfp4", torch.float32),
    # more whole tiles than CTA pairs, and a long-K problem whose k-blocks are dealt out
    "many-tiles": ([(512, 512, 9728), (256, 512, 3000), (256, 8192, 512)], oracle.S_2_4, "hif4", torch.bfloat16),
    "quarter": ([(128, 1024, 384), (256, 1024, 768)], oracle.keep_quarters(oracle.S_2_4, 1), "hif4", torch.float32),
    # 100 short whole tiles and four long dealt ones: 26 pairs hold two whole tiles and still take a share of the dealt
    # k-blocks (both classes of the schedule's ranges in one launch)
    "two-classes": ([(256, 512, 25600), (256, 25600, 1024)], oracle.S_2_4, "hif4", torch.bfloat16),
    # prefill-sized problems: several rounds of whole tiles, rows beyond one M tile
    "tall": ([(2048, 1024, 4096), (1024, 4096, 1024)], oracle.S_DENSE, "hif4", torch.bfloat16),
    # at most 64 token rows everywhere: the decode kernel (weights as the MMA's M dimension, tokens as its N); tiles whose K
    # range is shared by several CTAs, ragged N, token counts that are not multiples of 16
    "decode-block": ([(16, 2048, 2560), (16, 2048, 2048), (16, 2048, 4352), (16, 11008, 2048)], oracle.S_2_4, "hif4", torch.bfloat16),
    "decode-ragged": ([(40, 1024, 520), (64, 512, 1000), (7, 2048, 264)], oracle.S_DENSE, "hif4", torch.float32),
    "decode-plain": ([(33, 704, 328), (48, 4160, 96)], oracle.S_NONE, "hif4", torch.float32),
    "decode-three-quarters": ([(24, 1024, 384), (64, 2048, 136)], oracle.keep_quarters(oracle.S_2_4, 3), "mxfp4", torch.float32),
    "decode-one": ([(64, 2048, 2048)], oracle.S_2_4, "mxfp4", torch.bfloat16),
    # the 7B block's layers (gate_up narrowed for the oracle's sake) at 24 tokens: long K ranges shared by many CTAs
    "decode-7b": ([(24, 3584, 4608), (24, 3584, 3584), (24, 3584, 4736), (24, 18944, 3584)], oracle.S_2_4, "hif4", torch.bfloat16),
}


@pytest.mark.parametrize("name", sorted(GROUPS))
def test_linear_group_matches_the_oracle_problem_by_problem(name, monkeypatch, capfd):
    """*_resq_linear_group: one quantizer launch and one GEMM launch over the tiles of all problems; every problem is
    checked element by element against the oracle, and a second run must reproduce the first bit for bit (the partial
    tiles are summed in a fixed order)."""
    m = rq()
    shapes, pattern, fmt, out_dtype = GROUPS[name]
    tensors, problems = [], []
    for i, (M, K, N) in enumerate(shapes):
        xb, wb = synth_xw(100 * len(name) + i, M, K, N, n_out=max(1, K // 512))
        wc, ws = m.pack_weight(to_dev(wb), fmt)
        tensors.append((xb, wb))
        problems.append((to_dev(xb), wc, ws))
    work = m.alloc_workspace(m.resq_group_workspace_bytes(problems, pattern, fmt, out_dtype))
    monkeypatch.setenv("RESQ_GEMM_DEBUG", "1")           # the launcher prints the schedule it planned
    if name == "two-classes":                            # (the planner's own choice gives the first 26 pairs no dealt units)
        monkeypatch.setenv("RESQ_GEMM_GROUP_DP", "100")
        monkeypatch.setenv("RESQ_GEMM_GROUP_HI", "16")
    launches0 = m.kernel_launches()
    ys = m.resq_linear_group(problems, pattern, fmt, out_dtype=out_dtype, workspace=work)
    assert m.kernel_launches() - launches0 == 2          # one quantizer kernel, one GEMM kernel
    plan = capfd.readouterr().err
    monkeypatch.delenv("RESQ_GEMM_DEBUG")
    if name == "two-classes":
        assert "100 whole tiles" in plan and "first 26 pairs take 16 each" in plan, plan
    assert m.check(work) == 0, m.last_error()
    first = [y.clone() for y in ys]
    ys2 = m.resq_linear_group([p + (y,) for p, y in zip(problems, ys)], pattern, fmt, out_dtype=out_dtype, workspace=work)
    assert m.check(work) == 0, m.last_error()
    for (xb, wb), y, y1 in zip(tensors, ys2, first):
        assert torch.equal(y, y1)
        want = oracle.resq_linear(bf16_bits_to_f32(xb), bf16_bits_to_f32(wb), pattern, fmt)
        check_close(y.float().cpu().numpy(), want["y"], want["abs_sum"], bf16_out=out_dtype == torch.bfloat16)


def test_linear_group_argument_errors():
    m = rq()
    xb, wb = synth_xw(3, 64, 256, 128)
    wc, ws = m.pack_weight(to_dev(wb))
    x = to_dev(xb)
    with pytest.raises(m.ResqError) as e:
        m.resq_linear_group([(x, wc, ws)], oracle.S_CHAN50)     # tensor-wide selections run through the single call
    assert e.value.status == 5
    with pytest.raises(m.ResqError) as e:
        m.resq_linear_group([(x, wc, ws)] * 9, oracle.S_2_4, workspace=m.alloc_workspace(1 << 20))
    assert e.value.status == 2
    with pytest.raises(m.ResqError) as e:
        m.resq_linear_group([(x, wc, ws)], oracle.S_2_4, workspace=m.alloc_workspace(4096))
    assert e.value.status == 4


@pytest.mark.parametrize("fmt", ["hif4", "mxfp4"])
@pytest.mark.parametrize("shape", [(256, 512, 384), (64, 128, 1000), (1024, 2048, 640)])
def test_backward_products_match_the_oracle(shape, fmt):
    """*_pack_weight_transposed, *_dgrad_linear, *_wgrad_linear: Eq. (1) on the transposed operands of the backward
    pass (blocks along each product's contraction axis); packed W^T bit-exact, dX^ and dW^ element by element."""
    m = rq()
    M, N, K = shape
    rng = np.random.default_rng(M + N + K)
    dy = (rng.standard_normal((M, N)) * 1e-3).astype(np.float32)
    dy[:, rng.choice(N, 2, replace=False)] *= 30.0
    dyb = f32_to_bf16_bits(dy)
    xb, wb = synth_xw(5 * M + K, M, K, N, n_out=2)
    # dgrad
    want = oracle.dgrad_linear(bf16_bits_to_f32(dyb), bf16_bits_to_f32(wb), fmt)
    wtc, wts = m.pack_weight_transposed(to_dev(wb), fmt)
    assert np.array_equal(wtc.cpu().numpy(), want["wt_codes"])
    side = wts.cpu().numpy()
    assert np.array_equal(side.view(np.uint32) if side.dtype == np.int32 else side, want["wt_side"])
    dx = m.dgrad_linear(to_dev(dyb), wtc, wts, fmt, out_dtype=torch.float32)
    check_close(dx.cpu().numpy(), want["y"], want["abs_sum"])
    # wgrad
    want2 = oracle.wgrad_linear(bf16_bits_to_f32(dyb), bf16_bits_to_f32(xb), fmt)
    dw = m.wgrad_linear(to_dev(dyb), to_dev(xb), fmt, out_dtype=torch.float32)
    check_close(dw.cpu().numpy(), want2["y"], want2["abs_sum"])
    dwb = m.wgrad_linear(to_dev(dyb), to_dev(xb), fmt, out_dtype=torch.bfloat16)
    check_close(dwb.float().cpu().numpy(), want2["y"], want2["abs_sum"], bf16_out=True)


def test_backward_products_argument_errors():
    m = rq()
    dy = torch.zeros((96, 128), dtype=torch.bfloat16, device="cuda")    # M = 96 is not a multiple of 64
    x = torch.zeros((96, 256), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(m.ResqError) as e:
        m.wgrad_linear(dy, x)
    assert e.value.status == 2
    w = torch.zeros((96, 256), dtype=torch.bfloat16, device="cuda")      # N = 96: the blocks of W^T run along N
    with pytest.raises(m.ResqError) as e:
        m.pack_weight_transposed(w)
    assert e.value.status == 2


@pytest.mark.parametrize("pattern", [oracle.S_NONE, oracle.S_DENSE, oracle.S_2_4, oracle.S_ROW50])
@pytest.mark.parametrize("shape", [(288, 1024, 1000), (1024, 2048, 1100), (200, 256, 256)])
def test_mxfp4_fp4_route_on_cta_pairs(shape, pattern, monkeypatch):
    """The block-scaled FP4 route with tcgen05.mma.cta_group::2 (256 x 256 tiles over two SMs; opt-in): several tiles per
    pair, ragged M and N, rows beyond one M tile."""
    M, K, N = shape
    monkeypatch.setenv("RESQ_MXFP4_NATIVE", "1")
    monkeypatch.setenv("RESQ_MXFP4_PAIR", "1")
    xb, wb = synth_xw(3 * M + N + pattern, M, K, N, n_out=max(1, K // 256))
    run_case(xb, wb, pattern, fmt="mxfp4")
    run_case(xb, wb, pattern, fmt="mxfp4", out_dtype=torch.bfloat16)


@pytest.mark.parametrize("fmt", ["hif4", "mxfp4"])
@pytest.mark.parametrize("case", [(288, 512, 600, False, {}), (160, 192, 80, False, {}), (1056, 1152, 1100, False, {"RESQ_GEMM_STREAMK": "0"}),
                                  (2432, 1152, 2600, False, {}), (1024, 2048, 1100, True, {}), (300, 4160, 520, False, {"RESQ_GEMM_SPLITS": "2"})],
                         ids=["streamed-k", "ragged", "whole-tiles", "many-tiles", "per-strip", "k-split"])
def test_block_selection_through_keep_flags(case, fmt, monkeypatch):
    """BLOCK with the residual image left unmasked: the GEMM reads the keep flags and loads a zero tile in place of every
    dropped block of 32 rows x 64 channels (the default from 2048 rows on; forced here on small shapes, every schedule)."""
    M, K, N, strips, env = case
    if M % 32:
        pytest.skip("the block pattern needs M % 32 == 0")
    monkeypatch.setenv("RESQ_BLOCK_LISTS", "1")
    monkeypatch.setenv("RESQ_MXFP4_NATIVE", "0")
    for k, v in env.items():
        monkeypatch.setenv(k, v)
    pattern = oracle.per_strip(oracle.S_BLOCK) if strips else oracle.S_BLOCK
    xb, wb = synth_xw(1311 + M, M, K, N, n_out=max(1, K // 256))
    y = run_case(xb, wb, pattern, fmt=fmt)
    monkeypatch.setenv("RESQ_BLOCK_LISTS", "0")
    y_masked = run_case(xb, wb, pattern, fmt=fmt)
    assert torch.equal(y, y_masked)  # same operands, same order of accumulation
    monkeypatch.setenv("RESQ_BLOCK_LISTS", "1")
    run_case(xb, wb, pattern, fmt=fmt, out_dtype=torch.bfloat16)


@pytest.mark.parametrize("pattern", [oracle.S_NONE, oracle.S_2_4, oracle.S_ROW50])
@pytest.mark.parametrize("case", [(288, 1024, 1000, "3"), (200, 2304, 520, "4"), (256, 2048, 2560, None), (64, 11008, 2048, None)],
                         ids=["two-splits", "three-uneven-splits", "decode-auto", "long-k-auto"])
def test_mxfp4_fp4_route_with_a_k_split(case, pattern, monkeypatch):
    """Decode-sized calls of the block-scaled FP4 route: (tile, K split) work items, fp32 partial slabs, fixed-order sum."""
    M, K, N, splits = case
    monkeypatch.setenv("RESQ_MXFP4_NATIVE", "1")
    if splits:
        monkeypatch.setenv("RESQ_MXFP4_SPLITS", splits)
    xb, wb = synth_xw(5 * M + N + pattern, M, K, N, n_out=max(1, K // 256))
    y = run_case(xb, wb, pattern, fmt="mxfp4")
    y2 = run_case(xb, wb, pattern, fmt="mxfp4")
    assert torch.equal(y, y2)
    run_case(xb, wb, pattern, fmt="mxfp4", out_dtype=torch.bfloat16)


@pytest.mark.parametrize("fmt", ["hif4", "mxfp4"])
@pytest.mark.parametrize("pattern", [oracle.S_NONE, oracle.S_DENSE, oracle.S_2_4])
@pytest.mark.parametrize("shape", [(16, 2048, 2048), (32, 64, 16), (7, 192, 80), (32, 4160, 96), (24, 704, 328), (1, 1024, 1000)])
def test_decode_kernel_on_single_problems(shape, pattern, fmt):
    """Groups of one problem with at most 32 token rows run on the decode kernel (128 weight rows per tile as the MMA's M
    dimension, K ranges cut evenly over the CTAs, last arrival sums a tile): one k-block, ragged N, long K, a single row."""
    m = rq()
    M, K, N = shape
    xb, wb = synth_xw(7 * M + N + pattern, M, K, N, n_out=max(1, K // 256))
    want = oracle.resq_linear(bf16_bits_to_f32(xb), bf16_bits_to_f32(wb), pattern, fmt)
    wc, ws = m.pack_weight(to_dev(wb), fmt)
    problems = [(to_dev(xb), wc, ws)]
    for out_dtype in (torch.float32, torch.bfloat16):
        work = m.alloc_workspace(m.resq_group_workspace_bytes(problems, pattern, fmt, out_dtype))
        (y,) = m.resq_linear_group(problems, pattern, fmt, out_dtype=out_dtype, workspace=work)
        assert m.check(work) == 0, m.last_error()
        (y2,) = m.resq_linear_group(problems, pattern, fmt, out_dtype=out_dtype, workspace=work)
        assert torch.equal(y, y2)
        check_close(y.float().cpu().numpy(), want["y"], want["abs_sum"], bf16_out=out_dtype == torch.bfloat16)
