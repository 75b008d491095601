"""Parity of the CUDA quantizer / residual / mask kernels with the CPU oracle: bit-exact codes,
metadata, scales and masks on the same seeded inputs, called through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from workloads import CONFIGS, bf16_bits_to_f32, f32_to_bf16_bits, make_activation, make_weight

pytestmark = pytest.mark.gpu


def rq():
    import paper_2607_26515_b200 as m
    return m


def to_dev(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def side_np(t: torch.Tensor) -> np.ndarray:
    a = t.cpu().numpy()
    return a.view(np.uint32) if a.dtype == np.int32 else a


def synth(seed, rows, K, n_out=6, scale=64.0, extremes=True):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((rows, K)).astype(np.float32)
    x[:, rng.choice(K, n_out, replace=False)] *= scale
    # edge content: zero block, tiny block, huge block, exact ties, negative zero
    x[0, :64] = 0
    if rows > 3 and extremes:
        x[1, :64] *= 2.0 ** -70
        x[2, :64] *= 2.0 ** 20
    if rows > 3 and K > 130:
        x[3, 64:128] = np.round(x[3, 64:128] * 4) / 4
        x[3, 130] = -0.0
    return f32_to_bf16_bits(x)


@pytest.mark.parametrize("fmt", ["hif4", "mxfp4"])
@pytest.mark.parametrize("shape", [(1, 64), (5, 192), (37, 2048), (64, 11008), (300, 3584)])
def test_quantize_act_and_pack_weight_bit_exact(fmt, shape):
    bits = synth(shape[0] * 7 + shape[1], *shape, n_out=min(6, shape[1] // 16))
    xf = bf16_bits_to_f32(bits)
    want_c, want_s = oracle.encode(fmt, xf)
    for fn in (rq().quantize_act, rq().pack_weight):
        codes, side = fn(to_dev(bits), fmt)
        torch.cuda.synchronize()
        assert np.array_equal(side_np(side), want_s)
        assert np.array_equal(codes.cpu().numpy(), want_c)
    deq = rq().dequantize(codes, side, fmt).cpu().numpy()
    assert np.array_equal(deq.astype(np.float64), oracle.decode(fmt, want_c, want_s))


@pytest.mark.parametrize("fmt", ["hif4", "mxfp4"])
def test_strided_input(fmt):
    bits = synth(3, 33, 512)
    big = torch.zeros((33, 1024), dtype=torch.bfloat16, device="cuda")
    big[:, :512] = to_dev(bits)
    codes, side = rq().quantize_act(big[:, :512], fmt)
    want_c, want_s = oracle.encode(fmt, bf16_bits_to_f32(bits))
    assert np.array_equal(codes.cpu().numpy(), want_c) and np.array_equal(side_np(side), want_s)


PATTERNS = [oracle.S_NONE, oracle.S_DENSE, oracle.S_2_4, oracle.S_ROW50, oracle.S_CHAN50, oracle.S_BLOCK]


@pytest.mark.parametrize("fmt", ["hif4", "mxfp4"])
@pytest.mark.parametrize("pattern", PATTERNS)
@pytest.mark.parametrize("shape", [(32, 64), (64, 2048), (96, 3584), (256, 11008), (320, 2048), (160, 4096 - 64)])
def test_residual_mask_bit_exact(fmt, pattern, shape):
    M, K = shape
    # the 2^-70 / 2^20 blocks would make the fp64 score sums inexact: leave them out for the global patterns
    bits = synth(M + K + pattern, M, K, n_out=max(1, K // 256),
                 extremes=pattern not in (oracle.S_CHAN50, oracle.S_BLOCK))
    xf = bf16_bits_to_f32(bits)
    want = oracle.quantize_residual_mask(xf, pattern, fmt)
    got = rq().residual_mask(to_dev(bits), pattern, fmt)
    torch.cuda.synchronize()
    assert np.array_equal(got["x_codes"].cpu().numpy(), want["x_codes"])
    assert np.array_equal(side_np(got["x_side"]), want["x_side"])
    if pattern == oracle.S_NONE:
        return
    assert np.array_equal(side_np(got["r_side"]), want["r_side"])
    assert np.array_equal(got["r_codes"].cpu().numpy(), want["r_codes"])
    info = want["mask_info"]
    mask = got["mask"].cpu().numpy()
    if pattern in (oracle.S_CHAN50, oracle.S_BLOCK) and not (info["exact"] or info["margin"] > 2.0 ** -40):
        pytest.skip("selection scores not exactly summable and boundary margin too small")
    assert np.array_equal(mask, want["mask"])


@pytest.mark.parametrize("fmt", ["hif4", "mxfp4"])
@pytest.mark.parametrize("q", [1, 3])
@pytest.mark.parametrize("base", [oracle.S_2_4, oracle.S_ROW50, oracle.S_CHAN50, oracle.S_BLOCK])
@pytest.mark.parametrize("shape", [(64, 256), (320, 2048), (2432, 192), (32, 4160)])
def test_sparsity_sweep_masks_bit_exact(shape, base, q, fmt):
    """Kept share 1/4 and 3/4 (1:4 / 3:4, row-, channel- and block-wise): masks bit-exact against the oracle on
    shapes that reach every quantizer kernel (chunk-per-lane, block-per-lane, both row-wise kernels)."""
    M, K = shape
    pattern = oracle.keep_quarters(base, q)
    bits = synth(M + K + base + q, M, K, n_out=max(1, K // 256), extremes=base not in (oracle.S_CHAN50, oracle.S_BLOCK))
    want = oracle.quantize_residual_mask(bf16_bits_to_f32(bits), pattern, fmt)
    got = rq().residual_mask(to_dev(bits), pattern, fmt)
    torch.cuda.synchronize()
    assert np.array_equal(got["r_codes"].cpu().numpy(), want["r_codes"])
    info = want["mask_info"]
    if base in (oracle.S_CHAN50, oracle.S_BLOCK) and not (info["exact"] or info["margin"] > 2.0 ** -40):
        pytest.skip("selection scores not exactly summable and boundary margin too small")
    assert np.array_equal(got["mask"].cpu().numpy(), want["mask"])


@pytest.mark.parametrize("fmt", ["hif4", "mxfp4"])
@pytest.mark.parametrize("q", [1, 2, 3])
@pytest.mark.parametrize("shape", [(32, 64), (64, 256), (320, 2048), (2432, 192), (96, 18944), (4096, 1024)])
def test_block_selection_per_strip_bit_exact(shape, q, fmt):
    """Block pattern with the selection inside every strip of 32 token rows: codes and masks bit-exact against
    the oracle on shapes that reach both quantizer kernels, from one block per strip (nothing or everything
    kept) to 296 blocks per strip and 128 strips."""
    M, K = shape
    pattern = oracle.keep_quarters(oracle.per_strip(oracle.S_BLOCK), q)
    bits = synth(5 * M + K + q, M, K, n_out=max(1, K // 256), extremes=False)
    want = oracle.quantize_residual_mask(bf16_bits_to_f32(bits), pattern, fmt)
    got = rq().residual_mask(to_dev(bits), pattern, fmt)
    torch.cuda.synchronize()
    for key in ("x_codes", "x_side", "r_codes", "r_side"):
        assert np.array_equal(side_np(got[key]), want[key]), key
    info = want["mask_info"]
    if not (info["exact"] or info["margin"] > 2.0 ** -40):
        pytest.skip("selection scores not exactly summable and boundary margin too small")
    mask = got["mask"].cpu().numpy()
    assert np.array_equal(mask, want["mask"])
    kept = np.unpackbits(mask, axis=1, bitorder="little").reshape(M // 32, 32, K // 64, 64).all(axis=(1, 3))
    assert np.all(kept.sum(axis=1) == (K // 64) * q // 4)


def test_per_strip_flag_is_for_the_block_pattern_only():
    bits = synth(3, 64, 256)
    for base in (oracle.S_2_4, oracle.S_ROW50, oracle.S_CHAN50, oracle.S_DENSE, oracle.S_NONE):
        with pytest.raises(Exception):
            rq().residual_mask(to_dev(bits), oracle.per_strip(base), "hif4")


@pytest.mark.parametrize("fmt", ["hif4", "mxfp4"])
@pytest.mark.parametrize("shape", [(700, 4160), (416, 18944), (1300, 2048), (900, 3584)])
def test_row_selection_persistent_ctas(shape, fmt):
    """Row-wise selection with more rows than resident CTAs (each CTA or warp walks several rows, the next row
    loading while the current one is selected), for every variant: one warp per row (one and two segments),
    8-warp and 16-warp teams per row."""
    M, K = shape
    bits = synth(9 * M + K, M, K, n_out=max(1, K // 256), extremes=True)
    want = oracle.quantize_residual_mask(bf16_bits_to_f32(bits), oracle.S_ROW50, fmt)
    got = rq().residual_mask(to_dev(bits), oracle.S_ROW50, fmt)
    torch.cuda.synchronize()
    for key in ("x_codes", "x_side", "r_codes", "r_side"):
        assert np.array_equal(side_np(got[key]), want[key]), key
    assert np.array_equal(got["mask"].cpu().numpy(), want["mask"])


@pytest.mark.parametrize("q", [1, 2, 3])
@pytest.mark.parametrize("case", [(oracle.S_BLOCK, 4096, 12352), (oracle.S_CHAN50, 32, 24704)])
def test_selection_over_many_scores(case, q):
    """More than 24576 block / channel scores: the selection runs as grid-wide kernels over 16-bit digits."""
    base, M, K = case
    pattern = oracle.keep_quarters(base, q)
    bits = synth(5 * M + K + q, M, K, n_out=max(1, K // 256), extremes=False)
    want = oracle.quantize_residual_mask(bf16_bits_to_f32(bits), pattern, "hif4")
    got = rq().residual_mask(to_dev(bits), pattern, "hif4")
    torch.cuda.synchronize()
    info = want["mask_info"]
    if not (info["exact"] or info["margin"] > 2.0 ** -40):
        pytest.skip("selection scores not exactly summable and boundary margin too small")
    assert np.array_equal(got["mask"].cpu().numpy(), want["mask"])


@pytest.mark.parametrize("pattern", [oracle.S_NONE, oracle.S_2_4, oracle.S_BLOCK])
def test_many_rows_per_warp(pattern):
    """Tall, narrow input: every warp of the streaming kernel walks several rows (prefetch ring, row tail)."""
    M, K = 38400 + 32, 192
    bits = synth(11 + pattern, M, K, n_out=4, extremes=pattern != oracle.S_BLOCK)
    want = oracle.quantize_residual_mask(bf16_bits_to_f32(bits), pattern, "hif4")
    if pattern == oracle.S_NONE:
        codes, side = rq().quantize_act(to_dev(bits), "hif4")
        assert np.array_equal(codes.cpu().numpy(), want["x_codes"]) and np.array_equal(side_np(side), want["x_side"])
        return
    got = rq().residual_mask(to_dev(bits), pattern, "hif4")
    torch.cuda.synchronize()
    for key in ("x_codes", "x_side", "r_codes", "r_side"):
        assert np.array_equal(side_np(got[key]), want[key]), key
    info = want["mask_info"]
    if pattern == oracle.S_BLOCK and not (info["exact"] or info["margin"] > 2.0 ** -40):
        pytest.skip("score sum not exactly representable in fp64 for this draw")
    assert np.array_equal(got["mask"].cpu().numpy(), want["mask"])


@pytest.mark.parametrize("shape", [(64, 256), (64, 2304), (32, 24640)])
def test_residual_mask_ties_and_zero_rows(shape):
    # all-equal magnitudes: every selection is decided by the lower-index rule (the widest shape has more channel
    # scores than one CTA selects: grid-wide kernels, including their ordered pass over the ties)
    M, K = shape
    x = np.full((M, K), 0.75, dtype=np.float32)
    x[:, ::2] *= -1
    x[5] = 0
    bits = f32_to_bf16_bits(x)
    for pattern in (oracle.S_2_4, oracle.S_ROW50, oracle.S_CHAN50, oracle.S_BLOCK):
        want = oracle.quantize_residual_mask(bf16_bits_to_f32(bits), pattern)
        got = rq().residual_mask(to_dev(bits), pattern)
        assert np.array_equal(got["mask"].cpu().numpy(), want["mask"]), pattern


@pytest.mark.parametrize("cfg_idx,layer", [(0, 0), (1, 0), (1, 3), (3, 1)])
def test_config_tensors_bit_exact(cfg_idx, layer):
    cfg = CONFIGS[cfg_idx]
    bits = make_activation(cfg, layer)
    pattern = cfg.patterns[0]
    want = oracle.quantize_residual_mask(bf16_bits_to_f32(bits), pattern)
    got = rq().residual_mask(to_dev(bits), pattern)
    for k_got, k_want in (("x_codes", "x_codes"), ("r_codes", "r_codes"), ("mask", "mask")):
        assert np.array_equal(got[k_got].cpu().numpy(), want[k_want]), k_got
    assert np.array_equal(side_np(got["x_side"]), want["x_side"])
    assert np.array_equal(side_np(got["r_side"]), want["r_side"])
    if layer == 0:
        wbits = make_weight(cfg, layer)[:512]
        wc, ws = rq().pack_weight(to_dev(np.ascontiguousarray(wbits)))
        want_c, want_s = oracle.hif4_encode(bf16_bits_to_f32(wbits))
        assert np.array_equal(wc.cpu().numpy(), want_c) and np.array_equal(side_np(ws), want_s)


def test_argument_errors_are_reported_on_the_host():
    m = rq()
    x = torch.zeros((4, 96), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(m.ResqError) as e:
        m.quantize_act(x, "hif4")          # K % 64 != 0
    assert e.value.status == 2
    x = torch.zeros((40, 128), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(m.ResqError) as e:
        m.residual_mask(x, m.S_BLOCK)      # M % 32 != 0
    assert e.value.status == 2
    with pytest.raises(m.ResqError) as e:
        m.residual_mask(x, 17)
    assert e.value.status == 5
    with pytest.raises(m.ResqError) as e:
        m.residual_mask(x, m.S_CHAN50, workspace=torch.empty(256, dtype=torch.uint8, device="cuda"))
    assert e.value.status == 4
    y = torch.zeros((8, 130), dtype=torch.bfloat16, device="cuda")[:, 1:129]
    with pytest.raises(m.ResqError) as e:
        m.quantize_act(y, "hif4")          # misaligned base
    assert e.value.status == 3
