"""The benchmark configurations at their full sizes, in the launch configuration bench.py times.

The GPU runs the whole layer.  The oracle recomputes (a) the quantizer outputs and the selection mask of the
WHOLE activation tensor wherever the selection is not row-local (channel-wise: scores over all M rows; block-wise:
top half over all blocks of the tensor) -- codes, metadata and masks are compared bit for bit -- and (b) the
output on sampled token rows, element by element, using the oracle's own mask rows.  Row-local selections
(2:4, per-row top half, dense) need only the sampled rows.

Tolerance of Y as in test_linear_gpu.py: |y - y_ref| <= 2e-3 |y_ref| + 1e-5 sum_k |(a + r)_k w_k| (+ 2^-8 |y_ref| for
bf16 output); the raw maximum relative error is printed next to it."""
import numpy as np
import pytest
import torch

import oracle
from workloads import CONFIGS, bf16_bits_to_f32, make_activation, make_weight

pytestmark = pytest.mark.gpu

ROW_LOCAL = (oracle.S_NONE, oracle.S_DENSE, oracle.S_2_4, oracle.S_ROW50)


def rq():
    import paper_2607_26515_b200 as m
    return m


def to_dev(bits):
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def side_np(t):
    a = t.cpu().numpy()
    return a.view(np.uint32) if a.dtype == np.int32 else a


def sample_rows(M, n_random=10, seed=5):
    fixed = [0, 31, 32, 127, 128, 255, 256 % M, M - 1]
    return np.unique(np.concatenate([fixed, np.random.default_rng(seed).integers(0, M, n_random)])).astype(np.int64)


def oracle_whole_tensor_mask(xb, pattern, fmt, got, chunk=2048):
    """Oracle quantizer over the whole tensor in row chunks (rows are independent up to the selection), compared
    with the GPU's codes / metadata chunk by chunk; then the oracle's selection over the whole decoded residual."""
    M, K = xb.shape
    v = np.empty((M, K), dtype=np.float64)
    gx, gxs = got["x_codes"].cpu().numpy(), side_np(got["x_side"])
    gr, grs = got["r_codes"].cpu().numpy(), side_np(got["r_side"])
    for r0 in range(0, M, chunk):
        r1 = min(M, r0 + chunk)
        x = bf16_bits_to_f32(np.ascontiguousarray(xb[r0:r1]))
        xc, xs = oracle.encode(fmt, x)
        assert np.array_equal(gx[r0:r1], xc) and np.array_equal(gxs[r0:r1], xs), f"Q(X) rows {r0}..{r1}"
        dx = oracle.residual(x, oracle.decode(fmt, xc, xs))
        rc, rs = oracle.encode(fmt, dx)
        assert np.array_equal(gr[r0:r1], rc) and np.array_equal(grs[r0:r1], rs), f"Q(dX) rows {r0}..{r1}"
        v[r0:r1] = oracle.decode(fmt, rc, rs)
    bits, info = oracle.mask(v, pattern)
    return bits, info


def oracle_rows(xb_rows, wb, pattern, fmt, mask_rows=None):
    """Eq. (5) on a few token rows; for a tensor-wide selection the mask rows come from the whole-tensor oracle."""
    x = bf16_bits_to_f32(np.ascontiguousarray(xb_rows))
    w = bf16_bits_to_f32(wb)
    if mask_rows is None:
        o = oracle.resq_linear(x, w, pattern, fmt)
        return o["y"], o["abs_sum"]
    xc, xs = oracle.encode(fmt, x)
    a = oracle.decode(fmt, xc, xs)
    rc, rs = oracle.encode(fmt, oracle.residual(x, a))
    r_masked = oracle.apply_mask(oracle.decode(fmt, rc, rs), np.ascontiguousarray(mask_rows))
    wd = oracle.decode(fmt, *oracle.encode(fmt, w))
    return oracle.matmul(a, r_masked, wd)


def check_close(y, ref, abs_sum, bf16_out, label):
    y = np.asarray(y, dtype=np.float64)
    tol = 2e-3 * np.abs(ref) + 1e-5 * abs_sum + (2.0 ** -8 * np.abs(ref) if bf16_out else 0.0)
    err = np.abs(y - ref)
    big = np.abs(ref) > 1e-3 * abs_sum            # entries that are not the result of heavy cancellation
    rel = float((err[big] / np.abs(ref[big])).max()) if big.any() else 0.0
    print(f"{label}: max err/tol {float((err / np.maximum(tol, 1e-300)).max()):.3f}, raw max relative error {rel:.3e}")
    assert (err <= tol).all(), f"{label}: {(err > tol).sum()} of {err.size} outside tolerance"


CASES = [
    # config 2 (3B prefill, M = 8192): its named patterns on the two large layers
    (2, 2, oracle.S_ROW50, "hif4"), (2, 3, oracle.S_ROW50, "hif4"),
    (2, 2, oracle.S_CHAN50, "hif4"), (2, 3, oracle.S_CHAN50, "hif4"),
    (2, 0, oracle.S_ROW50, "mxfp4"),
    # config 3 (7B decode, M = 512): all four layers with its block pattern, selected over the whole tensor
    (3, 0, oracle.S_BLOCK, "hif4"), (3, 1, oracle.S_BLOCK, "hif4"), (3, 2, oracle.S_BLOCK, "hif4"),
    (3, 3, oracle.S_BLOCK, "hif4"),
    # config 4 (7B prefill, M = 16384): gate_up and down with 2:4 and the block pattern; one layer in MXFP4
    (4, 2, oracle.S_2_4, "hif4"), (4, 3, oracle.S_2_4, "hif4"),
    (4, 2, oracle.S_BLOCK, "hif4"), (4, 3, oracle.S_BLOCK, "hif4"),
    (4, 0, oracle.S_2_4, "mxfp4"), (4, 1, oracle.S_DENSE, "hif4"),
]


@pytest.mark.parametrize("cfg_idx,layer,pattern,fmt", CASES)
def test_full_size_layer(cfg_idx, layer, pattern, fmt):
    m = rq()
    cfg = CONFIGS[cfg_idx]
    xb, wb = make_activation(cfg, layer), make_weight(cfg, layer)
    M, K = xb.shape
    N = wb.shape[0]
    label = f"config {cfg_idx} {cfg.layers[layer].name} M={M} K={K} N={N} {m.PATTERN_NAMES[pattern]} {fmt}"
    x = to_dev(xb)
    rows = sample_rows(M)
    mask_rows = None
    if pattern not in ROW_LOCAL:
        got = m.residual_mask(x, pattern, fmt)
        torch.cuda.synchronize()
        bits, info = oracle_whole_tensor_mask(xb, pattern, fmt, got)
        gmask = got["mask"].cpu().numpy()
        if info["exact"] or info["margin"] > 2.0 ** -40:
            assert np.array_equal(gmask, bits), f"{label}: mask differs in {(gmask != bits).sum()} bytes"
        assert int(np.unpackbits(bits).sum()) == int(np.unpackbits(gmask).sum())
        mask_rows = bits[rows]
        del got, gmask
    wc, ws = m.pack_weight(to_dev(wb), fmt)
    work = m.alloc_workspace(m.resq_workspace_bytes(M, N, K, pattern, fmt))
    y = m.resq_linear(x, wc, ws, pattern, fmt, out_dtype=torch.bfloat16, workspace=work)
    assert m.check(work) == 0, m.last_error()
    got_y = y[torch.from_numpy(rows).cuda()].float().cpu().numpy()
    del y, work
    torch.cuda.empty_cache()
    ref, abs_sum = oracle_rows(xb[rows], wb, pattern, fmt, mask_rows)
    check_close(got_y, ref, abs_sum, True, label)
