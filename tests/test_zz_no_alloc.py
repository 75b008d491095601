"""resq_residual_mask_static, the entry point for callers that cannot allocate device memory (its
selection scratch is a fixed array inside the library), must give exactly what resq_residual_mask gives
with a caller workspace: codes, metadata and masks are integer data, so the comparison is bit-exact.
Two calls in a row exercise the stale contents the shared array keeps between calls.  Collected last."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _inputs(seed, M, K):
    g = torch.Generator(device="cpu").manual_seed(seed)
    x = torch.randn((M, K), generator=g)
    x[:, ::97] *= 50.0
    return x.to(torch.bfloat16).cuda()


def _same(a, b):
    for key in ("x_codes", "x_side", "r_codes", "r_side", "mask"):
        if a[key] is None:
            assert b[key] is None
        else:
            assert torch.equal(a[key], b[key]), key


@pytest.mark.parametrize("pattern", [4, 5, 2])   # channel-wise and block-wise use the scratch; 2:4 does not
def test_static_scratch_matches_workspace_variant_twice(pattern):
    import paper_2607_26515_b200 as rq
    # first call: a large selection (leaves many scores and flags behind in the shared array) ...
    x1 = _inputs(1, 256, 4096)
    want1 = rq.residual_mask(x1, pattern)
    got1 = rq.residual_mask_static(x1, pattern)
    torch.cuda.synchronize()
    _same(want1, got1)
    # ... second call right after it: a smaller, different problem must not see the leftovers
    x2 = _inputs(2, 96, 1024)
    want2 = rq.residual_mask(x2, pattern)
    got2 = rq.residual_mask_static(x2, pattern)
    torch.cuda.synchronize()
    _same(want2, got2)
    # and the first problem again
    got1b = rq.residual_mask_static(x1, pattern)
    torch.cuda.synchronize()
    _same(want1, got1b)


@pytest.mark.parametrize("pattern", ["chan25", "block-strip", "block-strip75", "1:4"])
def test_static_scratch_takes_the_pattern_modifiers(pattern):
    """Kept share in quarters and the per-strip block rule: the same masks as the workspace variant."""
    import paper_2607_26515_b200 as rq
    pat = {"chan25": rq.keep_quarters(rq.S_CHAN50, 1), "block-strip": rq.per_strip(rq.S_BLOCK),
           "block-strip75": rq.keep_quarters(rq.per_strip(rq.S_BLOCK), 3), "1:4": rq.keep_quarters(rq.S_2_4, 1)}[pattern]
    for seed, (M, K) in enumerate([(256, 4096), (96, 1024)]):
        x = _inputs(10 + seed, M, K)
        want = rq.residual_mask(x, pat)
        got = rq.residual_mask_static(x, pat)
        torch.cuda.synchronize()
        _same(want, got)


def test_static_scratch_at_its_largest_selection():
    """32768 channel scores is the limit: accepted, and selected by the one-CTA kernel (the workspace variant uses
    the grid-wide selection from 24577 scores on): both must keep the same channels."""
    import paper_2607_26515_b200 as rq
    K = rq.STATIC_SCRATCH_MAX_SCORES
    x = _inputs(5, 32, K)
    want = rq.residual_mask(x, rq.S_CHAN50)
    for _ in range(2):
        got = rq.residual_mask_static(x, rq.S_CHAN50)
        torch.cuda.synchronize()
        _same(want, got)
    xl = torch.zeros((32, K + 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(rq.ResqError) as e:
        rq.residual_mask_static(xl, rq.S_CHAN50)
    assert e.value.status == 4


def test_static_scratch_rejects_problems_beyond_its_size():
    import paper_2607_26515_b200 as rq
    K = 64 * 1024   # 65536 channel scores > 32768
    x = torch.zeros((32, K), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(rq.ResqError) as e:
        rq.residual_mask_static(x, rq.S_CHAN50)
    assert e.value.status == 4 and "32768" in str(e.value)
    # patterns that need no scores are not limited
    out = rq.residual_mask_static(x, rq.S_2_4)
    assert out["mask"].shape == (32, K // 8)
