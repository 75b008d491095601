"""Pins for the CPU oracle: what the paper and the mathematics fix, checked without a GPU.

Each test is chosen so that a plausible mistake in the oracle (dropped term, wrong sign or
index, transposed operand, wrong tie rule) fails at least one of them.  Nothing here retypes
the oracle's own loops: properties are stated independently (exact rationals, brute force,
library routines, hand-derived values).
"""
import itertools
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle
from workloads import bf16_bits_to_f32, f32_to_bf16_bits

GOLD = os.path.join(os.path.dirname(__file__), "golden")
F = Fraction


def nibbles(codes):
    c = np.asarray(codes, dtype=np.uint8)
    return np.stack([c & 15, c >> 4], axis=-1).reshape(c.shape[0], -1)


def bf16_round(x):
    return bf16_bits_to_f32(f32_to_bf16_bits(np.asarray(x, dtype=np.float32)))


def gaussian_with_outliers(seed, rows, K, n_out=4, scale=64.0):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((rows, K)).astype(np.float32)
    ch = rng.choice(K, n_out, replace=False)
    x[:, ch] *= scale
    return bf16_round(x)


# ----------------------------------------------------------------- tables (Section 3)

def test_s1p2_equals_e1m2_table():
    # E1M2 with bias 1: exponent bit 0 -> subnormal 0.mm, exponent bit 1 -> 1.mm (times 2^0)
    for code in range(16):
        e, m = (code >> 2) & 1, code & 3
        mag = F(m, 4) if e == 0 else 1 + F(m, 4)
        want = -mag if code & 8 else mag
        assert F(oracle.s1p2_value(code)) == want
    assert [oracle.s1p2_value(q) for q in range(8)] == [0, .25, .5, .75, 1, 1.25, 1.5, 1.75]


def test_e6m2_table_structure():
    vals = [F(oracle.e6m2_value(s)) for s in range(256)]
    assert all(b > a for a, b in zip(vals, vals[1:]))            # codes are monotone in value
    assert vals[48 << 2] == 1                                    # bias 48
    for s in range(256):
        E, Mn = s >> 2, s & 3
        assert vals[s] == F(4 + Mn, 4) * F(2) ** (E - 48)
    assert vals[0] == F(2) ** -48 and vals[255] == F(7, 4) * 2 ** 15


def test_e2m1_e8m0_tables_match_library(nvref):
    for c in range(16):
        assert oracle.e2m1_value(c) == nvref.nv_e2m1_to_float(c)
        assert np.signbit(oracle.e2m1_value(c)) == bool(c & 8)
    for c in range(255):
        assert oracle.e8m0_value(c) == nvref.nv_e8m0_to_float(c)


def test_e8m0_table_matches_torch():
    import torch
    b = torch.arange(255, dtype=torch.uint8)
    v = b.view(torch.float8_e8m0fnu).to(torch.float32).numpy()
    assert all(oracle.e8m0_value(c) == float(v[c]) for c in range(255))


# ----------------------------------------------------------------- golden worked example

def _load_worked_example():
    rows, mask, mx, meta = [], None, [], {}
    with open(os.path.join(GOLD, "hif4_worked_example.txt")) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if not line:
                continue
            t = line.split()
            if t[0] in ("meta_x", "meta_r"):
                meta[t[0]] = int(t[1], 16)
            elif t[0] == "mask":
                mask = [int(v, 16) for v in t[1:]]
            elif t[0] == "mx_scale":
                meta["mx_scale"] = [int(v) for v in t[1:]]
            elif t[0] == "mx":
                mx.append((int(t[1]), int(t[2])))
            else:
                rows.append((int(t[0]), float(t[1]), int(t[2]), float(t[3]), float(t[4]), int(t[5]), float(t[6])))
    return rows, mask, mx, meta


def test_worked_example_hif4_residual_mask():
    rows, mask, mx, meta = _load_worked_example()
    x = np.zeros((1, 64), dtype=np.float32)
    for k, xv, *_ in rows:
        x[0, k] = xv
    out = oracle.quantize_residual_mask(x, oracle.S_2_4)
    assert int(out["x_side"][0, 0]) == meta["meta_x"]
    assert int(out["r_side"][0, 0]) == meta["meta_r"]
    qx, qr = nibbles(out["x_codes"])[0], nibbles(out["r_codes"])[0]
    listed = set()
    for k, xv, cx, dqx, dx, cr, dqr in rows:
        listed.add(k)
        assert qx[k] == cx, k
        assert out["a"][0, k] == dqx and np.signbit(out["a"][0, k]) == np.signbit(dqx)
        assert out["dx"][0, k] == dx
        assert qr[k] == cr, k
        assert out["r"][0, k] == dqr
    for k in range(64):
        if k not in listed:
            assert qx[k] == 0 and qr[k] == 0
    assert list(out["mask"][0]) == mask


def test_worked_example_mxfp4():
    rows, mask, mx, meta = _load_worked_example()
    x = np.zeros((1, 64), dtype=np.float32)
    for k, xv, *_ in rows:
        x[0, k] = xv
    codes, scale = oracle.mxfp4_encode(x)
    assert list(scale[0]) == meta["mx_scale"]
    q = nibbles(codes)[0]
    for k, c in mx:
        assert q[k] == c, k


# ----------------------------------------------------------------- HiF4 invariants (exact rationals)

def _hif4_check_block(xb, cb, meta):
    """No-clip, minimality and nearest-with-ties-to-even, stated as properties over exact rationals."""
    s = meta & 255
    S1 = F(4 + (s & 3), 4) * F(2) ** ((s >> 2) - 48)
    ax = [abs(F(float(v))) for v in xb]
    amax = max(ax)
    if amax == 0:
        assert s == 0
    else:
        if s < 255:
            assert 7 * S1 >= amax                                   # level 1 does not clip
        if s > 0:
            sp = s - 1
            assert 7 * F(4 + (sp & 3), 4) * F(2) ** ((sp >> 2) - 48) < amax   # ... and is minimal
    for i in range(8):
        e2 = (meta >> (8 + i)) & 1
        g8 = max(ax[8 * i: 8 * i + 8])
        # e2 = 0 would allow at most 1.75 * 2 * S1 (with e3 = 1)
        assert (e2 == 1) == (g8 > F(7, 2) * S1)
        for jj in range(2):
            j = 2 * i + jj
            e3 = (meta >> (16 + j)) & 1
            g4 = max(ax[4 * j: 4 * j + 4])
            top = F(7, 4) * S1 * 2 ** (e2 + e3)
            if s < 255:
                assert g4 <= top                                     # never clips
            if e3 == 1:
                assert g4 > F(7, 4) * S1 * 2 ** e2                    # lowering e3 would clip
            step = S1 * 2 ** (e2 + e3) / 4
            for k in range(4 * j, 4 * j + 4):
                q, sign = cb[k] & 7, cb[k] >> 3
                assert sign == int(np.signbit(xb[k]))
                err = abs(ax[k] - q * step)
                if s < 255 or ax[k] <= 7 * step:
                    assert err <= step / 2
                    if err == step / 2:
                        assert q % 2 == 0                            # ties to even
                else:
                    assert q == 7                                     # saturation


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_hif4_invariants_random_blocks(seed):
    x = gaussian_with_outliers(seed, 8, 256)
    # mix in tiny, huge and exactly-zero blocks
    x[0, :64] = 0
    x[1, :64] *= np.float32(2.0 ** -60)
    x[2, :64] *= np.float32(2.0 ** 12)
    x[3, 64:128] = bf16_round(np.round(x[3, 64:128] * 4) / 4)      # many exact ties
    codes, meta = oracle.hif4_encode(x)
    q = nibbles(codes)
    for r in range(x.shape[0]):
        for b in range(x.shape[1] // 64):
            _hif4_check_block(x[r, 64 * b: 64 * b + 64], q[r, 64 * b: 64 * b + 64], int(meta[r, b]))


def test_hif4_scale_saturation_and_underflow():
    x = np.zeros((2, 64), dtype=np.float32)
    x[0, 5] = 3.0e38  # far above 7 * max S1: clamps to s = 255 and q = 7
    x[1, 7] = 1e-30   # far below the smallest step: s = 0 and the element rounds to 0
    codes, meta = oracle.hif4_encode(x)
    q = nibbles(codes)
    assert meta[0, 0] & 255 == 255 and q[0, 5] == 7
    assert meta[1, 0] & 255 == 0 and q[1, 7] == 0
    d = oracle.hif4_decode(codes, meta)
    assert d[0, 5] == 7 * 1.75 * 2.0 ** 15


def test_hif4_amax_group_invariant():
    x = gaussian_with_outliers(5, 16, 512)
    codes, meta = oracle.hif4_encode(x)
    q = nibbles(codes) & 7
    for r in range(16):
        for b in range(8):
            blk = np.abs(x[r, 64 * b: 64 * b + 64])
            k = int(np.argmax(blk))
            m = int(meta[r, b])
            if m & 255:
                # 7*S1(s-1) < amax and S1(s)/S1(s-1) <= 1.25  =>  amax > 5.6 * S1: top group uses both exponents
                assert (m >> (8 + k // 8)) & 1 == 1 and (m >> (16 + k // 4)) & 1 == 1
                assert q[r, 64 * b + k] >= 6


def representable_hif4_blocks(seed, G, s_lo=1, s_hi=255):
    """G blocks of values that ARE HiF4 values under scales that satisfy the encoder's own
    minimality rules (every raised exponent is needed, the level-1 scale is the smallest that
    covers the maximum), so that re-encoding must reproduce exactly these bits."""
    rng = np.random.default_rng(seed)
    x = np.zeros(64 * G, dtype=np.float64)
    want_meta = np.zeros(G, dtype=np.uint32)
    want_q = np.zeros(64 * G, dtype=np.uint8)
    for b in range(G):
        s = int(rng.integers(s_lo, s_hi))
        S1 = float(F(4 + (s & 3), 4) * F(2) ** ((s >> 2) - 48))
        e3 = rng.integers(0, 2, 16)
        q = rng.integers(0, 8, 64)
        sign = rng.integers(0, 2, 64)
        top = int(rng.integers(0, 16))          # the 4-group that holds the block maximum 7*S1
        e3[top] = 1
        q[4 * top] = 7
        # a raised level-2 exponent needs a raised level-3 group below it
        e2 = np.array([int(rng.integers(0, 2)) if (e3[2 * i] or e3[2 * i + 1]) else 0 for i in range(8)])
        e2[top // 2] = 1
        for j in range(16):
            if e3[j]:
                q[4 * j + 1] = max(q[4 * j + 1], 4)   # the raised exponent must be needed (q >= 4)
        want_meta[b] = s | sum(int(e2[i]) << (8 + i) for i in range(8)) | sum(int(e3[j]) << (16 + j) for j in range(16))
        for k in range(64):
            v = q[k] / 4.0 * 2.0 ** (int(e2[k // 8]) + int(e3[k // 4])) * S1
            x[64 * b + k] = -v if sign[k] else v
            want_q[64 * b + k] = (sign[k] << 3) | q[k]
    return x, want_meta, want_q


def test_hif4_round_trip_of_representable_blocks():
    G = 200
    x, want_meta, want_q = representable_hif4_blocks(7, G)
    x = x.reshape(1, -1)
    xf = x.astype(np.float32)
    assert np.array_equal(xf.astype(np.float64), x)                 # representable values are fp32-exact
    codes, meta = oracle.hif4_encode(xf)
    assert np.array_equal(meta[0], want_meta)
    assert np.array_equal(nibbles(codes)[0], want_q)
    assert np.array_equal(oracle.hif4_decode(codes, meta), x)       # decode inverts it
    # and the residual of a representable tensor is identically zero (Eq. 3)
    assert not np.any(oracle.residual(xf, oracle.hif4_decode(codes, meta)))


def test_hif4_rne_and_monotone_sweep():
    # block whose scales are pinned by one element of magnitude 7 (S1 = 1, e2 = e3 = 1 in group 0);
    # the probe sits in group 8 (e2 = e3 = 0 as long as it stays <= 1.75): step 1/4.
    probes = np.arange(0, 1.75 + 1 / 64, 1 / 64)
    x = np.zeros((len(probes), 64), dtype=np.float32)
    x[:, 0] = 7.0
    x[:, 40] = probes
    codes, meta = oracle.hif4_encode(x)
    assert np.all(meta == ((48 << 2) | (1 << 8) | (1 << 16)))
    q = nibbles(codes)[:, 40]
    assert np.all(np.diff(q.astype(int)) >= 0)
    for p, qq in zip(probes, q):
        t = F(float(p)) * 4
        if t.denominator == 2:                    # exact midpoint -> even
            assert qq % 2 == 0 and abs(qq - t) == F(1, 2)
        else:
            assert qq == round(t)
    # negative probes mirror
    x[:, 40] = -probes
    codes2, _ = oracle.hif4_encode(x)
    assert np.array_equal(nibbles(codes2)[:, 40], q | 8)


def test_packing_nibble_order_and_meta_bits():
    x = np.zeros((1, 64), dtype=np.float32)
    x[0, 0], x[0, 1] = 1.75, -0.25          # S1 = 0.25 (7*.25 = 1.75): q0 = 7 at e2=e3=1 in group 0
    codes, meta = oracle.hif4_encode(x)
    # element 0 -> low nibble, element 1 -> high nibble of byte 0
    assert codes[0, 0] & 15 == 7
    assert codes[0, 0] >> 4 == (8 | 1)      # step in the raised group is 0.25*4/4 = 0.25 -> q = 1, negative
    assert int(meta[0, 0]) & 255 == (46 << 2)
    assert (int(meta[0, 0]) >> 8) & 255 == 1 and int(meta[0, 0]) >> 16 == 1


# ----------------------------------------------------------------- MXFP4

def test_mxfp4_element_rounding_matches_library(nvref):
    # block scale pinned to 2^0 by an element of 4.0; the probe must not exceed 8 (would change the scale)
    probes = np.concatenate([np.arange(0, 7.99, 1 / 32), [0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0, 6.0, 7.0, 7.9]])
    probes = probes.astype(np.float32)
    x = np.zeros((len(probes), 32), dtype=np.float32)
    x[:, 0] = 4.0
    x[:, 9] = probes
    x[1::2, 9] *= -1
    codes, scale = oracle.mxfp4_encode(x)
    assert np.all(scale == 127)
    q = nibbles(codes)[:, 9]
    for i, p in enumerate(x[:, 9]):
        assert int(q[i]) == nvref.nv_float_to_e2m1(float(p)), p


def test_mxfp4_scale_property():
    x = gaussian_with_outliers(11, 8, 256)
    x[0, :32] = 0
    codes, scale = oracle.mxfp4_encode(x)
    for r in range(8):
        for b in range(8):
            amax = float(np.abs(x[r, 32 * b: 32 * b + 32]).max())
            if amax == 0:
                assert scale[r, b] == 0
                continue
            t = F(amax) / F(2) ** (int(scale[r, b]) - 127)
            assert 4 <= t < 8                      # the block maximum lands in E2M1's top binade
    d = oracle.mxfp4_decode(codes, scale)
    # decode is value(code) * 2^(scale-127), checked against the tables
    q = nibbles(codes)
    for (r, k) in [(1, 3), (2, 77), (7, 255)]:
        assert d[r, k] == oracle.e2m1_value(int(q[r, k])) * oracle.e8m0_value(int(scale[r, k // 32]))


def test_mxfp4_round_trip():
    rng = np.random.default_rng(3)
    G = 64
    sc = rng.integers(100, 150, G)
    q = rng.integers(0, 16, (G, 32))
    q[:, 0] = 7 - (rng.integers(0, 2, G))          # top binade present (6 or 4): scale is recoverable
    x = np.zeros((1, 32 * G))
    for b in range(G):
        for k in range(32):
            x[0, 32 * b + k] = oracle.e2m1_value(int(q[b, k])) * oracle.e8m0_value(int(sc[b]))
    codes, scale = oracle.mxfp4_encode(x.astype(np.float32))
    assert np.array_equal(scale[0], sc)
    assert np.array_equal(nibbles(codes)[0], q.reshape(-1))
    # and back: the decoder returns every value the blocks were built from (the sign of -0 included)
    d = oracle.mxfp4_decode(codes, scale)
    assert d.shape == x.shape and np.array_equal(d, x)
    assert np.array_equal(np.signbit(d), np.signbit(x))
    # decoding codes that no encoder produced (arbitrary nibbles under arbitrary scales, code 0 and 254 included)
    # is value(code) * 2^(scale - 127), element by element
    rng2 = np.random.default_rng(4)
    codes2 = rng2.integers(0, 256, (3, 64), dtype=np.uint8)
    scale2 = np.array([[0, 1, 126, 254], [127, 128, 200, 60], [5, 250, 127, 127]], dtype=np.uint8)
    d2 = oracle.mxfp4_decode(codes2, scale2)
    q2 = nibbles(codes2)
    for r in range(3):
        for k in range(128):
            want = F(oracle.e2m1_value(int(q2[r, k]))) * F(2) ** (int(scale2[r, k // 32]) - 127)
            assert F(float(d2[r, k])) == want


def test_hif4_is_more_accurate_than_mxfp4_on_outlier_data():
    x = gaussian_with_outliers(21, 32, 1024, n_out=6)
    xd = x.astype(np.float64)
    eh = np.linalg.norm(xd - oracle.hif4_decode(*oracle.hif4_encode(x)))
    em = np.linalg.norm(xd - oracle.mxfp4_decode(*oracle.mxfp4_encode(x)))
    assert eh < em


# ----------------------------------------------------------------- residual (Eq. 3) and bounds

@pytest.mark.parametrize("fmt", ["hif4", "mxfp4"])
def test_residual_identity_and_bound(fmt):
    x = gaussian_with_outliers(4, 16, 512)
    o = oracle.quantize_residual_mask(x, oracle.S_DENSE, fmt)
    xd = x.astype(np.float64)
    assert np.array_equal(o["dx"].astype(np.float64), xd - o["a"])          # Eq. (3), exactly
    # the second quantization shrinks the error: ||x - a - r|| < ||x - a||
    assert np.linalg.norm(xd - o["a"] - o["r"]) < 0.25 * np.linalg.norm(xd - o["a"])
    if fmt == "hif4":
        # |dx - r| <= step_r / 2 for every element (no clipping in the residual encode)
        meta = o["r_side"]
        for r in range(4):
            for k in range(0, 512, 37):
                m = int(meta[r, k // 64])
                kk = k % 64
                S1 = oracle.e6m2_value(m & 255)
                step = S1 * 2.0 ** (((m >> (8 + kk // 8)) & 1) + ((m >> (16 + kk // 4)) & 1)) / 4
                assert abs(float(o["dx"][r, k]) - o["r"][r, k]) <= step / 2


def test_outliers_collapse_their_block_to_zero():
    # Figure 1's effect: an outlier forces a large scale and the bulk of its block underflows
    rng = np.random.default_rng(9)
    x = bf16_round(rng.standard_normal((64, 64)).astype(np.float32))
    xo = x.copy()
    xo[:, 17] *= 64
    z = lambda c: float(((nibbles(c) & 7) == 0).mean())
    z_plain = z(oracle.hif4_encode(x)[0])
    z_out = z(oracle.hif4_encode(xo)[0])
    assert z_out > 0.5 > z_plain


# ----------------------------------------------------------------- masks (Section 4.3)

def _bits_to_bool(bits, K):
    return np.unpackbits(bits, axis=1, bitorder="little")[:, :K].astype(bool)


@pytest.mark.parametrize("fmt", ["hif4", "mxfp4"])
def test_mask_counts(fmt):
    M, K = 64, 256
    x = gaussian_with_outliers(31, M, K)
    for pattern in (oracle.S_2_4, oracle.S_ROW50, oracle.S_CHAN50, oracle.S_BLOCK, oracle.S_DENSE):
        o = oracle.quantize_residual_mask(x, pattern, fmt)
        mb = _bits_to_bool(o["mask"], K)
        if pattern == oracle.S_2_4:
            assert np.all(mb.reshape(M, K // 4, 4).sum(-1) == 2)
        elif pattern == oracle.S_ROW50:
            assert np.all(mb.sum(1) == K // 2)
        elif pattern == oracle.S_CHAN50:
            assert mb[0].sum() == K // 2 and np.all(mb == mb[0])
        elif pattern == oracle.S_BLOCK:
            blk = mb.reshape(M // 32, 32, K // 64, 64).transpose(0, 2, 1, 3).reshape(-1, 32 * 64)
            assert np.all((blk.sum(1) == 0) | (blk.sum(1) == 2048))
            assert (blk.sum(1) == 2048).sum() == (M // 32) * (K // 64) // 2
        else:
            assert mb.all()
        # kept entries keep their value, dropped ones are zero
        assert np.array_equal(o["r_masked"], np.where(mb, o["r"], 0.0))


def _check_topk_valid(keys, kept):
    """No dropped key exceeds a kept one; among equal boundary keys the lower index is kept."""
    keys, kept = np.asarray(keys), np.asarray(kept, dtype=bool)
    if kept.all() or not kept.any():
        return
    lo = keys[kept].min()
    hi = keys[~kept].max()
    assert hi <= lo
    if hi == lo:
        tied = np.nonzero(keys == lo)[0]
        kt = kept[tied]
        assert np.all(np.diff(kt.astype(int)) <= 0)      # kept ties come first


def test_mask_optimality_bruteforce_small():
    rng = np.random.default_rng(5)
    M, K = 32, 128
    # few distinct magnitudes => many ties
    v = rng.integers(-3, 4, (M, K)).astype(np.float64) * 0.25
    bits, _ = oracle.mask(v, oracle.S_2_4)
    mb = _bits_to_bool(bits, K)
    for m in range(M):
        for g in range(K // 4):
            grp = np.abs(v[m, 4 * g: 4 * g + 4])
            # brute force over the 6 ways to keep 2 of 4: the kept set has the maximal key sum and,
            # among those, the lexicographically smallest positions
            best = max(itertools.combinations(range(4), 2), key=lambda c: (grp[list(c)].sum(), [-i for i in c]))
            assert tuple(np.nonzero(mb[m, 4 * g: 4 * g + 4])[0]) == best
    bits, _ = oracle.mask(v, oracle.S_ROW50)
    mb = _bits_to_bool(bits, K)
    for m in range(M):
        _check_topk_valid(np.abs(v[m]), mb[m])
    bits, info = oracle.mask(v, oracle.S_CHAN50, want_scores=True)
    mb = _bits_to_bool(bits, K)
    assert np.array_equal(info["scores"], (v ** 2).sum(0)) and info["exact"]
    _check_topk_valid((v ** 2).sum(0), mb[0])
    M2, K2 = 128, 256
    v2 = rng.integers(-2, 3, (M2, K2)).astype(np.float64)
    bits, info = oracle.mask(v2, oracle.S_BLOCK, want_scores=True)
    mb = _bits_to_bool(bits, K2)
    sc = (v2 ** 2).reshape(M2 // 32, 32, K2 // 64, 64).sum((1, 3)).reshape(-1)
    assert np.array_equal(info["scores"], sc)
    kept_blk = mb.reshape(M2 // 32, 32, K2 // 64, 64)[:, 0, :, 0].reshape(-1)
    _check_topk_valid(sc, kept_blk)
    assert kept_blk.sum() == len(sc) // 2


def test_block_orientation_is_32_rows_by_64_columns():
    v = np.zeros((64, 128))
    v[0:32, 64:128] = 1.0      # one hot block at block-row 0, block-col 1
    v[32:64, 0:64] = 0.5       # a weaker one at block-row 1, block-col 0
    bits, _ = oracle.mask(v, oracle.S_BLOCK)
    mb = _bits_to_bool(bits, 128)
    assert mb[0:32, 64:128].all() and mb[32:64, 0:64].all() and mb.sum() == 2 * 2048


def test_sparsifying_the_residual_costs_less_than_sparsifying_the_activation():
    # Figure 4's observation, on synthetic data: 2:4 on Q(dX) loses less (absolute MSE) than 2:4 on Q(X)
    x = gaussian_with_outliers(41, 32, 1024, n_out=6)
    o = oracle.quantize_residual_mask(x, oracle.S_2_4)
    a_bits, _ = oracle.mask(o["a"], oracle.S_2_4)
    mse_a = np.mean((o["a"] - oracle.apply_mask(o["a"], a_bits)) ** 2)
    mse_r = np.mean((o["r"] - o["r_masked"]) ** 2)
    assert mse_r < mse_a


# ----------------------------------------------------------------- product (Eqs. 1, 4, 5)

def _to_frac(a):
    return [[F(float(v)) for v in row] for row in a]


@pytest.mark.parametrize("fmt", ["hif4", "mxfp4"])
@pytest.mark.parametrize("pattern", [oracle.S_NONE, oracle.S_DENSE, oracle.S_2_4])
def test_matmul_exact_rational_tiny(fmt, pattern):
    M, K, N = 3, 128, 5
    x = gaussian_with_outliers(51, M, K, n_out=2, scale=16.0)
    rng = np.random.default_rng(52)
    w = bf16_round(rng.standard_normal((N, K)).astype(np.float32) * 0.02)
    o = oracle.resq_linear(x, w, pattern, fmt)
    a, wv = _to_frac(o["a"]), _to_frac(o["w"])
    r = _to_frac(o["r_masked"]) if pattern != oracle.S_NONE else [[F(0)] * K for _ in range(M)]
    for m in range(M):
        for n in range(N):
            exact = sum((a[m][k] + r[m][k]) * wv[n][k] for k in range(K))
            # fp64 over 128 exact products of ~12-bit significands with a narrow exponent range is exact
            assert F(float(o["y"][m, n])) == exact
            # the cancellation floor of every Y tolerance, sum_k |(a + r)_k w_k|, is exact on these sizes too: a value
            # that is too large by any factor would loosen every GPU parity test unnoticed
            exact_abs = sum(abs((a[m][k] + r[m][k]) * wv[n][k]) for k in range(K))
            assert F(float(o["abs_sum"][m, n])) == exact_abs
            assert exact_abs >= abs(exact)
    assert o["y"].shape == (M, N) and o["abs_sum"].shape == (M, N)


def test_matmul_reduces_to_numpy_when_residual_vanishes():
    rng = np.random.default_rng(61)
    M, K, N = 8, 256, 12
    # X made of decoded codes => Q(X) = X, dX = 0, every S gives the same Y = X W^T (Eqs. 1, 4, 5 coincide)
    # (level-1 codes limited to 2^-8 .. 2^4 so that the fp64 sums stay well conditioned)
    xq = representable_hif4_blocks(62, M * K // 64, 40 << 2, 52 << 2)[0].reshape(M, K).astype(np.float32)
    assert np.array_equal(oracle.hif4_decode(*oracle.hif4_encode(xq)), xq.astype(np.float64))
    w = bf16_round(rng.standard_normal((N, K)).astype(np.float32) * 0.02)
    wq = oracle.hif4_decode(*oracle.hif4_encode(w))
    ref = xq.astype(np.float64) @ wq.T
    for pattern in (oracle.S_NONE, oracle.S_DENSE, oracle.S_2_4, oracle.S_ROW50):
        o = oracle.resq_linear(xq, w, pattern)
        np.testing.assert_allclose(o["y"], ref, rtol=1e-13, atol=1e-13)


def test_dense_is_eq4_and_none_is_eq1():
    x = gaussian_with_outliers(71, 8, 256)
    rng = np.random.default_rng(72)
    w = bf16_round(rng.standard_normal((16, 256)).astype(np.float32) * 0.02)
    o_none = oracle.resq_linear(x, w, oracle.S_NONE)
    o_dense = oracle.resq_linear(x, w, oracle.S_DENSE)
    np.testing.assert_allclose(o_none["y"], o_none["a"] @ o_none["w"].T, rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(o_dense["y"], o_dense["a"] @ o_dense["w"].T + o_dense["r"] @ o_dense["w"].T,
                               rtol=1e-13, atol=1e-13)
    # and the correction does what the paper says it does: it moves Y toward X deq(W)^T
    target = x.astype(np.float64) @ o_none["w"].T
    o_24 = oracle.resq_linear(x, w, oracle.S_2_4)
    e0 = np.linalg.norm(o_none["y"] - target)
    e24 = np.linalg.norm(o_24["y"] - target)
    ed = np.linalg.norm(o_dense["y"] - target)
    assert ed < e24 < e0


@pytest.mark.parametrize("fmt", ["hif4", "mxfp4"])
def test_w4a16_exact_rational_tiny_and_limit_of_the_residual_series(fmt):
    """Weight-only ablation (Table 1): exact rational check of the product on a tiny case; and it is what the
    two-term product approaches: for activations that are already decoded codes (zero residual) the W4A4 path
    and the W4A16 path coincide, otherwise W4A16 is the target that the residual term moves Y toward."""
    M, K, N = 3, 128, 4
    x = gaussian_with_outliers(81, M, K, n_out=2, scale=16.0)
    rng = np.random.default_rng(82)
    w = bf16_round(rng.standard_normal((N, K)).astype(np.float32) * 0.02)
    o = oracle.w4a16_linear(x, w, fmt)
    xv, wv = _to_frac(x.astype(np.float64)), _to_frac(o["w"])
    for m in range(M):
        for n in range(N):
            assert F(float(o["y"][m, n])) == sum(xv[m][k] * wv[n][k] for k in range(K))
    full = oracle.resq_linear(x, w, oracle.S_DENSE, fmt)
    none = oracle.resq_linear(x, w, oracle.S_NONE, fmt)
    assert np.linalg.norm(full["y"] - o["y"]) < np.linalg.norm(none["y"] - o["y"])
    xq = oracle.decode(fmt, *oracle.encode(fmt, x)).astype(np.float32)
    if np.array_equal(oracle.decode(fmt, *oracle.encode(fmt, xq)), xq.astype(np.float64)):
        same = oracle.resq_linear(xq, w, oracle.S_2_4, fmt)
        np.testing.assert_allclose(same["y"], oracle.w4a16_linear(xq, w, fmt)["y"], rtol=1e-13, atol=1e-13)


@pytest.mark.parametrize("fmt", ["hif4", "mxfp4"])
def test_w16a4_exact_rational_tiny_and_fixed_points(fmt):
    """Activation-only ablation (Table 1): the product is the exact rational sum over the decoded activation codes
    (and kept residual codes) and the weights as given; activations that are already decoded codes pass through
    unchanged, so the result is then the plain product X W^T; and with identity weights the output is the decoded
    operand itself."""
    M, K, N = 3, 128, 4
    x = gaussian_with_outliers(91, M, K, n_out=2, scale=16.0)
    rng = np.random.default_rng(92)
    w = bf16_round(rng.standard_normal((N, K)).astype(np.float32) * 0.02)
    for pattern in (oracle.S_NONE, oracle.S_2_4, oracle.S_DENSE):
        o = oracle.w16a4_linear(x, w, pattern, fmt)
        av, wv = _to_frac(o["a"]), _to_frac(w.astype(np.float64))
        rv = _to_frac(o["r_masked"]) if pattern != oracle.S_NONE else None
        for m in range(M):
            for n in range(N):
                want = sum(av[m][k] * wv[n][k] for k in range(K))
                if rv is not None:
                    want += sum(rv[m][k] * wv[n][k] for k in range(K))
                assert F(float(o["y"][m, n])) == want
    xq = oracle.decode(fmt, *oracle.encode(fmt, x)).astype(np.float32)
    if np.array_equal(oracle.decode(fmt, *oracle.encode(fmt, xq)), xq.astype(np.float64)):
        o = oracle.w16a4_linear(xq, w, oracle.S_DENSE, fmt)
        np.testing.assert_allclose(o["y"], xq.astype(np.float64) @ w.astype(np.float64).T, rtol=1e-13, atol=1e-13)
    eye = np.eye(K, dtype=np.float32)
    o = oracle.w16a4_linear(x, eye, oracle.S_2_4, fmt)
    assert np.array_equal(o["y"], o["a"] + o["r_masked"])
    # the weights really stay unquantized: a weight between two 4-bit codes changes W4A4 but not this path's use of it
    w_off = bf16_round(w * np.float32(1.0078125))
    assert not np.array_equal(oracle.w16a4_linear(x, w_off, oracle.S_NONE, fmt)["y"], oracle.w16a4_linear(x, w, oracle.S_NONE, fmt)["y"])


def test_swiglu_producer_fixed_procedure():
    """Fused producer of the down projection: SiLU by the fixed fp32 procedure agrees with the closed form
    g / (1 + exp(-g)) in fp64 to fp32 accuracy; exact special cases; the product with `up` is a bf16 value; and the
    fused layer is Eq. (5) on exactly that tensor."""
    g = np.concatenate([np.linspace(-30, 30, 20001), np.random.default_rng(5).standard_normal(20000) * 4]).astype(np.float32)
    g = bf16_round(g)
    s = oracle.silu32(g).astype(np.float64)
    ref = g.astype(np.float64) / (1.0 + np.exp(-g.astype(np.float64)))
    assert np.all(np.abs(s - ref) <= 3e-6 * np.abs(ref) + 1e-37)
    assert oracle.silu32(np.float32(0.0)) == 0.0
    big = np.array([90.0, 128.0, 3.0e4], dtype=np.float32)
    assert np.array_equal(oracle.silu32(big), big)                    # exp(-g) vanishes against 1
    tiny = oracle.silu32(np.array([-90.0, -1.0e3], dtype=np.float32))
    assert np.all(tiny <= 0) and np.all(tiny > -1e-30)                # saturates at g * 2^-126
    assert np.all(np.diff(oracle.silu32(np.linspace(-1.0, 30, 4001).astype(np.float32))) >= 0)   # monotone right of the minimum
    u = bf16_round(np.random.default_rng(6).standard_normal(g.shape).astype(np.float32))
    x = oracle.swiglu_bf16(g, u)
    assert np.array_equal(bf16_round(x), x)
    exact = ref * u.astype(np.float64)
    assert np.all(np.abs(x - exact) <= 2.0 ** -8 * np.abs(exact) + 1e-37)   # half a bf16 ulp plus the fp32 error
    one = oracle.swiglu_bf16(g, np.ones_like(g))
    assert np.array_equal(one, bf16_round(oracle.silu32(g)))
    M, K, N = 4, 128, 3
    gu = bf16_round(np.random.default_rng(7).standard_normal((M, 2 * K)).astype(np.float32) * 2)
    w = bf16_round(np.random.default_rng(8).standard_normal((N, K)).astype(np.float32) * 0.02)
    o = oracle.swiglu_resq_linear(gu, w, oracle.S_2_4)
    assert np.array_equal(o["x"], oracle.swiglu_bf16(gu[:, :K], gu[:, K:]))
    assert np.array_equal(o["y"], oracle.resq_linear(o["x"], w, oracle.S_2_4)["y"])


def test_rmsnorm_producer_fixed_procedure():
    """Fused RMSNorm producer: the row scale against exact rational arithmetic (sum of squares exact, one rounding
    to fp32, then correctly rounded fp32 operations), closed-form cases, and the bf16 output against the fp64
    definition."""
    import math
    rng = np.random.default_rng(11)
    h = bf16_round(rng.standard_normal((6, 96)).astype(np.float32) * np.float32(3.0))
    h[1] *= np.float32(2.0 ** 40)       # the scale must not depend on the magnitude class of the row
    h[2] = 0.0
    eps = 1e-6
    r = oracle.rmsnorm_row_scale(h, eps)
    for m in range(h.shape[0]):
        exact_ss = sum(F(float(v)) * F(float(v)) for v in h[m])
        ss32 = np.float32(float(exact_ss))                      # Fraction -> float is correctly rounded; -> fp32 once more
        if float(np.float64(float(exact_ss))) == float(exact_ss):   # exactly representable in fp64: no double rounding
            v = np.float32(np.float32(ss32 / np.float32(96)) + np.float32(eps))
            want = np.float32(np.float32(1.0) / np.float32(math.sqrt(float(v))))   # fp64 sqrt of an fp32 value rounds correctly to fp32
            assert r[m] == want
    assert r[2] == np.float32(np.float32(1.0) / np.sqrt(np.float32(eps)))          # zero row: 1 / sqrt(eps)
    const = np.full((1, 64), 2.0, dtype=np.float32)
    assert oracle.rmsnorm_row_scale(const, 0.0)[0] == np.float32(0.5)                # mean square 4 -> 1/2 exactly
    assert np.array_equal(oracle.rmsnorm_bf16(const, np.full(64, 3.0, np.float32), 0.0), np.full((1, 64), 3.0, np.float32))
    gamma = bf16_round(1.0 + 0.1 * rng.standard_normal(96).astype(np.float32))
    x = oracle.rmsnorm_bf16(h, gamma, eps)
    assert np.array_equal(bf16_round(x), x)
    h64 = h.astype(np.float64)
    ref = h64 / np.sqrt((h64 ** 2).mean(axis=1, keepdims=True) + eps) * gamma.astype(np.float64)
    assert np.all(np.abs(x - ref) <= 2.0 ** -8 * np.abs(ref) + 1e-30)
    w = bf16_round(rng.standard_normal((3, 96)).astype(np.float32) * 0.02)
    h2 = bf16_round(rng.standard_normal((4, 128)).astype(np.float32))
    g2 = bf16_round(1.0 + 0.1 * rng.standard_normal(128).astype(np.float32))
    w2 = bf16_round(rng.standard_normal((3, 128)).astype(np.float32) * 0.02)
    o = oracle.rmsnorm_resq_linear(h2, g2, eps, w2, oracle.S_2_4)
    assert np.array_equal(o["y"], oracle.resq_linear(oracle.rmsnorm_bf16(h2, g2, eps), w2, oracle.S_2_4)["y"])


def test_randomized_hadamard_transform():
    """Rotation baseline: the fast transform equals the Sylvester Hadamard matrix product (exact on small integers),
    is orthogonal (applying it twice with the signs moved to the other side returns the input; the dot product of
    two rotated vectors equals that of the originals), spreads an outlier over its block, and the rotated layer is
    Eq. (5) on the rotated operands."""
    from scipy.linalg import hadamard
    H = hadamard(64).astype(np.float64)
    rng = np.random.default_rng(21)
    signs = int(rng.integers(0, 2 ** 63)) | (1 << 63)
    s = np.array([-1.0 if (signs >> j) & 1 else 1.0 for j in range(64)])
    x = rng.integers(-8, 9, (5, 192)).astype(np.float32)
    got = oracle.rht64_bf16(x, signs)
    want = np.concatenate([(x[:, b * 64:(b + 1) * 64] * s) @ H.T / 8 for b in range(3)], axis=1)
    assert np.array_equal(got, want)                                     # small integers: every step exact
    back = oracle.rht64_bf16(got, 0) * s[None, :].repeat(3, axis=0).reshape(1, 192)   # H/8 is symmetric and orthogonal
    assert np.array_equal(back, x)
    y = rng.integers(-8, 9, (5, 192)).astype(np.float32)
    assert np.array_equal((oracle.rht64_bf16(y, signs).astype(np.float64) * got).sum(axis=1), (x.astype(np.float64) * y).sum(axis=1))
    g = bf16_round(rng.standard_normal((4, 128)).astype(np.float32))
    g[:, 7] *= 80.0
    r = oracle.rht64_bf16(g, signs).astype(np.float64)
    ref = np.concatenate([(g[:, b * 64:(b + 1) * 64].astype(np.float64) * s) @ H.T / 8 for b in range(2)], axis=1)
    assert np.all(np.abs(r - ref) <= 2.0 ** -8 * np.abs(ref) + 2.0 ** -20 * np.abs(g).max())
    crest = lambda v: np.abs(v[:, :64]).max(axis=1) / np.sqrt((v[:, :64] ** 2).mean(axis=1))
    assert np.all(crest(r) < 0.5 * crest(g.astype(np.float64)))           # the outlier is spread over its block
    w = bf16_round(rng.standard_normal((3, 128)).astype(np.float32) * 0.02)
    o = oracle.rht_resq_linear(g, w, signs, oracle.S_NONE)
    assert np.array_equal(o["y"], oracle.resq_linear(oracle.rht64_bf16(g, signs), oracle.rht64_bf16(w, signs), oracle.S_NONE)["y"])
    # what the baseline is for: on a tensor with outlier channels the rotated FP4 product is closer to the exact one
    exact = g.astype(np.float64) @ w.astype(np.float64).T
    plain = oracle.resq_linear(g, w, oracle.S_NONE)["y"]
    assert np.linalg.norm(o["y"] - exact) < np.linalg.norm(plain - exact)


@pytest.mark.parametrize("q", [1, 3])
def test_sparsity_sweep_masks(q):
    """Kept share q/4 instead of one half: exact counts for every selecting pattern, brute-force optimality (no
    kept magnitude / score is smaller than a dropped one, ties resolved toward the lower index) and nesting
    (the kept set grows with q)."""
    rng = np.random.default_rng(40 + q)
    M, K = 64, 256
    v = np.round(rng.standard_normal((M, K)) * 3).astype(np.float64) / 4      # many ties
    v[5] = 0.0
    def unpack(bits):
        return np.unpackbits(bits, axis=1, bitorder="little").astype(bool)
    for base in (oracle.S_2_4, oracle.S_ROW50, oracle.S_CHAN50, oracle.S_BLOCK):
        bits, _ = oracle.mask(v, oracle.keep_quarters(base, q))
        kept = unpack(bits)
        half = unpack(oracle.mask(v, base)[0])
        same = unpack(oracle.mask(v, oracle.keep_quarters(base, 2))[0])
        assert np.array_equal(half, same)
        assert np.all(kept <= half) if q == 1 else np.all(half <= kept)          # nested selections
        a = np.abs(v)
        if base == oracle.S_2_4:
            g = kept.reshape(M, K // 4, 4)
            assert np.all(g.sum(axis=2) == q)
            ag = a.reshape(M, K // 4, 4)
            for m in range(M):
                for j in range(K // 4):
                    order = sorted(range(4), key=lambda t: (-ag[m, j, t], t))
                    assert sorted(order[:q]) == list(np.nonzero(g[m, j])[0])
        elif base == oracle.S_ROW50:
            assert np.all(kept.sum(axis=1) == K * q // 4)
            for m in range(M):
                order = sorted(range(K), key=lambda t: (-a[m, t], t))
                assert sorted(order[:K * q // 4]) == list(np.nonzero(kept[m])[0])
        elif base == oracle.S_CHAN50:
            assert np.all(kept == kept[0]) and kept[0].sum() == K * q // 4
            score = (v ** 2).sum(axis=0)
            order = sorted(range(K), key=lambda t: (-score[t], t))
            assert sorted(order[:K * q // 4]) == list(np.nonzero(kept[0])[0])
        else:
            blocks = kept.reshape(M // 32, 32, K // 64, 64)
            per = blocks.all(axis=(1, 3))
            assert np.array_equal(per, blocks.any(axis=(1, 3))) and per.sum() == per.size * q // 4
            score = (v ** 2).reshape(M // 32, 32, K // 64, 64).sum(axis=(1, 3)).reshape(-1)
            order = sorted(range(score.size), key=lambda t: (-score[t], t))
            assert sorted(order[:score.size * q // 4]) == list(np.nonzero(per.reshape(-1))[0])
    with pytest.raises(ValueError):
        oracle.mask(v, oracle.S_2_4 | (4 << 8))


@pytest.mark.parametrize("q", [1, 2, 3])
def test_block_selection_per_strip(q):
    """The 32x64 block pattern with the selection inside every strip of 32 token rows: whole blocks only, exactly
    floor(nbc q / 4) per strip, no kept block of a strip scores below a dropped one of the same strip (ties to
    the lower column block), a single strip reduces to the tensor-wide selection, and strips of very different
    loudness separate the two definitions (tensor-wide keeps the loud strips whole, per-strip keeps its share in
    each)."""
    rng = np.random.default_rng(70 + q)
    M, K = 128, 640                                                            # 4 strips x 10 column blocks
    v = np.round(rng.standard_normal((M, K)) * 2).astype(np.float64) / 2
    v[32:64] = 0.0                                                             # a strip of ties at zero
    v[64:96, 64:192] = v[64:96, 192:320]                                       # equal scores inside a strip
    v[96:] *= 1024.0                                                           # a loud strip
    def blocks_of(bits):
        kept = np.unpackbits(bits, axis=1, bitorder="little").astype(bool).reshape(M // 32, 32, K // 64, 64)
        per = kept.all(axis=(1, 3))
        assert np.array_equal(per, kept.any(axis=(1, 3)))                      # whole blocks only
        return per
    pat = oracle.keep_quarters(oracle.per_strip(oracle.S_BLOCK), q)
    bits, info = oracle.mask(v, pat)
    per = blocks_of(bits)
    nbc = K // 64
    assert info["exact"] and np.all(per.sum(axis=1) == nbc * q // 4)
    score = np.array([[sum(Fraction(x) ** 2 for x in v[32 * a:32 * a + 32, 64 * b:64 * b + 64].ravel())
                       for b in range(nbc)] for a in range(M // 32)], dtype=object)   # exact rational scores
    for a in range(M // 32):
        order = sorted(range(nbc), key=lambda b: (-score[a, b], b))
        assert sorted(order[:nbc * q // 4]) == list(np.nonzero(per[a])[0])
    # one strip alone: the same blocks as the tensor-wide definition on that strip
    for a in range(M // 32):
        alone = np.unpackbits(oracle.mask(v[32 * a:32 * a + 32], oracle.keep_quarters(oracle.S_BLOCK, q))[0], axis=1,
                              bitorder="little").astype(bool).reshape(32, nbc, 64).all(axis=(0, 2))
        assert np.array_equal(alone, per[a])
    # the tensor-wide selection is a different set here: it keeps every block of the loud strip first
    glob = blocks_of(oracle.mask(v, oracle.keep_quarters(oracle.S_BLOCK, q))[0])
    assert glob.sum() == (M // 32) * nbc * q // 4 and glob[3].all() and not per[3].all()
    # nesting with q, and the flag belongs to the block pattern only
    if q > 1:
        smaller = blocks_of(oracle.mask(v, oracle.keep_quarters(oracle.per_strip(oracle.S_BLOCK), q - 1))[0])
        assert np.all(smaller <= per)
    for other in (oracle.S_2_4, oracle.S_ROW50, oracle.S_CHAN50, oracle.S_DENSE):
        with pytest.raises(ValueError):
            oracle.mask(v, oracle.per_strip(other))


def test_mxfp8_e4m3_activations_for_w4a8():
    """8-bit activations of the W4A8 ablation (this project's reading: MXFP8, E4M3 elements): the value table and
    the element rounding against torch's float8_e4m3fn, the scale property 256 <= amax / 2^e < 512, saturation,
    round trip of representable blocks, and the exact rational product on a tiny case."""
    import torch
    codes = np.arange(256, dtype=np.uint8)
    tv = torch.from_numpy(codes.copy()).view(torch.float8_e4m3fn).to(torch.float32).numpy()
    ov = np.array([oracle.e4m3_value(int(c)) for c in codes])
    assert np.array_equal(np.isnan(tv), np.isnan(ov)) and np.array_equal(tv[~np.isnan(tv)], ov[~np.isnan(ov)])
    rng = np.random.default_rng(31)
    x = bf16_round((rng.standard_normal((16, 128)) * np.exp2(rng.integers(-20, 20, (16, 1)))).astype(np.float32))
    x[3, :32] = 0.0
    x[4, 5] *= 300.0                                                     # an outlier: the rest of its block goes subnormal
    c, sc, deq = oracle.mxfp8_e4m3_quantize(x)
    e = sc.astype(np.int64) - 127
    amax = np.abs(x.reshape(16, 4, 32)).max(axis=2).astype(np.float64)
    nz = amax > 0
    r = amax[nz] / np.exp2(e[nz].astype(np.float64))
    assert np.all((r >= 256) & (r < 512)) and np.all(sc[~nz] == 0)
    t = (x.reshape(16, 4, 32).astype(np.float64) / np.exp2(e.astype(np.float64))[:, :, None]).astype(np.float32)
    tt = torch.from_numpy(t).clamp(-448, 448).to(torch.float8_e4m3fn).view(torch.uint8).numpy().reshape(16, 128)
    same = (tt & 0x7F) == (c & 0x7F)                                     # (torch keeps the sign of a rounded-to-zero value too)
    assert np.all(same) and np.array_equal(tt >> 7, c >> 7)
    dec = np.array([oracle.e4m3_value(int(v)) for v in c.reshape(-1)]).reshape(16, 4, 32) * np.exp2(e.astype(np.float64))[:, :, None]
    assert np.array_equal(dec.reshape(16, 128), deq)
    assert np.all(np.abs(deq) <= 448 * np.exp2(e.astype(np.float64)).repeat(32, axis=1))
    assert np.all(np.abs(deq - x) <= np.maximum(2.0 ** -4 * np.abs(x), 2.0 ** -10 * np.exp2(e.astype(np.float64)).repeat(32, axis=1)) + 64 * np.exp2(e.astype(np.float64)).repeat(32, axis=1) * (np.abs(x) > 448 * np.exp2(e.astype(np.float64)).repeat(32, axis=1)))
    c2, sc2, deq2 = oracle.mxfp8_e4m3_quantize(deq.astype(np.float32))  # representable blocks come back unchanged
    assert np.array_equal(deq2, deq)
    M, K, N = 3, 64, 4
    xs = bf16_round(rng.standard_normal((M, K)).astype(np.float32))
    w = bf16_round(rng.standard_normal((N, K)).astype(np.float32) * 0.02)
    o = oracle.w4a8_linear(xs, w, "hif4")
    av, wv = _to_frac(o["a"]), _to_frac(o["w"])
    for m in range(M):
        for n in range(N):
            assert F(float(o["y"][m, n])) == sum(av[m][k] * wv[n][k] for k in range(K))
    # 8-bit activations sit between the 4-bit and the unquantized ones
    exact = oracle.w4a16_linear(xs, w, "hif4")["y"]
    four = oracle.resq_linear(xs, w, oracle.S_NONE, "hif4")["y"]
    assert np.linalg.norm(o["y"] - exact) < np.linalg.norm(four - exact)


# ----------------------------------------------------------------- regression digest of a seeded tensor

def test_seeded_digest():
    """Statistics of a seeded tensor, first derived with an independent throw-away script under the
    same reading and reproduced by this oracle; a change in any rule moves at least one of them."""
    rng = np.random.default_rng(0)
    X = rng.standard_normal((16, 2048)).astype(np.float32)
    ch = rng.choice(2048, 8, replace=False)
    assert sorted(int(c) for c in ch) == [79, 179, 520, 868, 1194, 1550, 1752, 1982]
    X[:, ch] *= 64
    X = bf16_round(X)
    o = oracle.quantize_residual_mask(X, oracle.S_2_4)

    def stats(codes, meta):
        q = nibbles(codes)
        return (int(((q & 7) == 0).sum()), int((q & 7).sum()), int((meta & 255).sum()),
                sum(bin((int(m) >> 8) & 255).count("1") for m in meta.ravel()),
                sum(bin(int(m) >> 16).count("1") for m in meta.ravel()))

    assert stats(o["x_codes"], o["x_side"]) == (7496, 75391, 97397, 2429, 4637)
    assert stats(o["r_codes"], o["r_side"]) == (2452, 111754, 89308, 2555, 5588)
    assert int((nibbles(o["x_codes"]) >> 3).sum()) == 16425
    XX = X.astype(np.float64)
    rel = lambda e: float(np.linalg.norm(e) / np.linalg.norm(XX))
    assert abs(rel(XX - o["a"]) - 0.0881) < 5e-4
    assert abs(rel(XX - o["a"] - o["r"]) - 0.0076) < 5e-4
    assert abs(rel(XX - o["a"] - o["r_masked"]) - 0.0346) < 5e-4


# ----------------------------------------------------------------- training-side GEMMs (backward pass of Eq. (1))

@pytest.mark.parametrize("fmt", ["hif4", "mxfp4"])
def test_backward_products_exact_rational_tiny_and_fixed_points(fmt):
    M, K, N = 64, 128, 64          # every contraction axis (n for dX, m for dW) holds whole blocks
    rng = np.random.default_rng(91)
    dy = bf16_round((rng.standard_normal((M, N)) * 1e-3).astype(np.float32))
    dy[:, 5] *= 40.0                # an outlier column of the output gradient
    w = bf16_round((rng.standard_normal((N, K)) * 0.02).astype(np.float32))
    x = gaussian_with_outliers(92, M, K, n_out=2, scale=16.0)
    # dX^ = Q(dY) Q(W^T)^T: the blocks of both operands run along n
    o = oracle.dgrad_linear(dy, w, fmt)
    assert o["y"].shape == (M, K)
    assert np.array_equal(o["g"], oracle.decode(fmt, *oracle.encode(fmt, dy)))
    assert np.array_equal(o["wt"], oracle.decode(fmt, *oracle.encode(fmt, np.ascontiguousarray(w.T))))
    g, wt = _to_frac(o["g"][:3]), _to_frac(o["wt"][:4])
    for m in range(3):
        for k in range(4):
            assert F(float(o["y"][m, k])) == sum(g[m][n] * wt[k][n] for n in range(N))
            assert F(float(o["abs_sum"][m, k])) == sum(abs(g[m][n] * wt[k][n]) for n in range(N))
    # dW^ = Q(dY^T) Q(X^T)^T: the blocks run along m
    o2 = oracle.wgrad_linear(dy, x, fmt)
    assert o2["y"].shape == (N, K)
    gt, xt = _to_frac(o2["gt"][:3]), _to_frac(o2["xt"][:4])
    for n in range(3):
        for k in range(4):
            assert F(float(o2["y"][n, k])) == sum(gt[n][m] * xt[k][m] for m in range(M))
    # quantizing along the contraction axis is not the same as quantizing along the other one: a loud token row of X
    # costs its own row nothing when the blocks run along d, but dominates the blocks of every channel along m
    x2 = x.copy()
    x2[7, :] *= 64.0
    along_d = oracle.decode(fmt, *oracle.encode(fmt, x2))
    along_m = oracle.decode(fmt, *oracle.encode(fmt, np.ascontiguousarray(x2.T))).T
    quiet = np.arange(M) != 7
    assert np.abs(along_m - x2)[quiet].max() > 4 * np.abs(along_d - x2)[quiet].max()
    # fixed points: operands that already are decoded codes (along the right axis) give the exact products
    if fmt == "hif4":
        dyq = representable_hif4_blocks(93, M * N // 64, 30 << 2, 40 << 2)[0].reshape(M, N).astype(np.float32)
        wtq = representable_hif4_blocks(94, K * N // 64, 40 << 2, 48 << 2)[0].reshape(K, N).astype(np.float32)
        o3 = oracle.dgrad_linear(dyq, np.ascontiguousarray(wtq.T))
        np.testing.assert_allclose(o3["y"], dyq.astype(np.float64) @ wtq.astype(np.float64).T, rtol=1e-13, atol=0)
        gtq = representable_hif4_blocks(95, N * M // 64, 30 << 2, 40 << 2)[0].reshape(N, M).astype(np.float32)
        xtq = representable_hif4_blocks(96, K * M // 64, 44 << 2, 52 << 2)[0].reshape(K, M).astype(np.float32)
        o4 = oracle.wgrad_linear(np.ascontiguousarray(gtq.T), np.ascontiguousarray(xtq.T))
        np.testing.assert_allclose(o4["y"], gtq.astype(np.float64) @ xtq.astype(np.float64).T, rtol=1e-13, atol=0)
