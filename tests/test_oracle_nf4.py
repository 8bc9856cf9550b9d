"""Pins for the oracle's NF4 quantiser / dequantiser (Section 5.1 of the paper).

None of these re-call the oracle's own formula: they use the closed-form
quantile construction, a pure-Python brute force, exact special cases and
torch's bf16 conversion.
"""
import math
import os

import numpy as np
import pytest
import torch
from hypothesis import given, settings, strategies as st
from scipy.stats import norm

from oracle import loqt_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "nf4_levels_qlora.txt")


def test_levels_match_published_table():
    vals = [float(l) for l in open(GOLDEN) if l.strip() and not l.startswith("#")]
    assert len(vals) == 16
    assert np.array_equal(np.array(vals, dtype=np.float32), O.NF4_LEVELS)
    # every published decimal is exactly an fp32 number
    assert all(float(np.float32(v)) == v for v in vals)


def test_levels_closed_form():
    """8 positive and 7 negative equal-probability normal quantiles (tail
    probability offset 0.9677083), an exact zero, all divided by the largest."""
    offset = 0.9677083
    pos = norm.ppf(np.linspace(offset, 0.5, 9)[:-1])
    neg = -norm.ppf(np.linspace(offset, 0.5, 8)[:-1])
    v = np.sort(np.concatenate([pos, [0.0], neg]))
    v = v / v.max()
    assert v.shape == (16,)
    assert np.max(np.abs(v - O.NF4_LEVELS.astype(np.float64))) < 2e-7
    lv = O.NF4_LEVELS
    assert lv[0] == -1.0 and lv[7] == 0.0 and lv[15] == 1.0
    assert np.all(np.diff(lv) > 0)
    assert (lv < 0).sum() == 7 and (lv > 0).sum() == 8


def _brute_quantize_block(vals):
    """Pure-Python statement of the displayed equations for one block."""
    m = np.float32(0)
    for v in vals:
        m = max(m, np.float32(abs(np.float32(v))))
    if m == 0:
        return [7] * len(vals), np.float32(0)
    out = []
    for v in vals:
        n = float(np.float32(v) / np.float32(m))
        best, bi = None, None
        for i in range(16):
            d = abs(n - float(O.NF4_LEVELS[i]))
            if best is None or d < best:
                best, bi = d, i
        out.append(bi)
    return out, m


@pytest.mark.parametrize("rows,cols", [(3, 64), (2, 192), (4, 100), (1, 1), (5, 32), (2, 129)])
def test_quantize_matches_brute_force(rows, cols):
    rng = np.random.default_rng(rows * 1000 + cols)
    w = (rng.standard_normal((rows, cols)) * 0.02).astype(np.float32)
    codes, absmax = O.nf4_quantize(w)
    ld = O.padded_cols(cols)
    assert codes.shape == (rows, ld) and absmax.shape == (rows, ld // 64)
    for r in range(rows):
        for b in range(ld // 64):
            c0, c1 = b * 64, min(b * 64 + 64, cols)
            bc, bm = _brute_quantize_block(list(w[r, c0:c1]))
            assert list(codes[r, c0:c1]) == bc
            assert absmax[r, b] == bm
            assert np.all(codes[r, c1 : b * 64 + 64] == 7)  # padding holds the zero level


def test_threshold_form_agrees():
    """argmin over levels == number of midpoints strictly below n (ties go low)."""
    rng = np.random.default_rng(7)
    w = rng.standard_normal((64, 256)).astype(np.float32)
    codes, absmax = O.nf4_quantize(w)
    lv = O.NF4_LEVELS.astype(np.float64)
    mid = (lv[:-1] + lv[1:]) / 2
    n = (w / np.repeat(absmax, 64, axis=1)).astype(np.float32).astype(np.float64)
    assert np.array_equal((n[:, :, None] > mid[None, None, :]).sum(axis=2), codes)


@pytest.mark.parametrize("scale", [1.0, 2.0 ** -7, 2.0 ** 5, 0.75])
def test_levels_round_trip_exactly(scale):
    """The 16 levels, scaled by M, code to 0..15 and decode to themselves."""
    blk = np.zeros((1, 64), dtype=np.float32)
    blk[0, :16] = O.NF4_LEVELS * np.float32(scale)
    codes, absmax = O.nf4_quantize(blk)
    assert absmax[0, 0] == np.float32(scale)
    assert list(codes[0, :16]) == list(range(16))
    assert np.all(codes[0, 16:] == 7)
    if math.log2(scale).is_integer():
        assert np.array_equal(O.nf4_dequantize(codes, absmax), blk)


def test_block_maximum_maps_to_unit():
    rng = np.random.default_rng(11)
    w = (rng.standard_normal((32, 512)) * 0.02).astype(np.float32)
    codes, absmax = O.nf4_quantize(w)
    blocks = w.reshape(32, 8, 64)
    cb = codes.reshape(32, 8, 64)
    am = np.argmax(np.abs(blocks), axis=2)
    for r in range(32):
        for b in range(8):
            v = blocks[r, b, am[r, b]]
            assert abs(v) == absmax[r, b]
            assert np.float32(v) / absmax[r, b] in (np.float32(1), np.float32(-1))
            assert cb[r, b, am[r, b]] == (15 if v > 0 else 0)
            assert ((cb[r, b] == 0) | (cb[r, b] == 15)).any()


def test_zero_block_and_signed_zero():
    w = np.zeros((2, 128), dtype=np.float32)
    w[0, 3] = -0.0
    w[1, 70] = 1e-30
    codes, absmax = O.nf4_quantize(w)
    assert np.all(codes[0] == 7) and np.all(absmax[0] == 0)
    assert np.all(codes[1, :64] == 7) and absmax[1, 0] == 0
    assert codes[1, 70] == 15 and absmax[1, 1] == np.float32(1e-30)
    assert np.array_equal(O.nf4_dequantize(codes, absmax)[0], np.zeros(128, np.float32))


def test_idempotent():
    """quantize(dequantize32(c, M)) returns (c, M) bit for bit."""
    rng = np.random.default_rng(5)
    w = (rng.standard_normal((16, 320)) * 0.02).astype(np.float32)
    c1, m1 = O.nf4_quantize(w)
    c2, m2 = O.nf4_quantize(O.nf4_dequantize(c1, m1))
    assert np.array_equal(c1, c2) and np.array_equal(m1, m2)


def test_dequantize_definition():
    rng = np.random.default_rng(9)
    codes = rng.integers(0, 16, size=(7, 128)).astype(np.uint8)
    absmax = rng.random((7, 2)).astype(np.float32)
    got = O.nf4_dequantize(codes, absmax)
    for r in range(7):
        for c in range(128):
            assert got[r, c] == np.float32(absmax[r, c // 64]) * np.float32(O.NF4_LEVELS[codes[r, c]])
    assert np.array_equal(O.nf4_dequantize(codes, absmax, cols=100), got[:, :100])


def test_quantisation_error_bound():
    """|w - deq(q(w))| <= M * (half the widest level gap)."""
    rng = np.random.default_rng(13)
    w = rng.standard_normal((8, 256)).astype(np.float32)
    codes, absmax = O.nf4_quantize(w)
    half_gap = float(np.max(np.diff(O.NF4_LEVELS.astype(np.float64)))) / 2
    err = np.abs(w.astype(np.float64) - O.nf4_dequantize(codes, absmax).astype(np.float64))
    bound = np.repeat(absmax.astype(np.float64), 64, axis=1) * half_gap * (1 + 1e-6)
    assert np.all(err <= bound)


def test_pack_layout():
    codes = np.tile(np.arange(16, dtype=np.uint8), 4).reshape(1, 64)
    packed = O.pack_codes(codes)
    assert packed.shape == (1, 32)
    assert packed[0, 0] == (0 | (1 << 4)) and packed[0, 7] == (14 | (15 << 4))
    assert np.array_equal(O.unpack_codes(packed), codes)


def test_bf16_round_matches_torch():
    rng = np.random.default_rng(3)
    a = np.concatenate(
        [
            (rng.standard_normal(20000) * 10.0 ** rng.integers(-20, 20, 20000)).astype(np.float32),
            np.array([0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895314e38, 1e-40], dtype=np.float32),
        ]
    )
    want = torch.from_numpy(a).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(O.bf16_round(a).view(np.uint32), want.view(np.uint32))


@settings(max_examples=200, deadline=None)
@given(
    st.lists(
        st.floats(width=32, allow_nan=False, allow_infinity=False, allow_subnormal=True),
        min_size=1,
        max_size=64,
    )
)
def test_quantize_hypothesis_blocks(vals):
    w = np.array([vals], dtype=np.float32)
    codes, absmax = O.nf4_quantize(w)
    bc, bm = _brute_quantize_block(vals)
    assert list(codes[0, : len(vals)]) == bc
    assert absmax[0, 0] == bm
