"""Pins for the oracle's double quantisation of the block scales (Section 2.4:
the quantisation state is re-quantised, following QLoRA).  The paper prints no
numbers for it, so the pins are: the FP8 E4M3 codec against torch's own
float8_e4m3fn conversion (an independent library routine) and against the
format's published constants, the round-trip error bound that the format's
3-bit mantissa implies, exactness on representable inputs, and the storage
count the reading implies."""
import numpy as np
import pytest
import torch

from oracle import loqt_oracle as O


def test_e4m3_decode_matches_torch_and_the_published_constants():
    codes = np.arange(256, dtype=np.uint8)
    mine = O.e4m3_decode(codes)
    ref = torch.from_numpy(codes.copy()).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    assert np.array_equal(np.isnan(mine), np.isnan(ref))
    ok = ~np.isnan(ref)
    assert np.array_equal(mine[ok], ref[ok])
    assert np.nanmax(mine) == 448.0 and np.nanmin(mine) == -448.0          # largest finite value
    assert mine[0x01] == 2.0 ** -9 and mine[0x08] == 2.0 ** -6             # smallest subnormal, smallest normal
    assert mine[0x38] == 1.0 and mine[0x3C] == 1.5
    assert int(np.isnan(mine).sum()) == 2                                   # S.1111.111 only; no infinities


def test_e4m3_encode_is_round_to_nearest_even_like_torch():
    rng = np.random.default_rng(0)
    x = np.concatenate([
        rng.uniform(-448, 448, 20000), rng.normal(0, 1, 20000), rng.normal(0, 0.01, 20000),
        O.e4m3_decode(np.array([c for c in range(256) if (c & 0x7F) != 0x7F])),                 # representable
        np.array([17.0, 19.0, 21.0, 23.0, 2.0 ** -10, 3 * 2.0 ** -10, 0.0, 448.0, -448.0, 447.9, 1e-9]),  # ties and edges
    ]).astype(np.float32)
    mine = O.e4m3_decode(O.e4m3_encode(x))
    ref = torch.from_numpy(x.copy()).to(torch.float8_e4m3fn).to(torch.float64).numpy()
    assert np.array_equal(mine, ref)
    # brute force on a sample: the chosen value is a nearest finite value
    vals = O.e4m3_decode(np.array([c for c in range(256) if (c & 0x7F) != 0x7F]))
    for xi, mi in zip(x[:500], mine[:500]):
        assert abs(mi - xi) == np.min(np.abs(vals - float(xi)))


def _scales(seed, n, sigma=0.02):
    rng = np.random.default_rng(seed)
    w = rng.normal(0, sigma, (n, 64)).astype(np.float32)
    return np.max(np.abs(w), axis=1).astype(np.float32)


@pytest.mark.parametrize("n", [256, 1000, 4096 + 77, 5])
def test_round_trip_error_is_within_the_format_bound(n):
    c2 = _scales(1, n)
    codes, c1, off = O.dq_quantize_absmax(c2)
    assert codes.shape == (n,) and c1.shape == ((n + 255) // 256,)
    assert abs(float(off) - float(np.mean(c2.astype(np.float64)))) <= np.spacing(np.float32(off))
    back = O.dq_dequantize_absmax(codes, c1, off)
    d = (c2 - off).astype(np.float64)
    err = np.abs(back.astype(np.float64) - c2.astype(np.float64))
    scale = np.repeat(c1.astype(np.float64), 256)[:n] * 448.0      # the block's largest centred scale
    # E4M3 keeps 3 mantissa bits: relative half-spacing 2^-4 for normal values, absolute half-spacing
    # 2^-10 below 2^-6 (in units where the block maximum is 448); plus fp32 roundings of the arithmetic
    bound = np.maximum(np.abs(d) * 2.0 ** -4, scale * 2.0 ** -10 / 448.0) + 8 * np.spacing(c2).astype(np.float64)
    assert np.all(err <= bound)
    # each block's largest centred scale is hit exactly up to fp32 rounding (code +-448)
    for b in range(len(c1)):
        blk = slice(b * 256, min((b + 1) * 256, n))
        k = np.argmax(np.abs(d[blk]))
        assert (codes[blk][k] & 0x7F) == 0x7E
        assert err[blk][k] <= 4 * np.spacing(c2[blk][k])
    # a typical weight matrix (scales spread about +-30 % around their mean): they come back within 5 %
    assert np.max(err / c2) < 0.05


def test_representable_scales_round_trip_exactly():
    # scales of the form offset + c1 * (E4M3 value / 448) with power-of-two c1 and offset 0 come back bit for bit
    vals = O.e4m3_decode(np.array([c for c in range(128) if c != 0x7F])).astype(np.float32)
    c2 = np.concatenate([vals, -vals]).astype(np.float32)            # mean exactly 0, max 448
    assert c2.size == 254
    codes, c1, off = O.dq_quantize_absmax(c2)
    assert off == 0.0 and c1[0] == 1.0                             # one E4M3 unit stands for 1.0
    assert np.array_equal(O.dq_dequantize_absmax(codes, c1, off), c2)
    # all-equal scales: everything sits in the offset, codes are +0
    c2 = np.full(300, 0.0371, dtype=np.float32)
    codes, c1, off = O.dq_quantize_absmax(c2)
    assert np.all(codes == 0) and np.all(c1 == 0) and off == np.float32(0.0371)
    assert np.array_equal(O.dq_dequantize_absmax(codes, c1, off), c2)


def test_given_offset_is_used_and_storage_count():
    c2 = _scales(3, 700)
    codes_a, c1_a, off_a = O.dq_quantize_absmax(c2)
    nudged = np.nextafter(off_a, np.float32(1.0))
    codes_b, c1_b, off_b = O.dq_quantize_absmax(c2, offset=nudged)
    assert off_b == nudged and np.mean(codes_a != codes_b) < 0.2
    assert abs(O.dq_bits_per_weight() - 4.127) < 5e-4                  # QLoRA's figure for this scheme
    assert O.dq_bits_per_weight() == 4 + 8 / 64 + 32 / (64 * 256)


def test_layer_with_doubly_quantised_scales_stays_close():
    # the forward through scales that went through double quantisation differs from the plain NF4 layer by
    # at most the scale error times the weight magnitude
    from paper_2405_16528_b200 import synth

    d = synth.make_layer(5, "dq", 128, 256, 16, 1e-2, 8)
    codes, absmax = O.nf4_quantize(d["W"].numpy())
    c8, c1, off = O.dq_quantize_absmax(absmax)
    absmax2 = O.dq_dequantize_absmax(c8, c1, off, absmax.shape)
    w1 = O.nf4_dequantize(codes, absmax, 256).astype(np.float64)
    w2 = O.nf4_dequantize(codes, absmax2, 256).astype(np.float64)
    assert np.max(np.abs(w1 - w2)) <= 0.02 * np.max(np.abs(w1))
    assert np.linalg.norm(w1 - w2) <= 0.01 * np.linalg.norm(w1)
