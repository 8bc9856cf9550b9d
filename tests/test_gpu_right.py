"""GPU parity of the right-side variant (W = deq(W_q) + s B deq(Q_q), Section 2.1:
G Q for m > n) against the CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import loqt_oracle as O
from paper_2405_16528_b200 import binding as L
from paper_2405_16528_b200 import synth
from tests.gpu_util import check_close, check_merge, f32, from_dev_nf4, padded, to_dev_nf4

pytestmark = pytest.mark.gpu

# (out, in, r, T): tall matrices (the case the variant is for) with ragged edges, one wide
SHAPES = [(512, 256, 32, 300), (1376, 512, 128, 257), (384, 320, 64, 200), (5461, 256, 40, 133), (200, 136, 24, 512)]


def _setup(seed, out, inn, r, T, sigma_B=1e-2):
    W = synth.normal(seed, ("W", out, inn), (out, inn), 0.02)
    Q = synth.orthonormal(seed, ("Q", inn, r), inn, r).T.contiguous()          # r x in, orthonormal rows
    B = synth.normal(seed, ("B", out, r), (out, r), sigma_B, torch.bfloat16)
    x = synth.normal(seed, ("x", T, inn), (T, inn), 1.0, torch.bfloat16)
    dy = synth.normal(seed, ("dy", T, out), (T, out), 1.0, torch.bfloat16)
    wq, qq = O.nf4_quantize(W.numpy()), O.nf4_quantize(Q.numpy())
    dev = {"Wq": to_dev_nf4(*wq, inn), "Qq": to_dev_nf4(*qq, inn), "B": padded(B), "x": padded(x), "dy": padded(dy)}
    host = {"wq": wq, "qq": qq, "B": f32(B), "x": f32(x), "dy": f32(dy)}
    return host, dev


@pytest.mark.parametrize("shape", SHAPES)
def test_forward_and_backward(shape):
    out, inn, r, T = shape
    s = 0.5
    h, d = _setup(80, out, inn, r, T)
    ref_y = O.loqt_forward_right(h["wq"], h["qq"], h["B"], s, h["x"], (out, inn, r))
    ref_dx, ref_dB = O.loqt_backward_right(h["wq"], h["qq"], h["B"], s, h["x"], h["dy"], (out, inn, r))
    y = L.loqt_linear_fwd_right(d["Wq"], d["Qq"], d["B"], s, d["x"])
    check_close(f32(y), ref_y, f"y {shape}")
    dx, dB = L.loqt_linear_bwd_right(d["Wq"], d["Qq"], d["B"], s, d["x"], d["dy"])
    check_close(f32(dx), ref_dx, f"dx {shape}")
    check_close(f32(dB), ref_dB, f"dB {shape}")
    first = dB.clone()
    L.loqt_linear_bwd_right(d["Wq"], d["Qq"], d["B"], s, d["x"], d["dy"], dB=dB, accumulate_dB=True)
    check_close(f32(dB), 2 * ref_dB, f"dB accumulated {shape}")
    _, again = L.loqt_linear_bwd_right(d["Wq"], d["Qq"], d["B"], s, d["x"], d["dy"])
    assert torch.equal(again, first)


@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("sigma_B", [1e-3, 1e-2])
def test_merge(shape, sigma_B):
    out, inn, r, _ = shape
    s = 1.0
    h, d = _setup(81, out, inn, r, 8, sigma_B)
    vw = O.loqt_merge_values_right(h["wq"], h["qq"], h["B"], s, (out, inn, r))
    ref_c, ref_m = O.nf4_quantize(vw)
    L.loqt_merge_requant_right(d["Wq"], d["Qq"], d["B"], s)
    got_c, got_m = from_dev_nf4(d["Wq"])
    # error bound of the fp32 tensor-core sum, per element: the left variant's formula with
    # the roles of the factors exchanged (|B| |Q-hat| summed over r)
    Qh = np.abs(O.nf4_dequantize_bf16(*h["qq"], inn)).astype(np.float64)
    mag = np.abs(h["B"]).astype(np.float64) @ Qh
    ulp = np.spacing(np.abs(ref_m).astype(np.float32)).astype(np.float64)
    bound = (np.ceil(r / 16) + 1) * 2.0 ** -23 * abs(s) * mag + np.repeat(ulp, 64, axis=1)[:, :inn]
    n_diff, max_ulp, hist = check_merge(got_c, got_m, ref_c, ref_m, vw, inn, bound, f"merge {shape}")
    assert np.all(got_c[:, inn:] == 7)


def test_merge_zero_B_leaves_weights_untouched():
    out, inn, r = 384, 320, 32
    h, d = _setup(82, out, inn, r, 8)
    before = d["Wq"].clone()
    L.loqt_merge_requant_right(d["Wq"], d["Qq"], torch.zeros_like(d["B"]), 1.0)
    assert torch.equal(before.codes, d["Wq"].codes) and torch.equal(before.absmax, d["Wq"].absmax)
