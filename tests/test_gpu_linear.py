"""GPU parity: loqt_linear_fwd / loqt_linear_bwd / loqt_merge_requant against
the CPU oracle on the same seeded inputs, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import loqt_oracle as O
from paper_2405_16528_b200 import binding as L
from paper_2405_16528_b200 import synth
from tests.gpu_util import check_close, check_merge, f32, from_dev_nf4, merge_error_bound, padded, to_dev_nf4

pytestmark = pytest.mark.gpu

# (out, in, r, T): config 0 of the benchmark, then shapes that span several
# tiles with ragged edges in every dimension (1376 and 5461 are the paper's MLP
# widths; r = 32 is below one K stage).
SHAPES = [
    (256, 256, 32, 512),
    (384, 320, 64, 200),
    (512, 1376, 128, 300),
    (1376, 512, 128, 257),
    (200, 136, 24, 130),
    (640, 5461, 96, 140),
    (5461, 256, 40, 133),
]


def _setup(seed, out, inn, r, T, sigma_B=1e-2):
    d = synth.make_layer(seed, "g", out, inn, r, sigma_B, T)
    wq = O.nf4_quantize(d["W"].numpy())
    pq = O.nf4_quantize(d["P"].numpy())
    dev = {
        "Wq": to_dev_nf4(*wq, inn),
        "Pq": to_dev_nf4(*pq, r),
        "B": padded(d["B"]),
        "x": padded(d["x"]),
        "dy": padded(d["dy"]),
    }
    host = {"wq": wq, "pq": pq, "B": f32(d["B"]), "x": f32(d["x"]), "dy": f32(d["dy"])}
    return host, dev


@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("s", [1.0, 0.5])
def test_forward(shape, s):
    out, inn, r, T = shape
    h, d = _setup(10, out, inn, r, T)
    ref = O.loqt_forward(h["wq"], h["pq"], h["B"], s, h["x"], (out, inn, r))
    y = padded(torch.zeros((T, out), dtype=torch.bfloat16))
    ws = L.new_workspace(L.loqt_workspace_bytes(L.LOQT_OP_FWD, out, inn, r, T))
    L.loqt_linear_fwd(d["Wq"], d["Pq"], d["B"], s, d["x"], y=y, ws=ws)
    L.loqt_device_status(ws)
    check_close(f32(y), ref, f"y {shape}")


@pytest.mark.parametrize("shape", SHAPES)
def test_backward(shape):
    out, inn, r, T = shape
    s = 0.5
    h, d = _setup(11, out, inn, r, T)
    ref_dx, ref_dB = O.loqt_backward(h["wq"], h["pq"], h["B"], s, h["x"], h["dy"], (out, inn, r))
    dx = padded(torch.zeros((T, inn), dtype=torch.bfloat16))
    dB = torch.full((r, inn), 7.0, dtype=torch.float32, device="cuda")
    ws = L.new_workspace(L.loqt_workspace_bytes(L.LOQT_OP_BWD, out, inn, r, T))
    L.loqt_linear_bwd(d["Wq"], d["Pq"], d["B"], s, d["x"], d["dy"], dx=dx, dB=dB, ws=ws)
    L.loqt_device_status(ws)
    check_close(f32(dx), ref_dx, f"dx {shape}")
    check_close(f32(dB), ref_dB, f"dB {shape}")
    # gradient accumulation adds to what is there, and the result is reproducible
    first = dB.clone()
    L.loqt_linear_bwd(d["Wq"], d["Pq"], d["B"], s, d["x"], d["dy"], dx=dx, dB=dB, accumulate_dB=True, ws=ws)
    check_close(f32(dB), 2 * ref_dB, f"dB accumulated {shape}")
    dB2 = torch.empty_like(dB)
    L.loqt_linear_bwd(d["Wq"], d["Pq"], d["B"], s, d["x"], d["dy"], dx=None, dB=dB2, ws=ws, need_dx=False)
    assert torch.equal(dB2, first)


@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("sigma_B", [1e-3, 1e-2])
def test_merge(shape, sigma_B):
    out, inn, r, _ = shape
    s = 1.0
    h, d = _setup(12, out, inn, r, 8, sigma_B)
    vw = O.loqt_merge_values(h["wq"], h["pq"], h["B"], s, (out, inn, r))
    ref_c, ref_m = O.nf4_quantize(vw)
    L.loqt_merge_requant(d["Wq"], d["Pq"], d["B"], s)
    got_c, got_m = from_dev_nf4(d["Wq"])
    bound, _ = merge_error_bound(h["pq"], h["B"], s, r, ref_m)
    n_diff, max_ulp, hist = check_merge(got_c, got_m, ref_c, ref_m, vw, inn, bound, f"merge {shape}")
    print(f"merge {shape} sigma_B={sigma_B}: {n_diff} codes differ; scale differences in ulps {hist}")
    assert np.all(got_c[:, inn:] == 7)


@pytest.mark.parametrize("shape", SHAPES)
def test_merge_split_matches_fused(shape):
    # the two-pass merge takes the same accumulators through the same arithmetic
    out, inn, r, _ = shape
    h, d = _setup(16, out, inn, r, 8, 1e-2)
    fused = L.loqt_merge_requant(d["Wq"].clone(), d["Pq"], d["B"], 0.5)
    split = L.loqt_merge_requant_split(d["Wq"].clone(), d["Pq"], d["B"], 0.5)
    assert torch.equal(fused.codes, split.codes) and torch.equal(fused.absmax, split.absmax)


@pytest.mark.parametrize("shape", [(256, 256), (200, 136), (96, 5461), (1376, 512)])
@pytest.mark.parametrize("s", [1.0, 0.5])
def test_requantize_bit_exact(shape, s):
    # s is a power of two, so s * delta is exact and the oracle's single rounding of
    # the float64 sum equals the kernel's fused multiply-add.
    out, inn = shape
    h, d = _setup(17, out, inn, 8, 8)
    delta = synth.normal(17, ("delta", out, inn), (out, inn), 5e-3, torch.float32)
    delta[::7, ::5] = 0.0
    ref_c, ref_m = O.nf4_requantize(h["wq"], delta.numpy(), s, inn)
    ld = (inn + 3) // 4 * 4
    dev_delta = torch.zeros((out, ld), dtype=torch.float32, device="cuda")[:, :inn]
    dev_delta.copy_(delta)
    L.loqt_nf4_requantize(dev_delta, s, d["Wq"])
    got_c, got_m = from_dev_nf4(d["Wq"])
    assert np.array_equal(got_c, ref_c) and np.array_equal(got_m, ref_m)


@pytest.mark.parametrize("shape", SHAPES)
def test_full_gradient(shape):
    out, inn, r, T = shape
    h, d = _setup(18, out, inn, r, T)
    ref = O.full_gradient(h["x"], h["dy"])
    G = L.loqt_full_gradient(d["x"], d["dy"])
    check_close(f32(G), ref, f"G^W {shape}")
    first = G.clone()
    L.loqt_full_gradient(d["x"], d["dy"], G=G, accumulate=True)
    check_close(f32(G), 2 * ref, f"G^W accumulated {shape}")
    assert torch.equal(L.loqt_full_gradient(d["x"], d["dy"]), first)   # fixed reduction order


def test_merge_zero_B_leaves_weights_untouched():
    out, inn, r = 256, 320, 32
    h, d = _setup(13, out, inn, r, 8)
    before = d["Wq"].clone()
    L.loqt_merge_requant(d["Wq"], d["Pq"], torch.zeros_like(d["B"]), 1.0)
    assert torch.equal(before.codes, d["Wq"].codes) and torch.equal(before.absmax, d["Wq"].absmax)


def test_merge_zero_B_with_rows_of_very_different_scale():
    # Scales beyond 2^+-60 take the IEEE division in the requantising epilogue, the others the
    # division by reciprocal, all-zero blocks neither; with the three kinds in neighbouring
    # rows the lanes of one epilogue warp part ways inside a block.  A merge with B = 0 must
    # still hand back every code and scale as it found them.
    out, inn, r = 256, 320, 32
    h, d = _setup(14, out, inn, r, 8)
    Wq = d["Wq"]
    k = torch.tensor([0, 70, -70, 0, 65, -65, 0, 0], dtype=torch.float32, device="cuda")[torch.arange(out, device="cuda") % 8]
    Wq.absmax.mul_(torch.exp2(k)[:, None])
    zero = torch.arange(out, device="cuda") % 16 == 5
    Wq.absmax[zero] = 0.0
    Wq.codes[zero] = 0x77
    before = Wq.clone()
    L.loqt_merge_requant(Wq, d["Pq"], torch.zeros_like(d["B"]), 1.0)
    assert torch.equal(before.codes, Wq.codes) and torch.equal(before.absmax, Wq.absmax)


def test_merge_many_matches_single():
    # 18 matrices of mixed shapes (ragged and not, several ranks) through one call: the batched launch walks
    # the tiles of all of them as one sequence and must leave every matrix exactly as a merge of its own does;
    # a few are also compared with the oracle.  A small workspace forces the call to split into several batches.
    shapes = [(256, 256, 32), (384, 320, 64), (200, 136, 24), (512, 1376, 128), (1376, 512, 128), (640, 5461, 96),
              (130, 70, 8), (128, 256, 64), (1024, 1024, 256), (96, 4096, 48), (2736, 192, 40), (257, 257, 16),
              (64, 64, 64), (768, 1000, 72), (1000, 768, 200), (5461, 256, 40), (600, 2100, 512), (2048, 640, 320)]
    sets = [_setup(14 + i, o, n, r, 8) for i, (o, n, r) in enumerate(shapes)]
    devs = [d for _, d in sets]
    singles = [L.loqt_merge_requant(x["Wq"].clone(), x["Pq"], x["B"], 0.5) for x in devs]
    for group in (8, 1):
        trial = [x["Wq"].clone() for x in devs]
        ws = L.new_workspace(L.merge_many_workspace_bytes(trial, [x["Pq"] for x in devs], group=group))
        L.loqt_merge_requant_many(trial, [x["Pq"] for x in devs], [x["B"] for x in devs], 0.5, ws=ws)
        L.loqt_device_status(ws)
        for one, got in zip(singles, trial):
            assert torch.equal(one.codes, got.codes) and torch.equal(one.absmax, got.absmax)
    for i in (0, 5, 11, 16):
        (h, d), (o, n, r) = sets[i], shapes[i]
        vw = O.loqt_merge_values(h["wq"], h["pq"], h["B"], 0.5, (o, n, r))
        ref_c, ref_m = O.nf4_quantize(vw)
        got_c, got_m = from_dev_nf4(singles[i])
        bound, _ = merge_error_bound(h["pq"], h["B"], 0.5, r, ref_m)
        check_merge(got_c, got_m, ref_c, ref_m, vw, n, bound, f"merge-many {shapes[i]}")


def test_forward_special_cases_on_device():
    out, inn, r, T = 256, 256, 32, 128
    h, d = _setup(15, out, inn, r, T)
    # B = 0: plain quantised linear
    y0 = L.loqt_linear_fwd(d["Wq"], d["Pq"], torch.zeros_like(d["B"]), 1.0, d["x"])
    W = O.nf4_dequantize_bf16(*h["wq"]).astype(np.float64)
    check_close(f32(y0), h["x"].astype(np.float64) @ W.T, "B=0")


def test_argument_errors():
    out, inn, r, T = 256, 256, 32, 128
    h, d = _setup(16, out, inn, r, T)
    y = torch.empty((T, out), dtype=torch.bfloat16, device="cuda")
    small = L.new_workspace(256)
    with pytest.raises(L.LoqtError, match="workspace"):
        L.loqt_linear_fwd(d["Wq"], d["Pq"], d["B"], 1.0, d["x"], y=y, ws=small)
    with pytest.raises(L.LoqtError, match="misaligned"):
        L.loqt_linear_fwd(d["Wq"], d["Pq"], d["B"], 1.0, d["x"][:, 1:], y=y)
