"""GPU parity: loqt_nf4_quantize / loqt_nf4_dequantize against the CPU oracle,
bit for bit, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import loqt_oracle as O
from paper_2405_16528_b200 import binding as L
from paper_2405_16528_b200 import synth
from tests.gpu_util import from_dev_nf4, to_dev_nf4

pytestmark = pytest.mark.gpu

SHAPES = [(256, 256), (1, 1), (3, 64), (37, 100), (130, 1376), (64, 5461), (700, 512)]


@pytest.mark.parametrize("rows,cols", SHAPES)
def test_quantize_bit_exact(rows, cols):
    w = synth.normal(0, ("q", rows, cols), (rows, cols), 0.02)
    ref_c, ref_m = O.nf4_quantize(w.numpy())
    q = L.loqt_nf4_quantize(w.cuda())
    got_c, got_m = from_dev_nf4(q)
    assert np.array_equal(got_m.view(np.uint32), ref_m.view(np.uint32))
    assert np.array_equal(got_c, ref_c)


def test_quantize_strided_and_unaligned_source():
    big = synth.normal(1, "strided", (50, 333), 1.0).cuda()
    for c0, cols in [(0, 200), (1, 130), (3, 64)]:
        view = big[:, c0 : c0 + cols]
        ref_c, ref_m = O.nf4_quantize(view.cpu().numpy().copy())
        got_c, got_m = from_dev_nf4(L.loqt_nf4_quantize(view))
        assert np.array_equal(got_c, ref_c) and np.array_equal(got_m, ref_m)


def test_quantize_decision_boundaries_and_special_values():
    """Values sitting exactly on, just below and just above every level midpoint,
    plus zeros, signed zero, denormals and huge magnitudes."""
    lv = O.NF4_LEVELS.astype(np.float64)
    mid = ((lv[:-1] + lv[1:]) / 2).astype(np.float32)
    pts = []
    for m in mid:
        pts += [m, np.nextafter(m, np.float32(-2)), np.nextafter(m, np.float32(2))]
    pts += list(O.NF4_LEVELS)
    rows = []
    # 0x1.fffffep-5 has an all-ones significand; 2.5e30 and 1e-38 lie outside the
    # range of the reciprocal-based division: all three take the IEEE-divide path
    for scale in (1.0, 0.03125, 3.0, 0.75, 1.7e-3, 0.0523, float(np.nextafter(np.float32(0.0625), np.float32(0))), 2.5e30, 1e-38, 7e17, 3e-18):
        blk = np.zeros(64, dtype=np.float32)
        blk[: len(pts)] = np.array(pts, dtype=np.float32) * np.float32(scale)
        blk[63] = np.float32(scale)  # pins the block scale
        rows.append(blk)
    rows.append(np.zeros(64, dtype=np.float32))
    z = np.zeros(64, dtype=np.float32)
    z[5] = -0.0
    z[9] = 1e-45
    rows.append(z)
    w = np.stack(rows)
    ref_c, ref_m = O.nf4_quantize(w)
    got_c, got_m = from_dev_nf4(L.loqt_nf4_quantize(torch.from_numpy(w).cuda()))
    assert np.array_equal(got_m.view(np.uint32), ref_m.view(np.uint32))
    assert np.array_equal(got_c, ref_c)


def test_quantize_many_random_blocks_bit_exact():
    g = torch.Generator().manual_seed(5)
    w = torch.randn((2048, 1024), generator=g) * torch.exp(torch.randn((2048, 1), generator=g) * 3)
    ref_c, ref_m = O.nf4_quantize(w.numpy())
    got_c, got_m = from_dev_nf4(L.loqt_nf4_quantize(w.cuda()))
    assert np.array_equal(got_m, ref_m) and np.array_equal(got_c, ref_c)


@pytest.mark.parametrize("rows,cols", SHAPES)
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_dequantize_bit_exact(rows, cols, dtype):
    rng = np.random.default_rng(rows + cols)
    ld = O.padded_cols(cols)
    codes = rng.integers(0, 16, size=(rows, ld)).astype(np.uint8)
    codes[:, cols:] = 7
    absmax = (rng.random((rows, ld // 64)) * 0.1).astype(np.float32)
    q = to_dev_nf4(codes, absmax, cols)
    got = L.loqt_nf4_dequantize(q, dtype)
    if dtype == torch.float32:
        ref = O.nf4_dequantize(codes, absmax, cols)
        assert np.array_equal(got.cpu().numpy().view(np.uint32), ref.view(np.uint32))
    else:
        ref = O.nf4_dequantize_bf16(codes, absmax, cols)
        assert np.array_equal(got.to(torch.float32).cpu().numpy().view(np.uint32), ref.view(np.uint32))


def test_dequantize_into_strided_destination():
    rng = np.random.default_rng(2)
    codes = rng.integers(0, 16, size=(9, 128)).astype(np.uint8)
    absmax = rng.random((9, 2)).astype(np.float32)
    q = to_dev_nf4(codes, absmax, 128)
    buf = torch.full((9, 203), -1.0, device="cuda")
    L.loqt_nf4_dequantize(q, dst=buf[:, 3:131])
    assert np.array_equal(buf[:, 3:131].cpu().numpy(), O.nf4_dequantize(codes, absmax))
    assert torch.all(buf[:, :3] == -1) and torch.all(buf[:, 131:] == -1)


def test_round_trip_is_idempotent_on_device():
    w = synth.normal(3, "idem", (64, 320), 0.02).cuda()
    q1 = L.loqt_nf4_quantize(w)
    q2 = L.loqt_nf4_quantize(L.loqt_nf4_dequantize(q1))
    assert torch.equal(q1.codes, q2.codes) and torch.equal(q1.absmax, q2.absmax)


def test_argument_errors_are_reported():
    w = torch.zeros((4, 64), device="cuda")
    q = L.NF4Tensor.empty(4, 64)
    bad = q.view()
    bad.block = 32
    assert L.lib().loqt_nf4_quantize(w.data_ptr(), 64, bad, None) == 3
    assert L.lib().loqt_nf4_quantize(None, 64, q.view(), None) == 1
    assert L.lib().loqt_nf4_quantize(w.data_ptr(), 8, q.view(), None) == 1
    bad = q.view()
    bad.ld = 96
    assert L.lib().loqt_nf4_quantize(w.data_ptr(), 64, bad, None) in (1, 2)
