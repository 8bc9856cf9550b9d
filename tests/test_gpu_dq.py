"""GPU parity of the doubly quantised block scales (Section 2.4, the re-quantised
quantisation state) against the CPU oracle, through the C ABI: the scale codec
bit for bit, the dequantiser reading the 8-bit scales bit for bit, and the
forward / backward whose operand staging decodes them inside the kernels."""
import numpy as np
import pytest
import torch

from oracle import loqt_oracle as O
from paper_2405_16528_b200 import binding as L
from paper_2405_16528_b200 import synth
from tests.gpu_util import check_close, f32, padded, to_dev_nf4

pytestmark = pytest.mark.gpu


def _to_dev_dq(codes8, c1, off) -> L.DQScales:
    return L.DQScales(torch.from_numpy(codes8.copy()).cuda(), torch.from_numpy(c1.copy()).cuda(),
                      torch.tensor([float(off)], dtype=torch.float32, device="cuda"))


@pytest.mark.parametrize("shape", [(256, 256), (200, 136), (96, 5461), (1376, 512), (4096, 4096), (3, 64)])
def test_scale_codec_bit_exact(shape):
    rows, cols = shape
    W = synth.normal(60, ("dq", rows, cols), (rows, cols), 0.02)
    W[::5, : min(64, cols)] = 0.0                                    # some all-zero blocks: scale 0
    codes, absmax = O.nf4_quantize(W.numpy())
    dq = L.loqt_scales_double_quantize(torch.from_numpy(absmax).cuda())
    off_gpu = float(dq.offset.cpu()[0])
    ref_mean = np.float32(np.mean(absmax.astype(np.float64)))
    # the mean is summed in a different (fixed) order on the device: the same fp32 number or its neighbour
    assert abs(off_gpu - float(ref_mean)) <= float(np.spacing(ref_mean))
    # integer work from here on: with the device's offset the oracle must produce the same codes and scales
    r8, rc1, _ = O.dq_quantize_absmax(absmax, offset=np.float32(off_gpu))
    assert np.array_equal(dq.codes8.cpu().numpy(), r8)
    assert np.array_equal(dq.c1.cpu().numpy(), rc1)
    back = L.loqt_scales_double_dequantize(dq, absmax.shape).cpu().numpy()
    ref_back = O.dq_dequantize_absmax(r8, rc1, np.float32(off_gpu), absmax.shape)
    assert np.array_equal(back, ref_back)
    # the dequantiser that reads the 8-bit scales: equal to the oracle's dequantiser on the decoded scales
    Wq = to_dev_nf4(codes, absmax, cols)
    for dtype, ref in ((torch.float32, O.nf4_dequantize(codes, ref_back, cols)), (torch.bfloat16, O.nf4_dequantize_bf16(codes, ref_back, cols))):
        got = L.loqt_nf4_dequantize_dq(Wq, dq, dtype)
        assert np.array_equal(f32(got), ref)


def test_every_e4m3_code_decodes_like_the_oracle():
    # all 256 bit patterns as scale codes (NaN patterns excluded): c1 = 1, offset = 0 gives the E4M3 value itself
    codes8 = np.array([c for c in range(256) if (c & 0x7F) != 0x7F], dtype=np.uint8)
    dq = _to_dev_dq(codes8, np.ones(1, dtype=np.float32), 0.0)
    got = L.loqt_scales_double_dequantize(dq, (codes8.size,)).cpu().numpy()
    assert np.array_equal(got, O.e4m3_decode(codes8).astype(np.float32))


SHAPES = [(256, 256, 32, 512), (1376, 5461, 96, 300), (5461, 1376, 40, 389), (640, 2736, 512, 521)]


@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "x".join(map(str, s)))
def test_forward_backward_with_8bit_scales(shape):
    out, inn, r, T = shape
    s = 0.5
    d = synth.make_layer(61, ("dq",) + shape, out, inn, r, 1e-2, T)
    wq, pq = O.nf4_quantize(d["W"].numpy()), O.nf4_quantize(d["P"].numpy())
    w8, p8 = O.dq_quantize_absmax(wq[1]), O.dq_quantize_absmax(pq[1])
    # the layer the oracle sees: same codes, scales decoded from their 8-bit form
    wq2 = (wq[0], O.dq_dequantize_absmax(*w8, wq[1].shape))
    pq2 = (pq[0], O.dq_dequantize_absmax(*p8, pq[1].shape))
    Bh, xh, dyh = f32(d["B"]), f32(d["x"]), f32(d["dy"])
    ref_y = O.loqt_forward(wq2, pq2, Bh, s, xh, (out, inn, r))
    ref_dx, ref_dB = O.loqt_backward(wq2, pq2, Bh, s, xh, dyh, (out, inn, r))
    Wq, Pq = to_dev_nf4(*wq, inn), to_dev_nf4(*pq, r)
    Wq.absmax.fill_(float("nan"))                                    # the fp32 scales must not be read
    Pq.absmax.fill_(float("nan"))
    Wdq, Pdq = _to_dev_dq(*w8), _to_dev_dq(*p8)
    B, x, dy = padded(d["B"]), padded(d["x"]), padded(d["dy"])
    y = L.loqt_linear_fwd_dq(Wq, Wdq, Pq, Pdq, B, s, x)
    check_close(f32(y), ref_y, f"y (8-bit scales) {shape}")
    dx, dB = L.loqt_linear_bwd_dq(Wq, Wdq, Pq, Pdq, B, s, x, dy)
    check_close(f32(dx), ref_dx, f"dx (8-bit scales) {shape}")
    check_close(f32(dB), ref_dB, f"dB (8-bit scales) {shape}")
    # and it is a different layer from the one with fp32 scales: the test would notice if those were read
    plain = O.loqt_forward(wq, pq, Bh, s, xh, (out, inn, r))
    assert np.abs(plain - ref_y).max() > 1e-3 * np.abs(ref_y).max()


def test_dq_argument_errors():
    Wq = L.NF4Tensor.empty(64, 128)
    dq = L.DQScales.empty(64 * 2)
    bad = L.DQScales.empty(64 * 2 + 1)
    out = torch.empty((64, 128), dtype=torch.float32, device="cuda")
    assert L.lib().loqt_nf4_dequantize_dq(L._codes_only(Wq), bad.view(), out.data_ptr(), 128, 0, None) == 1
    assert L.lib().loqt_nf4_dequantize_dq(L._codes_only(Wq), dq.view(), None, 128, 0, None) == 1
