"""GPU parity: loqt_compensated_init (Section 2.5, Algorithm 2 compensation loop)
against the CPU oracle on the same seeded inputs, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import loqt_oracle as O
from paper_2405_16528_b200 import binding as L
from paper_2405_16528_b200 import synth
from tests.gpu_util import check_close, f32, from_dev_nf4

pytestmark = pytest.mark.gpu

# (out, in, r): several tiles with ragged edges; 5461 is the paper's 1B MLP width; then
# tiny and ragged cases: fewer rows than the 32 of an epilogue warp, a width below one
# staging tile, widths that end inside the first and inside the second half of a block;
# last, more tiles than the GPU has SMs, so that a CTA walks several tiles (272 of 128 x 256)
SHAPES = [(256, 256, 32), (384, 320, 64), (200, 136, 24), (640, 5461, 96), (1376, 512, 128),
          (24, 40, 8), (72, 24, 16), (136, 100, 8), (520, 1065, 40), (2176, 4000, 192)]


def _inputs(seed, out, inn, r):
    W = synth.normal(seed, ("W", out, inn), (out, inn), 0.02)
    P = synth.orthonormal(seed, ("P", out, r), out, r)
    ld = (inn + 3) // 4 * 4
    Wd = torch.zeros((out, ld), dtype=torch.float32, device="cuda")[:, :inn]
    Wd.copy_(W)
    return W.numpy(), P.numpy(), Wd, P.cuda()


def _error(W, P, codes, absmax, B, inn):
    Pb = O.bf16_round(P).astype(np.float64)
    return np.linalg.norm(W.astype(np.float64) - O.nf4_dequantize(codes, absmax, inn) - Pb @ B.astype(np.float64)) ** 2


@pytest.mark.parametrize("shape", SHAPES)
def test_one_step(shape):
    out, inn, r = shape
    W, P, Wd, Pd = _inputs(40, out, inn, r)
    (rc, rm), rB = O.loqt_compensate(W, P, 1)
    Wq, Pq, B = L.loqt_compensated_init(Wd, Pd, 1)
    c, m = from_dev_nf4(Wq)
    assert np.array_equal(c, rc) and np.array_equal(m, rm)          # Q_1 = q(W): integer work, bit-exact
    pc, pm = from_dev_nf4(Pq)
    qc, qm = O.nf4_quantize(P)
    assert np.array_equal(pc, qc) and np.array_equal(pm, qm)
    check_close(f32(B), rB, f"B_1 {shape}")
    # B holds bf16 values that differ from the oracle's by at most one bf16 step where
    # the fp32 and fp64 sums fall on different sides of a rounding boundary
    assert np.mean(f32(B) != rB) < 2e-2


@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("steps", [2, 5])
def test_each_step_from_the_previous_state(shape, steps):
    # The iteration amplifies differences: one code that falls on the other side of a
    # decision boundary shifts B in its column, which moves every corrected weight of
    # that column in the next step.  After several steps the codes are therefore not
    # unique (any fp32 summation order gives its own trajectory), but each step is a
    # function of the previous B.  The library is deterministic, so the run with
    # steps - 1 returns the state the longer run passes through: the oracle takes
    # one step from it and must land where the library does.
    out, inn, r = shape
    W, P, Wd, Pd = _inputs(41, out, inn, r)
    _, _, B_prev = L.loqt_compensated_init(Wd, Pd, steps - 1)
    (rc, rm), rB = O.loqt_compensate(W, P, 1, B0=f32(B_prev))
    Wq, Pq, B = L.loqt_compensated_init(Wd, Pd, steps)
    c, m = from_dev_nf4(Wq)
    # W - P B is summed in fp32 on the GPU: a value within that rounding of a
    # decision boundary may take the neighbouring code
    diff = c[:, :inn] != rc[:, :inn]
    assert diff.mean() <= 1e-4, f"{diff.mean():.2e} of the codes differ"
    assert np.all(np.abs(c[:, :inn].astype(int) - rc[:, :inn].astype(int))[diff] == 1)
    assert np.all(c[:, inn:] == 7)
    assert np.abs(m - rm).max() <= 2.0 ** -20 * np.abs(rm).max()
    # B against the oracle's in every column whose codes agree (a flipped code moves
    # its residual by a whole level gap), and against the definition evaluated by the
    # oracle's routines on the library's own codes everywhere
    clean = ~diff.any(axis=0)
    check_close(f32(B)[:, clean], rB[:, clean], f"B_{steps} {shape} (columns without a flipped code)")
    Pb = O.bf16_round(P).astype(np.float64)
    resid = O.bf16_round((W - O.nf4_dequantize(c, m, inn)).astype(np.float32)).astype(np.float64)
    check_close(f32(B), O.bf16_round((Pb.T @ resid).astype(np.float32)), f"B_{steps} {shape} (from the library's codes)")


@pytest.mark.parametrize("shape", SHAPES)
def test_five_steps_fit_as_well_as_the_oracle(shape):
    # what is unique after several steps: the quality of the fit
    out, inn, r = shape
    W, P, Wd, Pd = _inputs(44, out, inn, r)
    (rc, rm), rB = O.loqt_compensate(W, P, 5)
    Wq, Pq, B = L.loqt_compensated_init(Wd, Pd, 5)
    c, m = from_dev_nf4(Wq)
    e_gpu = _error(W, P, c, m, f32(B), inn)
    e_ref = _error(W, P, rc, rm, rB, inn)
    e_0 = np.linalg.norm(W - O.nf4_dequantize(*O.nf4_quantize(W), inn)) ** 2
    assert abs(e_gpu - e_ref) <= 2e-3 * e_ref and e_gpu < (1 - 0.7 * r / out) * e_0
    assert (c[:, :inn] != rc[:, :inn]).mean() <= 2e-2


def test_representable_weights_need_no_correction():
    out, inn, r = 256, 320, 32
    W, P, Wd, Pd = _inputs(42, out, inn, r)
    q0 = O.nf4_quantize(W)
    Wd.copy_(torch.from_numpy(O.nf4_dequantize(q0[0], q0[1], inn)))
    Wq, Pq, B = L.loqt_compensated_init(Wd, Pd, 3)
    c, m = from_dev_nf4(Wq)
    assert np.array_equal(c, q0[0]) and np.array_equal(m, q0[1]) and not f32(B).any()


def test_rows_of_very_different_scale_share_a_warp():
    # Block scales beyond 2^+-60 take the IEEE division, the others the division by
    # reciprocal, and all-zero rows neither: here the three kinds sit in neighbouring rows,
    # so the lanes of one epilogue warp part ways inside a block.  The weights are
    # representable (scaling a row by a power of two keeps them so), which makes the
    # expected result exact: the codes and scales of q(W), B = 0.
    out, inn, r = 256, 320, 32
    W, P, Wd, Pd = _inputs(47, out, inn, r)
    q0 = O.nf4_quantize(W)
    k = np.array([0, 70, -70, 0, 65, -65, 0, 0])[np.arange(out) % 8]
    Wr = (O.nf4_dequantize(q0[0], q0[1], inn) * (2.0 ** k)[:, None]).astype(np.float32)
    Wr[np.arange(out) % 16 == 5] = 0.0
    ref_c, ref_m = O.nf4_quantize(Wr)
    Wd.copy_(torch.from_numpy(Wr))
    Wq, Pq, B = L.loqt_compensated_init(Wd, Pd, 3)
    c, m = from_dev_nf4(Wq)
    assert np.array_equal(c, ref_c) and np.array_equal(m, ref_m) and not f32(B).any()


def test_argument_errors():
    out, inn, r = 256, 256, 32
    W, P, Wd, Pd = _inputs(43, out, inn, r)
    with pytest.raises(L.LoqtError, match="invalid argument"):
        L.loqt_compensated_init(Wd, Pd, 0)
    with pytest.raises(L.LoqtError, match="workspace"):
        L.loqt_compensated_init(Wd, Pd, 1, ws=L.new_workspace(1024))


# ---- right-side variant: W ~ Q_w + B Q, Q r x in with orthonormal rows
RIGHT_SHAPES = [(256, 256, 32), (1376, 512, 96), (5461, 256, 40), (320, 640, 64), (4000, 2176, 192)]  # the last: 288 tiles


def _inputs_right(seed, out, inn, r):
    W = synth.normal(seed, ("W", out, inn), (out, inn), 0.02)
    Q = synth.orthonormal(seed, ("Q", inn, r), inn, r).T.contiguous()
    ld = (inn + 3) // 4 * 4
    Wd = torch.zeros((out, ld), dtype=torch.float32, device="cuda")[:, :inn]
    Wd.copy_(W)
    return W.numpy(), Q.numpy(), Wd, Q.cuda()


@pytest.mark.parametrize("shape", RIGHT_SHAPES)
@pytest.mark.parametrize("steps", [1, 2, 4])
def test_right_variant_each_step_from_the_previous_state(shape, steps):
    out, inn, r = shape
    W, Q, Wd, Qd = _inputs_right(45, out, inn, r)
    if steps == 1:
        (rc, rm), rB = O.loqt_compensate_right(W, Q, 1)
    else:
        _, _, B_prev = L.loqt_compensated_init_right(Wd, Qd, steps - 1)
        (rc, rm), rB = O.loqt_compensate_right(W, Q, 1, B0=f32(B_prev))
    Wq, Qq, B = L.loqt_compensated_init_right(Wd, Qd, steps)
    c, m = from_dev_nf4(Wq)
    qc, qm = from_dev_nf4(Qq)
    oc, om = O.nf4_quantize(Q)
    assert np.array_equal(qc, oc) and np.array_equal(qm, om)
    diff = c[:, :inn] != rc[:, :inn]
    if steps == 1:
        assert not diff.any() and np.array_equal(m, rm)          # Q_1 = q(W): bit-exact
    assert diff.mean() <= 1e-4, f"{diff.mean():.2e} of the codes differ"
    assert np.all(np.abs(c[:, :inn].astype(int) - rc[:, :inn].astype(int))[diff] == 1)
    assert np.all(c[:, inn:] == 7)
    assert np.abs(m - rm).max() <= 2.0 ** -20 * np.abs(rm).max()
    clean = ~diff.any(axis=1)                                    # rows without a flipped code
    check_close(f32(B)[clean], rB[clean], f"B_{steps} {shape} (rows without a flipped code)")
    Qb = O.bf16_round(Q).astype(np.float64)
    resid = O.bf16_round((W - O.nf4_dequantize(c, m, inn)).astype(np.float32)).astype(np.float64)
    check_close(f32(B), O.bf16_round((resid @ Qb.T).astype(np.float32)), f"B_{steps} {shape} (from the library's codes)")


def test_right_variant_representable_weights_need_no_correction():
    out, inn, r = 256, 320, 32
    W, Q, Wd, Qd = _inputs_right(46, out, inn, r)
    q0 = O.nf4_quantize(W)
    Wd.copy_(torch.from_numpy(O.nf4_dequantize(q0[0], q0[1], inn)))
    Wq, Qq, B = L.loqt_compensated_init_right(Wd, Qd, 3)
    c, m = from_dev_nf4(Wq)
    assert np.array_equal(c, q0[0]) and np.array_equal(m, q0[1]) and not f32(B).any()
