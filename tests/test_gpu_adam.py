"""GPU parity: loqt_adam_step (Algorithm 1 update line, rho = Adam) against the
CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import loqt_oracle as O
from paper_2405_16528_b200 import binding as L
from paper_2405_16528_b200 import synth
from tests.gpu_util import f32, padded

pytestmark = pytest.mark.gpu

BF16_STEP = 2.0 ** -7  # spacing of bf16 numbers relative to their magnitude, at most


def _f(x):
    """The C ABI carries hyper-parameters as fp32: both sides get the same number."""
    return float(np.float32(x))


B1, B2, EPS = _f(0.9), _f(0.999), _f(1e-8)


def _check_bf16(got, ref, scale, what):
    """fp32 arithmetic against float64: a result may land on the neighbouring bf16
    number when the exact value is within fp32 rounding of a bf16 rounding
    boundary; where the update cancels most of the operand (`scale`, the larger of
    the two terms) the fp32 rounding of the terms, 2^-22 of them, shows directly.
    Nothing else may differ."""
    got, ref = np.asarray(got, np.float64), np.asarray(ref, np.float64)
    bad = got != ref
    assert bad.mean() <= 2e-3, f"{what}: {bad.mean():.2e} of the entries differ"
    tol = BF16_STEP * np.abs(ref) + 2.0 ** -21 * np.asarray(scale, np.float64)
    assert np.all(np.abs(got - ref)[bad] <= tol[bad]), f"{what}: more than one bf16 step"


@pytest.mark.parametrize("shape", [(32, 256), (24, 136), (96, 5461), (128, 1376)])
@pytest.mark.parametrize("wd", [0.0, 0.1])
def test_steps_from_given_state(shape, wd):
    r, inn = shape
    B = synth.normal(50, ("B", r, inn), (r, inn), 1e-2, torch.bfloat16)
    m = synth.normal(50, ("m", r, inn), (r, inn), 1e-4, torch.bfloat16)
    v = (synth.normal(50, ("v", r, inn), (r, inn), 1e-4, torch.float32) ** 2).to(torch.bfloat16)
    g = synth.normal(50, ("g", r, inn), (r, inn), 1e-3, torch.float32)
    g[::5, ::3] = 0.0
    ld4 = (inn + 3) // 4 * 4
    gd = torch.zeros((r, ld4), dtype=torch.float32, device="cuda")[:, :inn]
    gd.copy_(g)
    wd = _f(wd)
    for step, lr in [(1, _f(1e-2)), (7, _f(5e-3)), (1000, _f(1e-3))]:
        rB, rm, rv = O.adam_step(f32(B), g.numpy(), f32(m), f32(v), step, lr, B1, B2, EPS, wd)
        Bd, md, vd = padded(B), padded(m), padded(v)
        L.loqt_adam_step(Bd, gd, md, vd, step, lr, B1, B2, EPS, wd)
        _check_bf16(f32(Bd), rB, np.maximum(np.abs(f32(B)), lr), f"B {shape} step {step}")
        _check_bf16(f32(md), rm, np.maximum(np.abs(f32(m)), np.abs(g.numpy())), f"m {shape} step {step}")
        _check_bf16(f32(vd), rv, np.abs(f32(v)), f"v {shape} step {step}")


def test_first_step_from_zero_state_moves_against_the_sign():
    r, inn = 16, 64
    g = synth.normal(51, ("g",), (r, inn), 1e-3, torch.float32)
    B = torch.ones((r, inn), dtype=torch.bfloat16, device="cuda")
    m = torch.zeros_like(B)
    v = torch.zeros_like(B)
    L.loqt_adam_step(B, g.cuda(), m, v, 1, 2.0 ** -6)
    assert np.array_equal(f32(B), 1.0 - 2.0 ** -6 * np.sign(g.numpy()))


def test_argument_errors():
    B = torch.zeros((8, 64), dtype=torch.bfloat16, device="cuda")
    g = torch.zeros((8, 64), dtype=torch.float32, device="cuda")
    with pytest.raises(L.LoqtError, match="invalid argument"):
        L.loqt_adam_step(B, g, B.clone(), B.clone(), 0, 1e-3)
    with pytest.raises(L.LoqtError, match="invalid argument"):
        L.loqt_adam_step(B, g, B.clone(), B.clone(), 1, 1e-3, beta1=1.0)
