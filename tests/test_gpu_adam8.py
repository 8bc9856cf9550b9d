"""GPU parity: loqt_adam8_step (Adam with 8-bit block-wise quantised moments, the
paper's "8-bit Adam") against the CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import loqt_oracle as O
from paper_2405_16528_b200 import binding as L
from paper_2405_16528_b200 import synth
from tests.gpu_util import f32, padded
from tests.test_gpu_adam import B1, B2, EPS, _check_bf16, _f

pytestmark = pytest.mark.gpu


def _dev_state(m8, mM, v8, vM):
    return [torch.from_numpy(a.copy()).cuda() for a in (m8, mM, v8, vM)]


def _check_codes(got8, gotM, ref8, refM, signed, what):
    """Codes are integers decided by fp32 values: the device computes the new
    moments in fp32, the oracle in float64 rounded to fp32, so a value within an
    ulp of a decision midpoint may take the neighbouring magnitude, and a block
    scale may be the neighbouring fp32 number (then a few more of its block's
    codes sit on the other side of a midpoint).  Nothing else may differ."""
    ulp = np.spacing(np.maximum(np.abs(refM), 1e-37).astype(np.float32))
    assert np.all(np.abs(gotM.astype(np.float64) - refM.astype(np.float64)) <= 2 * ulp), f"{what}: block scale off"
    mask = 0x7F if signed else 0xFF
    bad = got8 != ref8
    assert bad.mean() <= 5e-3, f"{what}: {bad.mean():.2e} of the codes differ"
    gi, ri = (got8[bad] & mask).astype(np.int64), (ref8[bad] & mask).astype(np.int64)
    assert np.all(np.abs(gi - ri) <= 1), f"{what}: a code differs by more than one magnitude"
    if signed:
        same_sign = (got8[bad] & 0x80) == (ref8[bad] & 0x80)
        assert np.all(same_sign | (np.minimum(gi, ri) == 0)), f"{what}: sign flipped away from zero"


def test_every_code_dequantises_like_the_oracle():
    # lr = 0, beta = 0 would still requantise; instead read the tables through one step with g = 0, beta1 = beta2 = 0.5:
    # m' = 0.5 m exactly, so the new scale is half the old and every code must come back unchanged
    n = 2048
    m8 = np.arange(n, dtype=np.uint8)                # every bit pattern, 8 times (0x80 = -0 decodes to 0 and recodes to 0)
    v8 = np.arange(n, dtype=np.uint8)
    mM, vM = np.array([2.0], dtype=np.float32), np.array([4.0], dtype=np.float32)
    B = torch.zeros((8, 256), dtype=torch.bfloat16, device="cuda")
    g = torch.zeros((8, 256), dtype=torch.float32, device="cuda")
    st = _dev_state(m8, mM, v8, vM)
    L.loqt_adam8_step(B, g, *st, 1, 0.0, beta1=0.5, beta2=0.5)
    rB, r8, rM, rv8, rvM = O.adam8_step(f32(B) * 0, g.cpu().numpy(), m8, mM, v8, vM, 1, 0.0, 0.5, 0.5)
    assert np.array_equal(st[0].cpu().numpy(), r8) and np.array_equal(st[2].cpu().numpy(), rv8)
    assert st[1].item() == 1.0 and st[3].item() == 2.0 and rM[0] == 1.0 and rvM[0] == 2.0
    want = m8.copy()
    want[want == 0x80] = 0
    assert np.array_equal(st[0].cpu().numpy(), want) and np.array_equal(st[2].cpu().numpy(), v8)


@pytest.mark.parametrize("shape", [(32, 256), (24, 136), (96, 5461), (128, 1376), (512, 2048)])
@pytest.mark.parametrize("wd", [0.0, 0.1])
def test_steps_against_the_oracle(shape, wd):
    r, inn = shape
    n = r * inn
    B = synth.normal(70, ("B", r, inn), (r, inn), 1e-2, torch.bfloat16)
    ld4 = (inn + 3) // 4 * 4
    wd = _f(wd)
    m8, mM = O.dyn8_quantize(np.zeros(n, dtype=np.float32), True)
    v8, vM = O.dyn8_quantize(np.zeros(n, dtype=np.float32), False)
    Bh = f32(B)
    for step, lr in [(1, _f(1e-2)), (2, _f(5e-3)), (3, _f(1e-3))]:
        g = synth.normal(70, ("g", r, inn, step), (r, inn), 1e-3, torch.float32)
        g[::5, ::3] = 0.0
        gd = torch.zeros((r, ld4), dtype=torch.float32, device="cuda")[:, :inn]
        gd.copy_(g)
        # both sides start the step from the same (oracle) state
        rB, r8, rM, rv8, rvM = O.adam8_step(Bh, g.numpy(), m8, mM, v8, vM, step, lr, B1, B2, EPS, wd)
        Bd = padded(torch.from_numpy(Bh).to(torch.bfloat16))
        st = _dev_state(m8, mM, v8, vM)
        L.loqt_adam8_step(Bd, gd, *st, step, lr, B1, B2, EPS, wd)
        _check_bf16(f32(Bd), rB, np.maximum(np.abs(Bh), lr), f"B {shape} step {step}")
        _check_codes(st[0].cpu().numpy(), st[1].cpu().numpy(), r8, rM, True, f"m {shape} step {step}")
        _check_codes(st[2].cpu().numpy(), st[3].cpu().numpy(), rv8, rvM, False, f"v {shape} step {step}")
        Bh, m8, mM, v8, vM = rB, r8, rM, rv8, rvM


def test_argument_errors():
    B = torch.zeros((8, 64), dtype=torch.bfloat16, device="cuda")
    g = torch.zeros((8, 64), dtype=torch.float32, device="cuda")
    m8 = torch.zeros(512, dtype=torch.uint8, device="cuda")
    a = torch.zeros(1, dtype=torch.float32, device="cuda")
    with pytest.raises(L.LoqtError, match="invalid argument"):
        L.loqt_adam8_step(B, g, m8, a, m8.clone(), a.clone(), 0, 1e-3)
    with pytest.raises(L.LoqtError, match="do not match"):
        L.loqt_adam8_step(B, g, m8[:100], a, m8.clone(), a.clone(), 1, 1e-3)
