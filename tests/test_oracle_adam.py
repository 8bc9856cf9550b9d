"""Pins of the oracle's optimiser step (Algorithm 1 update line; Adam per Kingma &
Ba with decoupled weight decay) against PyTorch's CPU optimisers and closed forms."""
import numpy as np
import pytest
import torch

from oracle import loqt_oracle as O


def _bf(a):
    return O.bf16_round(np.asarray(a, dtype=np.float32))


@pytest.mark.parametrize("wd", [0.0, 0.1])
def test_matches_torch_adamw_over_several_steps(wd):
    # torch.optim.AdamW in float64 is the library routine; the oracle rounds its
    # state to bf16 after every step, so the comparison restarts the library from the
    # oracle's rounded state each step and must agree to float64 accuracy before
    # rounding, i.e. to half a bf16 step after it.
    rng = np.random.default_rng(0)
    B = _bf(rng.normal(0, 1e-2, (8, 24)))
    m = np.zeros_like(B)
    v = np.zeros_like(B)
    lr, b1, b2, eps = 1e-2, 0.9, 0.999, 1e-8
    for step in range(1, 6):
        g = rng.normal(0, 1e-3, B.shape).astype(np.float32)
        p = torch.tensor(B, dtype=torch.float64, requires_grad=True)
        opt = torch.optim.AdamW([p], lr=lr, betas=(b1, b2), eps=eps, weight_decay=wd)
        opt.state[p] = {"step": torch.tensor(float(step - 1)), "exp_avg": torch.tensor(m, dtype=torch.float64),
                        "exp_avg_sq": torch.tensor(v, dtype=torch.float64)}
        p.grad = torch.tensor(g, dtype=torch.float64)
        opt.step()
        Bn, mn, vn = O.adam_step(B, g, m, v, step, lr, b1, b2, eps, wd)
        ref = p.detach().numpy()
        assert np.all(np.abs(Bn - ref) <= 2.0 ** -8 * np.abs(ref) + 1e-30)
        assert np.all(np.abs(mn - opt.state[p]["exp_avg"].numpy()) <= 2.0 ** -8 * np.abs(mn) + 1e-30)
        assert np.all(np.abs(vn - opt.state[p]["exp_avg_sq"].numpy()) <= 2.0 ** -8 * np.abs(vn) + 1e-30)
        B, m, v = Bn, mn, vn


def test_first_step_moves_by_the_learning_rate_against_the_gradient_sign():
    # t = 1, zero state: mhat = g, vhat = g^2, so the step is lr * g / (|g| + eps)
    g = np.array([[0.5, -0.25, 2.0, -1e-3]], dtype=np.float32)
    B = _bf(np.array([[1.0, 1.0, -1.0, 0.5]]))
    Bn, m, v = O.adam_step(B, g, np.zeros_like(B), np.zeros_like(B), 1, lr=2.0 ** -6)
    assert np.array_equal(Bn, _bf(B - 2.0 ** -6 * np.sign(g)))
    assert np.array_equal(m, _bf(0.1 * g)) and np.array_equal(v, _bf(0.001 * g.astype(np.float64) ** 2))


def test_zero_gradient_with_weight_decay_only_shrinks():
    B = _bf(np.array([[1.0, -2.0, 0.5]]))
    z = np.zeros_like(B)
    Bn, m, v = O.adam_step(B, z, z, z, 3, lr=0.125, weight_decay=0.5)
    assert np.array_equal(Bn, _bf(B * (1 - 0.125 * 0.5))) and not m.any() and not v.any()
