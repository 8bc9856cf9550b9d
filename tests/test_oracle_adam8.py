"""Pins of the oracle's 8-bit optimiser states (the paper's "8-bit Adam"; reading:
block-wise quantised moments in the dynamic tree data type of Dettmers et al.).
No numbers are printed by the paper, so the pins are the data type's published
structure (sign, base-10 exponent run, indicator, linear fraction), brute-force
nearest-value quantisation, exact round trips, the error the type implies, and
the step itself against torch.optim.AdamW started from the dequantised moments."""
import numpy as np
import pytest
import torch

from oracle import loqt_oracle as O


@pytest.mark.parametrize("signed", [True, False])
def test_codebook_structure(signed):
    c = O.dyn8_codebook(signed).astype(np.float64)
    bits = 7 if signed else 8
    assert c.shape == (1 << bits,) and c[0] == 0.0
    assert np.all(np.diff(c) > 0)                                  # magnitudes ascend with the code
    assert c[-1] == 1.0                                            # all fraction bits set, no exponent zeros
    assert abs(c[1] - 10.0 ** -(bits - 1)) < 1e-12                 # longest zero run: the smallest decade, one value
    for f in range(bits):
        E = bits - 1 - f
        dec = c[(1 << f) : (1 << (f + 1))]                         # bit pattern: E zeros, indicator, f fraction bits
        assert len(dec) == 1 << f
        assert np.all((dec > 10.0 ** -(E + 1) * (1 - 1e-6)) & (dec <= 10.0 ** -E * (1 + 1e-6)))
        assert abs(dec[-1] - 10.0 ** -E) <= 1e-7 * 10.0 ** -E      # a decade ends at 10^-E
        if f >= 1:
            steps = np.diff(dec)
            assert np.allclose(steps, 0.9 * 10.0 ** -E / (1 << f), rtol=1e-5)  # linear inside the decade
    # finest resolution: the top decade of the unsigned type has 128 steps, the signed one 64
    assert abs((c[-1] - c[-2]) - 0.9 / (1 << (bits - 1))) < 1e-7


def _brute(n, c):
    d = np.abs(np.abs(n) - c.astype(np.float64))
    return int(np.argmin(d))  # first (smaller) on ties


@pytest.mark.parametrize("signed", [True, False])
def test_quantise_is_nearest_value_by_brute_force(signed):
    rng = np.random.default_rng(1)
    x = np.concatenate([rng.normal(0, 1, 3000), rng.normal(0, 1e-3, 1000), 10.0 ** rng.uniform(-9, 0, 1000), [0.0, 1e-30]])
    x = (np.abs(x) if not signed else x).astype(np.float32)
    codes, M = O.dyn8_quantize(x, signed)
    c = O.dyn8_codebook(signed)
    assert M.shape == ((x.size + 2047) // 2048,)
    for b in range(M.size):
        blk = x[b * 2048 : (b + 1) * 2048]
        assert M[b] == np.max(np.abs(blk))
        n = (blk / M[b]).astype(np.float32).astype(np.float64)
        for k in range(0, blk.size, 7):
            idx = _brute(n[k], c)
            want = idx | (0x80 if (signed and n[k] < 0 and idx > 0) else 0)
            assert codes[b * 2048 + k] == want
    # the block maximum normalises to exactly 1 and takes the top code
    k = int(np.argmax(np.abs(x[:2048])))
    assert (codes[k] & (0x7F if signed else 0xFF)) == (127 if signed else 255)


@pytest.mark.parametrize("signed", [True, False])
def test_codebook_values_round_trip_and_error_bound(signed):
    c = O.dyn8_codebook(signed)
    x = (c * np.float32(4.0)).astype(np.float32)                   # M = 4: every magnitude exactly representable
    if signed:
        x = np.concatenate([x, -x[1:]])
    codes, M = O.dyn8_quantize(x, signed)
    assert M[0] == 4.0
    assert np.array_equal(O.dyn8_dequantize(codes, M, signed), x)
    # relative error: at most half a linear step, 0.45 * 10^-E / 2^f over a value >= 10^-(E+1); worst in the
    # decades with few fraction bits, at most 0.45 / 0.1 / 2^f relative; in the top decade <= 0.45 / 2^f / 0.1
    rng = np.random.default_rng(2)
    y = rng.uniform(0.1, 1.0, 2048).astype(np.float32)
    y[0] = 1.0
    cy, My = O.dyn8_quantize(y, signed)
    back = O.dyn8_dequantize(cy, My, signed)
    f_top = 6 if signed else 7
    assert np.max(np.abs(back - y)) <= 0.45 / (1 << f_top) + 1e-6


def test_zero_block_and_short_last_block():
    x = np.zeros(2048 + 10, dtype=np.float32)
    x[2048 + 3] = -0.5
    codes, M = O.dyn8_quantize(x, True)
    assert M[0] == 0 and M[1] == 0.5 and not codes[:2048].any()
    assert codes[2048 + 3] == (0x80 | 127)
    assert np.array_equal(O.dyn8_dequantize(codes, M, True), x)


@pytest.mark.parametrize("wd", [0.0, 0.1])
def test_step_matches_torch_adamw_from_the_dequantised_moments(wd):
    rng = np.random.default_rng(3)
    shape = (24, 200)                                              # 4800 elements: two full blocks and a short one
    B = O.bf16_round(rng.normal(0, 1e-2, shape).astype(np.float32))
    m8, mM = O.dyn8_quantize(np.zeros(B.size, dtype=np.float32), True)
    v8, vM = O.dyn8_quantize(np.zeros(B.size, dtype=np.float32), False)
    lr, b1, b2, eps = 1e-2, 0.9, 0.999, 1e-8
    for step in range(1, 5):
        g = rng.normal(0, 1e-3, shape).astype(np.float32)
        m = O.dyn8_dequantize(m8, mM, True).reshape(shape)
        v = O.dyn8_dequantize(v8, vM, False).reshape(shape)
        p = torch.tensor(B, dtype=torch.float64, requires_grad=True)
        opt = torch.optim.AdamW([p], lr=lr, betas=(b1, b2), eps=eps, weight_decay=wd)
        opt.state[p] = {"step": torch.tensor(float(step - 1)), "exp_avg": torch.tensor(m, dtype=torch.float64),
                        "exp_avg_sq": torch.tensor(v, dtype=torch.float64)}
        p.grad = torch.tensor(g, dtype=torch.float64)
        opt.step()
        Bn, m8n, mMn, v8n, vMn = O.adam8_step(B, g, m8, mM, v8, vM, step, lr, b1, b2, eps, wd)
        ref = p.detach().numpy()
        assert np.all(np.abs(Bn - ref) <= 2.0 ** -8 * np.abs(ref) + 1e-30)            # half a bf16 step
        # the new moments are the library's, quantised: within the type's resolution of them
        m_ref, v_ref = opt.state[p]["exp_avg"].numpy(), opt.state[p]["exp_avg_sq"].numpy()
        m_new = O.dyn8_dequantize(m8n, mMn, True).reshape(shape)
        v_new = O.dyn8_dequantize(v8n, vMn, False).reshape(shape)
        # ... i.e. no further from them than half the gap between the two values of the type that enclose them
        def half_gap(ref, M, signed):
            c = O.dyn8_codebook(signed).astype(np.float64)
            Mx = np.repeat(M.astype(np.float64), 2048)[: B.size].reshape(shape)
            n = np.abs(ref) / np.where(Mx > 0, Mx, 1.0)
            hi = np.clip(np.searchsorted(c, n, side="left"), 1, len(c) - 1)
            return 0.5 * (c[hi] - c[hi - 1]) * Mx * (1 + 1e-5) + 1e-30
        assert np.all(np.abs(m_new - m_ref) <= half_gap(m_ref, mMn, True))
        assert np.all(np.abs(v_new - v_ref) <= half_gap(v_ref, vMn, False))
        assert np.all(mMn == np.array([np.max(np.abs(m_ref.astype(np.float32).reshape(-1)[k:k + 2048])) for k in range(0, B.size, 2048)]))
        B, m8, mM, v8, vM = Bn, m8n, mMn, v8n, vMn
    # after four steps the 8-bit run stays close to the plain bf16-state oracle started alike
    assert np.max(np.abs(B)) > 0
