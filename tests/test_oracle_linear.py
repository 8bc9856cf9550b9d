"""Pins for the oracle's forward, backward and merge.

Independent routes: the explicit dense matrix W_eff = W + s P B formed on the
CPU (Section 2 update rule / Alg. 1 merge line), the identity G^B = P^T G^W
("Equivalence of Gradient Updates"), torch float64 autograd on the dense layer,
and central finite differences of L = <y, dy>.
"""
import numpy as np
import pytest
import torch

from oracle import loqt_oracle as O
from paper_2405_16528_b200 import synth


def _layer(seed, out, inn, r, T, sigma_B=1e-2):
    d = synth.make_layer(seed, "t", out, inn, r, sigma_B, T)
    wq = O.nf4_quantize(d["W"].numpy())
    pq = O.nf4_quantize(d["P"].numpy())
    f = lambda t: t.to(torch.float32).numpy()
    return wq, pq, f(d["B"]), f(d["x"]), f(d["dy"])


def _dense(wq, pq, B, s, shape):
    """W_eff built entry by entry from the stored codes; no oracle GEMM code."""
    out, inn, r = shape
    lv = O.NF4_LEVELS
    W = np.zeros((out, inn))
    P = np.zeros((out, r))
    bf = lambda v: float(torch.tensor(float(v), dtype=torch.float32).to(torch.bfloat16))
    for o in range(out):
        for i in range(inn):
            W[o, i] = bf(np.float32(wq[1][o, i // 64]) * lv[wq[0][o, i]])
        for k in range(r):
            P[o, k] = bf(np.float32(pq[1][o, k // 64]) * lv[pq[0][o, k]])
    return W, P, W + s * (P @ B.astype(np.float64))


SHAPES = [(48, 80, 8, 5), (64, 64, 16, 9), (70, 130, 24, 3)]


@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("s", [1.0, 0.5])
def test_forward_equals_dense_layer(shape, s):
    out, inn, r, T = shape
    wq, pq, B, x, dy = _layer(1, out, inn, r, T)
    _, _, Weff = _dense(wq, pq, B, s, (out, inn, r))
    y = O.loqt_forward(wq, pq, B, s, x, (out, inn, r))
    ref = x.astype(np.float64) @ Weff.T
    assert np.max(np.abs(y - ref)) <= 1e-12 * np.max(np.abs(ref))


@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("s", [1.0, 0.25])
def test_backward_dense_route_and_projection_identity(shape, s):
    out, inn, r, T = shape
    wq, pq, B, x, dy = _layer(2, out, inn, r, T)
    W, P, Weff = _dense(wq, pq, B, s, (out, inn, r))
    dx, dB = O.loqt_backward(wq, pq, B, s, x, dy, (out, inn, r))
    x64, dy64 = x.astype(np.float64), dy.astype(np.float64)
    GW = dy64.T @ x64  # out x in, the full-rank gradient
    assert np.allclose(dx, dy64 @ Weff, rtol=0, atol=1e-11 * np.max(np.abs(dx)))
    assert np.allclose(dB, s * (P.T @ GW), rtol=0, atol=1e-11 * np.max(np.abs(dB)))


def test_backward_matches_torch_autograd():
    out, inn, r, T, s = 40, 72, 8, 6, 0.5
    wq, pq, B, x, dy = _layer(3, out, inn, r, T)
    W, P, _ = _dense(wq, pq, B, s, (out, inn, r))
    tW, tP = torch.tensor(W), torch.tensor(P)
    tB = torch.tensor(B, dtype=torch.float64, requires_grad=True)
    tx = torch.tensor(x, dtype=torch.float64, requires_grad=True)
    y = torch.nn.functional.linear(tx, tW + s * tP @ tB)
    (y * torch.tensor(dy, dtype=torch.float64)).sum().backward()
    dx, dB = O.loqt_backward(wq, pq, B, s, x, dy, (out, inn, r))
    assert np.allclose(y.detach().numpy(), O.loqt_forward(wq, pq, B, s, x, (out, inn, r)), rtol=1e-11, atol=1e-12)
    assert np.allclose(dx, tx.grad.numpy(), rtol=1e-10, atol=1e-12)
    assert np.allclose(dB, tB.grad.numpy(), rtol=1e-10, atol=1e-12)


def test_backward_finite_differences():
    out, inn, r, T, s = 24, 64, 4, 3, 0.5
    wq, pq, B, x, dy = _layer(4, out, inn, r, T)
    shape = (out, inn, r)
    L = lambda B_, x_: float(np.sum(O.loqt_forward(wq, pq, B_, s, x_, shape) * dy))
    dx, dB = O.loqt_backward(wq, pq, B, s, x, dy, shape)
    rng = np.random.default_rng(0)
    B64, x64 = B.astype(np.float64), x.astype(np.float64)
    h = 1e-4
    for _ in range(10):
        k, i = rng.integers(r), rng.integers(inn)
        Bp, Bm = B64.copy(), B64.copy()
        Bp[k, i] += h
        Bm[k, i] -= h
        assert abs((L(Bp, x64) - L(Bm, x64)) / (2 * h) - dB[k, i]) <= 1e-6 * (1 + abs(dB[k, i]))
        t, j = rng.integers(T), rng.integers(inn)
        xp, xm = x64.copy(), x64.copy()
        xp[t, j] += h
        xm[t, j] -= h
        assert abs((L(B64, xp) - L(B64, xm)) / (2 * h) - dx[t, j]) <= 1e-6 * (1 + abs(dx[t, j]))


def test_forward_special_cases():
    out, inn, r, T = 64, 128, 16, 4
    wq, pq, B, x, dy = _layer(5, out, inn, r, T)
    shape = (out, inn, r)
    # B = 0: a plain weight-only-quantised linear
    y0 = O.loqt_forward(wq, pq, np.zeros_like(B), 1.0, x, shape)
    W = O.nf4_dequantize_bf16(*wq).astype(np.float64)
    assert np.allclose(y0, x.astype(np.float64) @ W.T, rtol=1e-13)
    # W_q = 0: pure low-rank adapter
    z = (np.full_like(wq[0], 7), np.zeros_like(wq[1]))
    P = O.nf4_dequantize_bf16(*pq, r).astype(np.float64)
    y1 = O.loqt_forward(z, pq, B, 0.5, x, shape)
    assert np.allclose(y1, 0.5 * x.astype(np.float64) @ (P @ B.astype(np.float64)).T, rtol=1e-11, atol=1e-13)
    # the scale is linear in the adapter term
    ya = O.loqt_forward(wq, pq, B, 1.0, x, shape)
    yb = O.loqt_forward(wq, pq, B, 0.5, x, shape)
    assert np.allclose(ya - y0, 2 * (yb - y0), rtol=1e-9, atol=1e-12)


def test_merge_zero_B_is_identity():
    out, inn, r, T = 64, 192, 16, 2
    wq, pq, B, x, dy = _layer(6, out, inn, r, T)
    c, m = O.loqt_merge_requant(wq, pq, np.zeros_like(B), 1.0, (out, inn, r))
    assert np.array_equal(c, wq[0]) and np.array_equal(m, wq[1])


@pytest.mark.parametrize("shape", [(64, 128, 16), (40, 100, 8)])
def test_merge_equals_quantised_dense_sum(shape):
    out, inn, r = shape
    s = 0.5
    wq, pq, B, x, dy = _layer(7, out, inn, r, 2, sigma_B=3e-2)
    W, P, _ = _dense(wq, pq, B, s, shape)  # W here is bf16-rounded; rebuild the fp32 one
    W32 = np.zeros((out, inn))
    for o in range(out):
        for i in range(inn):
            W32[o, i] = float(np.float32(wq[1][o, i // 64]) * O.NF4_LEVELS[wq[0][o, i]])
    tP = torch.tensor(P, dtype=torch.float64)
    tB = torch.tensor(B, dtype=torch.float64)
    vw = (W32 + s * (tP @ tB).numpy()).astype(np.float32)
    assert np.array_equal(O.loqt_merge_values(wq, pq, B, s, shape), vw)
    # brute-force quantisation of that matrix, block by block
    from tests.test_oracle_nf4 import _brute_quantize_block

    c, m = O.loqt_merge_requant(wq, pq, B, s, shape)
    for o in range(0, out, 7):
        for b in range(O.padded_cols(inn) // 64):
            c0, c1 = b * 64, min(b * 64 + 64, inn)
            bc, bm = _brute_quantize_block(list(vw[o, c0:c1]))
            assert list(c[o, c0:c1]) == bc and m[o, b] == bm


def test_merge_changes_more_codes_for_larger_B():
    """Section 2.5: small P B leaves the quantised state (almost) unchanged, a
    larger one moves it."""
    out, inn, r = 128, 256, 32
    frac = []
    for sig in (1e-4, 1e-3, 1e-2, 1e-1):
        wq, pq, B, _, _ = _layer(8, out, inn, r, 2, sigma_B=sig)
        c, _ = O.loqt_merge_requant(wq, pq, B, 1.0, (out, inn, r))
        frac.append(float(np.mean(c != wq[0])))
    assert frac[0] <= frac[1] <= frac[2] <= frac[3]
    assert frac[0] < 0.01 and frac[3] > 0.3


def test_merged_weight_reproduces_adapter_output():
    """After a merge, the plain quantised layer approximates the adapted one to
    within NF4's quantisation error (half the widest level gap times absmax)."""
    out, inn, r, T, s = 64, 128, 16, 8, 1.0
    wq, pq, B, x, dy = _layer(9, out, inn, r, T, sigma_B=2e-2)
    shape = (out, inn, r)
    vw = O.loqt_merge_values(wq, pq, B, s, shape).astype(np.float64)
    c, m = O.loqt_merge_requant(wq, pq, B, s, shape)
    half_gap = float(np.max(np.diff(O.NF4_LEVELS.astype(np.float64)))) / 2
    err = np.abs(O.nf4_dequantize(c, m).astype(np.float64) - vw)
    assert np.all(err <= np.repeat(m.astype(np.float64), 64, axis=1)[:, :inn] * half_gap * (1 + 1e-6))
    y_adapt = O.loqt_forward(wq, pq, B, s, x, shape)
    y_merged = O.loqt_forward((c, m), pq, np.zeros_like(B), s, x, shape)
    bound = np.abs(x.astype(np.float64)) @ (np.repeat(m.astype(np.float64), 64, axis=1)[:, :inn] * (half_gap + 2 ** -8)).T
    assert np.all(np.abs(y_adapt - y_merged) <= bound + 1e-9)


def test_requantize_zero_delta_is_identity():
    out, inn, r, T = 48, 200, 8, 2
    wq, pq, B, x, dy = _layer(21, out, inn, r, T)
    c, m = O.nf4_requantize(wq, np.zeros((out, inn), np.float32), 1.0, inn)
    assert np.array_equal(c, wq[0]) and np.array_equal(m, wq[1])


def test_requantize_cancelling_delta_gives_zero_weights():
    # s * delta = -deq32(W) exactly (halving and doubling are exact): every block
    # becomes all-zero, i.e. code 7 and scale 0.  A wrong sign or a dropped s fails.
    out, inn, r, T = 32, 128, 8, 2
    wq, pq, B, x, dy = _layer(22, out, inn, r, T)
    W32 = O.nf4_dequantize(wq[0], wq[1], inn)
    c, m = O.nf4_requantize(wq, -0.5 * W32, 2.0, inn)
    assert np.all(c == 7) and np.all(m == 0)


@pytest.mark.parametrize("s", [1.0, 0.25])
def test_requantize_equals_merge_for_rank_one(s):
    # With r = 1 every element of P_BF16 @ B is one product of two bf16 numbers,
    # exact in fp32, so handing that product to the requantiser must reproduce the
    # merge bit for bit.
    out, inn, r, T = 40, 192, 1, 2
    wq, pq, B, x, dy = _layer(23, out, inn, r, T)
    P = O.nf4_dequantize_bf16(pq[0], pq[1], r).astype(np.float64)
    delta = (P @ B.astype(np.float64)).astype(np.float32)
    assert np.array_equal(delta.astype(np.float64), P @ B.astype(np.float64))
    c, m = O.nf4_requantize(wq, delta, s, inn)
    rc, rm = O.loqt_merge_requant(wq, pq, B, s, (out, inn, r))
    assert np.array_equal(c, rc) and np.array_equal(m, rm)


# ---- error-compensated initialisation (Section 2.5, Algorithm 2)
def _ortho(seed, out, r):
    return synth.orthonormal(seed, ("P", out, r), out, r).numpy()


def test_compensate_first_step_is_the_least_squares_fit():
    # After one step Q = q(W) exactly, and B is the minimiser of ||Q + P B - W||
    # over B: numpy's least-squares routine on the same 16-bit P gives it.
    out, inn, r = 96, 128, 24
    W = synth.normal(31, ("W",), (out, inn), 0.02).numpy()
    P = _ortho(31, out, r)
    (c, m), B = O.loqt_compensate(W, P, 1)
    rc, rm = O.nf4_quantize(W)
    assert np.array_equal(c, rc) and np.array_equal(m, rm)
    Pb = O.bf16_round(P).astype(np.float64)
    resid = W.astype(np.float64) - O.nf4_dequantize(c, m, inn)
    ls = np.linalg.lstsq(Pb, resid, rcond=None)[0]
    assert np.abs(B - ls).max() <= 2.0 ** -7 * np.abs(ls).max()   # two 16-bit roundings
    # a sign slip (B = P^+ (Q - W)) would give -ls
    assert np.abs(B + ls).max() > 0.5 * np.abs(ls).max()


def test_compensate_reduces_the_error_as_the_projection_predicts():
    # With B the least-squares fit for Q = q(W), the error W - (Q + P B) is the part
    # of W - Q outside the span of P: its squared norm drops by about r / out for a
    # quantisation error that is spread evenly over directions.  Further steps
    # re-quantise the corrected weights and keep lowering the error (Section 2.5:
    # "iteratively refine").
    out, inn, r = 128, 256, 32
    W = synth.normal(32, ("W",), (out, inn), 0.02).numpy()
    P = _ortho(32, out, r)
    Pb = O.bf16_round(P).astype(np.float64)
    e0 = np.linalg.norm(W - O.nf4_dequantize(*O.nf4_quantize(W), inn)) ** 2
    errs = []
    for steps in (1, 2, 3, 5):
        (c, m), B = O.loqt_compensate(W, P, steps)
        errs.append(np.linalg.norm(W.astype(np.float64) - O.nf4_dequantize(c, m, inn) - Pb @ B.astype(np.float64)) ** 2)
    assert (1 - 1.3 * r / out) * e0 < errs[0] < (1 - 0.7 * r / out) * e0
    assert all(b < a for a, b in zip(errs, errs[1:]))


def test_compensate_representable_weights_need_no_correction():
    out, inn, r = 64, 128, 16
    W0 = synth.normal(33, ("W",), (out, inn), 0.02).numpy()
    q0 = O.nf4_quantize(W0)
    W = O.nf4_dequantize(q0[0], q0[1], inn)      # exactly representable
    (c, m), B = O.loqt_compensate(W, _ortho(33, out, r), 3)
    assert np.array_equal(c, q0[0]) and np.array_equal(m, q0[1]) and not B.any()


def test_compensate_later_steps_use_the_corrected_weights():
    # Step 2 quantises W - P B_1, not W: feeding that matrix to the quantiser by hand
    # must give the same codes.
    out, inn, r = 96, 192, 24
    W = synth.normal(34, ("W",), (out, inn), 0.02).numpy()
    P = _ortho(34, out, r)
    _, B1 = O.loqt_compensate(W, P, 1)
    (c2, m2), _ = O.loqt_compensate(W, P, 2)
    what = (W.astype(np.float64) - O.bf16_round(P).astype(np.float64) @ B1.astype(np.float64)).astype(np.float32)
    rc, rm = O.nf4_quantize(what)
    assert np.array_equal(c2, rc) and np.array_equal(m2, rm)
    assert not np.array_equal(c2, O.nf4_quantize(W)[0])


def test_full_gradient_is_the_dense_weight_gradient_and_projects_to_dB():
    # G^W is what autograd gives for the dense layer y = x W^T, and the factor's
    # gradient is its projection: dB = s P^T G^W (Section 2, "Equivalence of
    # Gradient Updates").
    out, inn, r, T = 48, 80, 8, 24
    wq, pq, B, x, dy = _layer(61, out, inn, r, T)
    G = O.full_gradient(x, dy)
    Wt = torch.zeros((out, inn), dtype=torch.float64, requires_grad=True)
    (torch.tensor(x, dtype=torch.float64) @ Wt.T * torch.tensor(dy, dtype=torch.float64)).sum().backward()
    assert np.allclose(G, Wt.grad.numpy(), rtol=1e-12, atol=1e-12)
    s = 0.5
    _, dB = O.loqt_backward(wq, pq, B, s, x, dy, (out, inn, r))
    P = O.nf4_dequantize_bf16(pq[0], pq[1], r).astype(np.float64)
    assert np.allclose(dB, s * P.T @ G, rtol=1e-10, atol=1e-12)


# ---- right-side variant (Section 2.1: G Q for m > n)
def _layer_right(seed, out, inn, r, T):
    W = synth.normal(seed, ("W",), (out, inn), 0.02).numpy()
    Qm = synth.orthonormal(seed, ("Q",), inn, r).numpy().T.copy()      # r x in, orthonormal rows
    B = synth.normal(seed, ("B",), (out, r), 1e-2, torch.bfloat16).to(torch.float32).numpy()
    x = synth.normal(seed, ("x",), (T, inn), 1.0, torch.bfloat16).to(torch.float32).numpy()
    dy = synth.normal(seed, ("dy",), (T, out), 1.0, torch.bfloat16).to(torch.float32).numpy()
    return O.nf4_quantize(W), O.nf4_quantize(Qm), B, x, dy


@pytest.mark.parametrize("shape", [(80, 48, 8, 12), (64, 40, 16, 7)])
def test_right_variant_equals_the_dense_layer(shape):
    out, inn, r, T = shape
    s = 0.5
    wq, qq, B, x, dy = _layer_right(71, out, inn, r, T)
    W = O.nf4_dequantize_bf16(*wq, inn).astype(np.float64)
    Q = O.nf4_dequantize_bf16(*qq, inn).astype(np.float64)
    Weff = W + s * B.astype(np.float64) @ Q
    y = O.loqt_forward_right(wq, qq, B, s, x, (out, inn, r))
    assert np.allclose(y, x.astype(np.float64) @ Weff.T, rtol=1e-11, atol=1e-12)
    # gradients by autograd on the dense parametrisation W + s B Q
    Bt = torch.tensor(B, dtype=torch.float64, requires_grad=True)
    xt = torch.tensor(x, dtype=torch.float64, requires_grad=True)
    yt = xt @ (torch.tensor(W) + s * Bt @ torch.tensor(Q)).T
    (yt * torch.tensor(dy, dtype=torch.float64)).sum().backward()
    dx, dB = O.loqt_backward_right(wq, qq, B, s, x, dy, (out, inn, r))
    assert np.allclose(dx, xt.grad.numpy(), rtol=1e-10, atol=1e-12)
    assert np.allclose(dB, Bt.grad.numpy(), rtol=1e-10, atol=1e-12)
    # the projection identity of the right side: dB = s G^W Q^T
    assert np.allclose(dB, s * O.full_gradient(x, dy) @ Q.T, rtol=1e-10, atol=1e-12)


def test_right_variant_is_the_left_variant_of_the_transposed_layer():
    # W^T = W_q^T + s Q^T B^T: a left-side layer with P = Q^T and factor B^T.  With
    # square blocks of identical scales out of reach, the check uses the dequantised
    # matrices directly: the two merged weight matrices are transposes of each other.
    out, inn, r, T = 64, 128, 8, 4
    s = 0.25
    wq, qq, B, x, dy = _layer_right(72, out, inn, r, T)
    vw = O.loqt_merge_values_right(wq, qq, B, s, (out, inn, r))
    W32 = O.nf4_dequantize(*wq, inn).astype(np.float64)
    Q = O.nf4_dequantize_bf16(*qq, inn).astype(np.float64)
    ref = (W32.T + s * Q.T @ B.astype(np.float64).T).T.astype(np.float32)
    assert np.array_equal(vw, ref)
    # B = 0 leaves the quantised weights untouched
    c, m = O.nf4_quantize(O.loqt_merge_values_right(wq, qq, np.zeros_like(B), 1.0, (out, inn, r)))
    assert np.array_equal(c, wq[0]) and np.array_equal(m, wq[1])


@pytest.mark.parametrize("shape", [(40, 100, 8), (64, 128, 16)])
def test_right_merge_equals_the_dense_sum_built_entry_by_entry(shape):
    """The right variant's merged matrix, formed without any oracle routine:
    W enters as the unrounded fp32 product M * q, Q as that product rounded to
    bf16 (torch's conversion), each entry's sum over r evaluated exactly
    (math.fsum) and rounded once to fp32.  A wrong operand precision for Q or W
    changes low-order bits of many entries and fails the bit-for-bit comparison."""
    import math

    out, inn, r = shape
    s = 0.5
    wq, qq, B, _, _ = _layer_right(73, out, inn, r, 2)
    B = (B * 3.0).astype(np.float32)      # large enough to move values across fp32 roundings
    B = O.bf16_round(B)
    lv = O.NF4_LEVELS
    bf = lambda v: float(torch.tensor(float(v), dtype=torch.float32).to(torch.bfloat16))
    Q = [[bf(np.float32(qq[1][k, i // 64]) * lv[qq[0][k, i]]) for i in range(inn)] for k in range(r)]
    ref = np.zeros((out, inn), dtype=np.float32)
    for o in range(out):
        for i in range(inn):
            w32 = float(np.float32(wq[1][o, i // 64]) * lv[wq[0][o, i]])
            # s = 0.5 and the bf16 x bf16 products are exact in float64, so fsum sees the exact terms
            ref[o, i] = np.float32(math.fsum([w32] + [s * float(B[o, k]) * Q[k][i] for k in range(r)]))
    vw = O.loqt_merge_values_right(wq, qq, B, s, (out, inn, r))
    # float64 accumulation of <= 16 terms of this size differs from the exact sum by far less than
    # half an fp32 ulp except at rounding ties; allow the two roundings to disagree on at most a few
    # entries, and then only by one fp32 ulp
    diff = vw != ref
    assert diff.mean() < 2e-3
    assert np.all(np.abs(vw[diff] - ref[diff]) <= np.spacing(np.abs(ref[diff])))
    # the same construction with Q left unrounded (fp32) is visibly different: the pin has teeth
    Q32 = np.array([[float(np.float32(qq[1][k, i // 64]) * lv[qq[0][k, i]]) for i in range(inn)] for k in range(r)])
    wrong = (O.nf4_dequantize(*wq, inn).astype(np.float64) + s * B.astype(np.float64) @ Q32).astype(np.float32)
    assert np.mean(wrong != vw) > 0.2


def test_right_compensation_is_the_least_squares_fit_and_keeps_improving():
    # B_1 = (W - deq(q(W))) Q^+ is the minimiser of || B Q - (W - Q_1) ||_F (numpy's least-squares
    # routine on the transposed system), up to the 16-bit roundings of the operands and of B
    rng = np.random.default_rng(81)
    out, inn, r = 96, 160, 16
    W = (0.02 * rng.normal(size=(out, inn))).astype(np.float32)
    Qf, _ = np.linalg.qr(rng.normal(size=(inn, r)))
    Q = Qf.T.astype(np.float32)                       # r x in, orthonormal rows
    (c1, m1), B1 = O.loqt_compensate_right(W, Q, 1)
    q0 = O.nf4_quantize(W)
    assert np.array_equal(c1, q0[0]) and np.array_equal(m1, q0[1])
    R = W.astype(np.float64) - O.nf4_dequantize(q0[0], q0[1], inn)
    Bls = np.linalg.lstsq(Q.astype(np.float64).T, R.T, rcond=None)[0].T       # min || Q^T B^T - R^T ||
    assert np.abs(B1 - Bls).max() <= 2.0 ** -7 * np.abs(Bls).max()
    # the objective falls step by step, and the fit beats plain quantisation by about the share r / in
    def err(q, B):
        return np.linalg.norm(O.nf4_dequantize(q[0], q[1], inn) + B.astype(np.float64) @ O.bf16_round(Q) - W) ** 2
    e0 = np.linalg.norm(R) ** 2
    es = [err(*O.loqt_compensate_right(W, Q, c)) for c in (1, 2, 3, 5)]
    assert es[0] < e0 and all(es[i + 1] <= es[i] * (1 + 1e-9) for i in range(3))
    assert es[0] < (1 - 0.7 * r / inn) * e0
    # weights that NF4 represents exactly need no correction
    Wr = O.nf4_dequantize(q0[0], q0[1], inn)
    (c, m), B = O.loqt_compensate_right(Wr, Q, 3)
    assert np.array_equal(c, q0[0]) and np.array_equal(m, q0[1]) and not B.any()
    # one step from a given state equals the definition written out with that B
    B0 = O.bf16_round((1e-3 * rng.normal(size=(out, r))).astype(np.float32))
    (c2, m2), _ = O.loqt_compensate_right(W, Q, 1, B0=B0)
    ref = O.nf4_quantize((W.astype(np.float64) - B0.astype(np.float64) @ O.bf16_round(Q).astype(np.float64)).astype(np.float32))
    assert np.array_equal(c2, ref[0]) and np.array_equal(m2, ref[1])
