"""GPU parity: loqt_projection (Algorithm 2, the SVD lines: the projection P from
the full-rank gradient, found by randomised subspace iteration) against the CPU
oracle on the same seeded inputs, through the C ABI.

A basis of a subspace is not unique, so what is compared is the subspace: the
sines of the principal angles between the library's P and the oracle's.  The
library rounds G to bf16 on entry (stated in its header), so the oracle is
given the bf16 values; the test matrix Omega is bf16 on both sides."""
import numpy as np
import pytest
import torch

from oracle import loqt_oracle as O
from paper_2405_16528_b200 import binding as L
from paper_2405_16528_b200 import synth
from tests.gpu_util import f32

pytestmark = pytest.mark.gpu

# (out, in, r, iters): ragged tiles in every dimension, r not a multiple of 64,
# tall and wide matrices, the paper's 1B MLP width
CASES = [(256, 384, 32, 2), (640, 1376, 96, 2), (1376, 512, 40, 1), (200, 136, 24, 3), (768, 5461, 128, 1),
         (2048, 2048, 512, 2)]


def _inputs(seed, out, inn, r, tail=0.5, noise=1e-3):
    G = synth.lowrank_gradient(seed, ("G", out, inn, r), out, inn, r, tail, noise)
    Om = synth.normal(seed, ("Omega", inn, r), (inn, r), 1.0, torch.bfloat16)
    ld = (inn + 3) // 4 * 4
    Gd = torch.zeros((out, ld), dtype=torch.float32, device="cuda")[:, :inn]
    Gd.copy_(G)
    ldo = (r + 7) // 8 * 8
    Od = torch.zeros((inn, ldo), dtype=torch.bfloat16, device="cuda")[:, :r]
    Od.copy_(Om)
    Gb = O.bf16_round(G.numpy()).astype(np.float64)   # what the library's products see
    return Gb, f32(Om).astype(np.float64), Gd, Od


def _tolerance(Gb, Om, r, iters):
    """Largest principal-angle sine allowed between the library's subspace and the
    oracle's.  The products accumulate in fp32 (about 2^-22 relative to the norm of
    a row of the product after a few thousand terms); orthonormalising the first
    iterate Y0 = G Omega turns that into an angle error of 2^-22 cond(Y0), which
    every later iteration multiplies by at most rho = (sigma_(r+1) / sigma_r)^2;
    each later product adds 2^-17 sigma_1 / sigma_r (the bf16 pair carrying the
    basis) plus its own fp32 accumulation.  A factor 8 covers the constants
    (the errors add up over the r columns roughly like sqrt(r))."""
    sv = np.linalg.svd(Gb, compute_uv=False)
    cond0 = np.linalg.cond(Gb @ Om)
    rho = (sv[r] / sv[r - 1]) ** 2 if r < len(sv) else 0.0
    later = (2.0 ** -17 + 2.0 ** -22) * sv[0] / sv[r - 1] if iters > 0 else 0.0
    return 8.0 * (2.0 ** -22 * cond0 * rho ** iters + later), cond0


@pytest.mark.parametrize("case", CASES)
def test_projection_matches_the_oracle_subspace(case):
    out, inn, r, iters = case
    Gb, Om, Gd, Od = _inputs(50, out, inn, r)
    ws = L.new_workspace(L.loqt_workspace_bytes(L.LOQT_OP_PROJECTION, out, inn, r, 0))
    P = L.loqt_projection(Gd, Od, iters, ws=ws)
    L.loqt_device_status(ws)
    P = f32(P).astype(np.float64)
    assert P.shape == (out, r) and np.isfinite(P).all()
    # orthonormal columns (fp32 storage: each entry carries a relative 2^-24)
    assert np.abs(P.T @ P - np.eye(r)).max() < 2e-6
    Q = O.subspace_iteration(Gb, Om, iters)
    sines = O.subspace_sines(Q, P)
    tol, cond0 = _tolerance(Gb, Om, r, iters)
    print(f"projection {case}: max sine {sines.max():.3e} (tolerance {tol:.3e}, cond(G Omega) = {cond0:.1f})")
    assert sines.max() <= tol
    # and it serves the method as the oracle's basis does: the energy of G it captures, ||P^T G||_F^2, is the same
    # (below the optimum of the exact singular subspace by what the iteration count leaves)
    cap, cap_ref = np.linalg.norm(P.T @ Gb) ** 2, np.linalg.norm(Q.T @ Gb) ** 2
    opt = np.linalg.norm(O.top_r_left_subspace(Gb, r).T @ Gb) ** 2
    assert abs(cap - cap_ref) <= 1e-5 * cap_ref and cap <= opt * (1 + 1e-6)


def test_full_size_7b_attention_shape():
    """The projection at the benchmark's size (4096 x 4096, r = 1024: sixteen 64-column panels, eight
    128-wide tile rows, every level of the inversion by doubling), one round, against the oracle's iterate.
    The spectrum is the planted one (2 .. 1, then 0.5 .. 0.05), so the tolerance is formed from those values
    instead of a 4096 x 4096 SVD."""
    out, inn, r, iters = 4096, 4096, 1024, 1
    Gb, Om, Gd, Od = _inputs(53, out, inn, r)
    ws = L.new_workspace(L.loqt_workspace_bytes(L.LOQT_OP_PROJECTION, out, inn, r, 0))
    P = L.loqt_projection(Gd, Od, iters, ws=ws)
    L.loqt_device_status(ws)
    P = f32(P).astype(np.float64)
    assert np.isfinite(P).all() and np.abs(P.T @ P - np.eye(r)).max() < 2e-6
    Q = O.subspace_iteration(Gb, Om, iters)
    sines = O.subspace_sines(Q, P)
    cond0 = np.linalg.cond(Gb @ Om)
    tol = 8.0 * (2.0 ** -22 * cond0 * 0.25 ** iters + (2.0 ** -17 + 2.0 ** -22) * 2.0)
    print(f"projection {(out, inn, r, iters)}: max sine {sines.max():.3e} (tolerance {tol:.3e}, cond(G Omega) = {cond0:.1f})")
    assert sines.max() <= tol
    cap, cap_ref = np.linalg.norm(P.T @ Gb) ** 2, np.linalg.norm(Q.T @ Gb) ** 2
    assert abs(cap - cap_ref) <= 1e-5 * cap_ref


def test_converges_to_the_definition():
    # a wide spectral gap (tail 0.2): four rounds leave (0.2)^9 of the starting angle
    out, inn, r = 512, 640, 64
    Gb, Om, Gd, Od = _inputs(51, out, inn, r, tail=0.2, noise=0.0)
    P = f32(L.loqt_projection(Gd, Od, 4)).astype(np.float64)
    U = O.top_r_left_subspace(Gb, r)
    assert O.subspace_sines(U, P).max() < 1e-4


def test_reproducible_and_rank_deficient_input_is_reported():
    out, inn, r = 384, 320, 48
    Gb, Om, Gd, Od = _inputs(52, out, inn, r)
    ws = L.new_workspace(L.loqt_workspace_bytes(L.LOQT_OP_PROJECTION, out, inn, r, 0))
    P1 = L.loqt_projection(Gd, Od, 2, ws=ws).clone()
    P2 = L.loqt_projection(Gd, Od, 2, ws=ws)
    assert torch.equal(P1, P2)
    L.loqt_device_status(ws)
    # a zero gradient has no subspace to find: the factorisation meets a zero pivot and says so
    Gd.zero_()
    L.loqt_projection(Gd, Od, 0, ws=ws)
    with pytest.raises(L.LoqtError, match="rank deficient"):
        L.loqt_device_status(ws)
    ws.zero_()
    # the context is still usable
    Gd.copy_(torch.from_numpy(Gb.astype(np.float32)))
    P3 = L.loqt_projection(Gd, Od, 2, ws=ws)
    L.loqt_device_status(ws)
    assert torch.equal(P1, P3)


def test_argument_checks():
    Gd = torch.zeros((64, 64), dtype=torch.float32, device="cuda")
    Od = torch.zeros((64, 72), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(L.LoqtError, match="invalid argument"):
        L.loqt_projection(Gd, Od, 1)          # r = 72 > min(out, in)
    with pytest.raises(L.LoqtError, match="invalid argument"):
        L.loqt_projection(Gd, Od[:, :32], 17)  # too many iterations
    with pytest.raises(L.LoqtError, match="workspace"):
        L.loqt_projection(Gd, Od[:, :32], 1, ws=L.new_workspace(512))


@pytest.mark.parametrize("case", [(1376, 512, 40, 1), (640, 256, 96, 2), (2736, 1024, 256, 1)])
def test_right_side_projection_matches_the_oracle_subspace(case):
    """loqt_projection_right: the basis of the leading right singular subspace, stored r x in as the
    right-side variant's factor Q is, against the oracle's iterate on the same Omega (out x r)."""
    out, inn, r, iters = case
    G = synth.lowrank_gradient(54, ("G", out, inn, r), out, inn, r)
    Om = synth.normal(54, ("Omega", out, r), (out, r), 1.0, torch.bfloat16)
    Gd = torch.zeros((out, (inn + 3) // 4 * 4), dtype=torch.float32, device="cuda")[:, :inn]
    Gd.copy_(G)
    Od = torch.zeros((out, (r + 7) // 8 * 8), dtype=torch.bfloat16, device="cuda")[:, :r]
    Od.copy_(Om)
    Gb, Omf = O.bf16_round(G.numpy()).astype(np.float64), f32(Om).astype(np.float64)
    ws = L.new_workspace(L.loqt_workspace_bytes(L.LOQT_OP_PROJECTION, out, inn, r, 0))
    Q = L.loqt_projection_right(Gd, Od, iters, ws=ws)
    L.loqt_device_status(ws)
    Q = f32(Q).astype(np.float64)
    assert Q.shape == (r, inn) and np.isfinite(Q).all()
    assert np.abs(Q @ Q.T - np.eye(r)).max() < 2e-6
    Qo = O.subspace_iteration_right(Gb, Omf, iters)
    sines = O.subspace_sines(Qo.T, Q.T)
    tol, cond0 = _tolerance(Gb.T, Omf, r, iters)
    print(f"right projection {case}: max sine {sines.max():.3e} (tolerance {tol:.3e}, cond(G^T Omega) = {cond0:.1f})")
    assert sines.max() <= tol
    cap, cap_ref = np.linalg.norm(Gb @ Q.T) ** 2, np.linalg.norm(Gb @ Qo.T) ** 2
    assert abs(cap - cap_ref) <= 1e-5 * cap_ref
