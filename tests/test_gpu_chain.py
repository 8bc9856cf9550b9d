"""The initialisation chain of Algorithm 1 / Algorithm 2 through the library's entry points, end to end:
full-rank gradient -> projection -> error-compensated initialisation -> forward, one optimiser step and a
merge.  A basis of a subspace is not unique and the NF4 error of P depends on the basis, so the library's
(W_q, P_q, B) are not compared entry by entry with the oracle's; what is compared is what the method
needs of them: how well W_q + P B fits W, against the oracle's own chain on the same inputs."""
import numpy as np
import pytest
import torch

from oracle import loqt_oracle as O
from paper_2405_16528_b200 import binding as L
from paper_2405_16528_b200 import synth
from tests.gpu_util import check_close, f32, from_dev_nf4, padded

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("shape", [(384, 640, 64, 300), (640, 1376, 96, 260)])
def test_initialise_then_train_one_step_and_merge(shape):
    out, inn, r, T = shape
    W = synth.normal(70, ("W", out, inn), (out, inn), 0.02)
    x = synth.normal(70, ("x", T, inn), (T, inn), 1.0, torch.bfloat16)
    dy = synth.normal(70, ("dy", T, out), (T, out), 1.0, torch.bfloat16)
    Om = synth.normal(70, ("Omega", inn, r), (inn, r), 1.0, torch.bfloat16)
    Wd = torch.zeros((out, (inn + 3) // 4 * 4), dtype=torch.float32, device="cuda")[:, :inn]
    Wd.copy_(W)
    xd, dyd, Omd = padded(x), padded(dy), padded(Om)

    # library: G^W = dy^T x, P from two rounds of subspace iteration, five compensation steps
    G = L.loqt_full_gradient(xd, dyd)
    P = L.loqt_projection(G, Omd, 2)
    Wq, Pq, B = L.loqt_compensated_init(Wd, P, 5)

    # oracle, same inputs
    Go = O.full_gradient(f32(x), f32(dy))
    check_close(f32(G), Go, "G^W")
    Po = O.subspace_iteration(O.bf16_round(Go.astype(np.float32)).astype(np.float64), f32(Om).astype(np.float64), 2)
    assert O.subspace_sines(Po, f32(P).astype(np.float64)).max() < 1e-3
    (oc, om), oB = O.loqt_compensate(W.numpy(), Po.astype(np.float32), 5)

    def fit(codes, absmax, Pm, Bm):
        Pb = O.bf16_round(np.asarray(Pm, dtype=np.float32)).astype(np.float64)
        return np.linalg.norm(O.nf4_dequantize(codes, absmax, inn) + Pb @ Bm.astype(np.float64) - W.numpy()) ** 2

    c, m = from_dev_nf4(Wq)
    e_lib, e_ref = fit(c, m, f32(P), f32(B)), fit(oc, om, Po, oB)
    e_plain = np.linalg.norm(O.nf4_dequantize(*O.nf4_quantize(W.numpy()), inn) - W.numpy()) ** 2
    assert abs(e_lib - e_ref) <= 0.02 * e_ref and e_lib < (1 - 0.7 * r / out) * e_plain

    # the initialised layer through forward and backward against the oracle on the library's own state
    pq = from_dev_nf4(Pq)
    y = L.loqt_linear_fwd(Wq, Pq, B, 0.5, xd)
    check_close(f32(y), O.loqt_forward((c, m), pq, f32(B), 0.5, f32(x), (out, inn, r)), "y")
    dx, dB = L.loqt_linear_bwd(Wq, Pq, B, 0.5, xd, dyd)
    odx, odB = O.loqt_backward((c, m), pq, f32(B), 0.5, f32(x), f32(dy), (out, inn, r))
    check_close(f32(dx), odx, "dx")
    check_close(f32(dB), odB, "dB")

    # one Adam step on B, then the merge: the merged weights equal the oracle's merge of the same state
    mom, var = torch.zeros_like(B), torch.zeros_like(B)
    B0 = f32(B).copy()
    L.loqt_adam_step(B, dB, mom, var, 1, 1e-3)
    oBn, _, _ = O.adam_step(B0, f32(dB), np.zeros_like(B0), np.zeros_like(B0), 1, np.float32(1e-3),
                            float(np.float32(0.9)), float(np.float32(0.999)), float(np.float32(1e-8)))
    assert np.mean(f32(B) != oBn) < 2e-2 and np.abs(f32(B) - oBn).max() <= 2.0 ** -7 * np.abs(oBn).max()
    mc, mm = O.loqt_merge_requant((c, m), pq, f32(B), 0.5, (out, inn, r))
    L.loqt_merge_requant(Wq, Pq, B, 0.5)
    gc, gm = from_dev_nf4(Wq)
    assert (gc != mc).mean() <= 1e-4 and np.abs(gm - mm).max() <= 2.0 ** -20 * np.abs(mm).max()
