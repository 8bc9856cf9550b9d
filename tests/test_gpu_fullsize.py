"""GPU parity at the benchmark's full sizes (Llama-7B shapes, r = 1024,
T = 4096), in the launch configuration bench.py times, on sampled outputs the
CPU oracle computes one by one: sampled weight rows for the quantiser and the
merge, sampled token rows / output columns for y and dx, one 64-wide block of
rank rows for dB."""
import numpy as np
import pytest
import torch

from oracle import loqt_oracle as O
from paper_2405_16528_b200 import binding as L
from paper_2405_16528_b200 import synth
from tests.gpu_util import check_close, check_merge, f32, merge_error_bound

pytestmark = pytest.mark.gpu

CFG = synth.CONFIGS[4]
SHAPES = [(o, i) for _, o, i, _ in CFG.shapes()]


def _rows(q: L.NF4Tensor, idx):
    """(codes, absmax) of selected rows, in the oracle's unpacked form."""
    t = torch.as_tensor(idx, device=q.codes.device)
    return O.unpack_codes(q.codes[t].cpu().numpy()), q.absmax[t].cpu().numpy()


@pytest.mark.parametrize("out,inn", SHAPES)
def test_full_size_sampled(out, inn):
    r, T, s = CFG.r, CFG.T, 1.0
    rng = np.random.default_rng(out * 7 + inn)
    d = synth.make_layer(21, ("full", out, inn), out, inn, r, CFG.sigma_B, T, device="cuda")
    Wq, Pq = L.loqt_nf4_quantize(d["W"]), L.loqt_nf4_quantize(d["P"])
    B, x, dy = d["B"], d["x"], d["dy"]

    # ---- quantiser: sampled rows, bit for bit
    o_s = np.sort(rng.choice(out, size=64, replace=False))
    ref_c, ref_m = O.nf4_quantize(d["W"][torch.as_tensor(o_s, device="cuda")].cpu().numpy())
    got_c, got_m = _rows(Wq, o_s)
    assert np.array_equal(got_c, ref_c) and np.array_equal(got_m, ref_m)
    wq_s = (got_c, got_m)
    pq_s = _rows(Pq, o_s)

    # ---- forward: sampled tokens x sampled output columns
    y = L.loqt_linear_fwd(Wq, Pq, B, s, x)
    t_s = np.sort(rng.choice(T, size=48, replace=False))
    tt = torch.as_tensor(t_s, device="cuda")
    Bh, xh_s = f32(B), f32(x[tt])
    ref_y = O.loqt_forward(wq_s, pq_s, Bh, s, xh_s, (len(o_s), inn, r))
    check_close(f32(y[tt][:, torch.as_tensor(o_s, device="cuda")]), ref_y, f"y {out}x{inn}")

    # ---- backward: dx on sampled tokens (all columns), dB on one block of rank rows
    dx, dB = L.loqt_linear_bwd(Wq, Pq, B, s, x, dy)
    wq_all = _rows(Wq, np.arange(out))
    pq_all = _rows(Pq, np.arange(out))
    ref_dx, _ = O.loqt_backward(wq_all, pq_all, Bh, s, xh_s, f32(dy[tt]), (out, inn, r))
    check_close(f32(dx[tt]), ref_dx, f"dx {out}x{inn}")
    k0 = 64 * int(rng.integers(r // 64))
    pq_blk = (pq_all[0][:, k0 : k0 + 64].copy(), pq_all[1][:, k0 // 64 : k0 // 64 + 1].copy())
    _, ref_dB = O.loqt_backward(wq_all, pq_blk, Bh[k0 : k0 + 64], s, f32(x), f32(dy), (out, inn, 64))
    check_close(f32(dB[k0 : k0 + 64]), ref_dB, f"dB {out}x{inn}")
    del wq_all

    # ---- merge: sampled weight rows
    vw = O.loqt_merge_values(wq_s, pq_s, Bh, s, (len(o_s), inn, r))
    ref_c, ref_m = O.nf4_quantize(vw)
    L.loqt_merge_requant(Wq, Pq, B, s)
    got_c, got_m = _rows(Wq, o_s)
    bound, _ = merge_error_bound(pq_s, Bh, s, r, ref_m)
    n_diff, max_ulp = check_merge(got_c, got_m, ref_c, ref_m, vw, inn, bound, f"merge {out}x{inn}")
    print(f"full-size {out}x{inn}: merge {n_diff} of {ref_c.size} sampled codes differ, scales within {max_ulp:.1f} ulp")
