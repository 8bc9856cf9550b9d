"""Helpers shared by the GPU parity tests: conversions between the oracle's
numpy arrays and the library's device tensors, and the error metrics."""
import numpy as np
import torch

from oracle import loqt_oracle as O
from paper_2405_16528_b200 import binding as L

MAX_REL = 1e-2   # max |err| / max |ref|
MEAN_REL = 2e-3  # mean |err| / mean |ref|


def to_dev_nf4(codes: np.ndarray, absmax: np.ndarray, cols: int) -> L.NF4Tensor:
    return L.NF4Tensor(
        torch.from_numpy(O.pack_codes(codes)).cuda(), torch.from_numpy(absmax.copy()).cuda(), codes.shape[0], cols
    )


def from_dev_nf4(q: L.NF4Tensor):
    return O.unpack_codes(q.codes.cpu().numpy()), q.absmax.cpu().numpy()


def f32(t: torch.Tensor) -> np.ndarray:
    return t.detach().to(torch.float32).cpu().numpy()


def padded(t: torch.Tensor, mult: int = 8) -> torch.Tensor:
    """Device copy of a 2-D tensor whose row stride is a multiple of `mult`."""
    rows, cols = t.shape
    ld = (cols + mult - 1) // mult * mult
    buf = torch.zeros((rows, ld), dtype=t.dtype, device="cuda")
    buf[:, :cols] = t.cuda()
    return buf[:, :cols]


def check_close(got: np.ndarray, ref: np.ndarray, what: str):
    got = got.astype(np.float64)
    err = np.abs(got - ref)
    max_rel = err.max() / np.abs(ref).max()
    mean_rel = err.mean() / np.abs(ref).mean()
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    assert max_rel <= MAX_REL, f"{what}: max|err|/max|ref| = {max_rel:.3e}"
    assert mean_rel <= MEAN_REL, f"{what}: mean|err|/mean|ref| = {mean_rel:.3e}"
    return max_rel, mean_rel


def merge_error_bound(pq, B, s, r, ref_absmax):
    """Per-element bound on |v_gpu - v_oracle| for the merged fp32 value
    v = deq32(W_q) + s * sum_k P[o,k] B[k,i].

    The oracle rounds the exact sum once (half an ulp).  The tensor core adds
    the exact bf16 products into an fp32 accumulator 16 at a time; allowing one
    fp32 ulp of the running magnitude per accumulation step (and one for the
    final fused multiply-add) gives (ceil(r/16) + 1) * 2^-23 * s * sum_k |P||B|.
    Returned per element, plus one ulp of the block scale."""
    P = np.abs(O.nf4_dequantize_bf16(pq[0], pq[1], r).astype(np.float64))
    acc = (int(np.ceil(r / 16)) + 1) * 2.0 ** -23 * abs(float(s)) * (P @ np.abs(np.asarray(B, dtype=np.float64)))
    ulp = np.spacing(np.abs(ref_absmax).astype(np.float32)).astype(np.float64)
    cols = acc.shape[1]
    return acc + np.repeat(ulp, 64, axis=1)[:, :cols], ulp


def check_merge(got_codes, got_absmax, ref_codes, ref_absmax, vw, cols, bound, what):
    """Merged state against the oracle's.

    Codes, the strict clause: at most 0.01 % of them differ, each by one level,
    and only where the oracle's pre-quantisation value lies within ONE fp32 ulp
    (taken at the block scale's magnitude) of the decision boundary m_k * M.
    Block scales: within the accumulation bound of merge_error_bound().
    Returns (differing codes, largest scale difference in ulps, histogram of the
    scale differences in ulps: {0, 1, 2, 3+} -> count)."""
    rows, ld = ref_codes.shape
    nb = ld // 64
    bpad = np.zeros((rows, ld))
    bpad[:, :cols] = bound
    blk_bound = bpad.reshape(rows, nb, 64).max(axis=2)
    ulp = np.spacing(np.abs(ref_absmax).astype(np.float32)).astype(np.float64)
    dm = np.abs(got_absmax.astype(np.float64) - ref_absmax.astype(np.float64))
    dm_ulp = np.rint(dm / np.maximum(ulp, 1e-300)).astype(np.int64)
    hist = {k: int((dm_ulp == k).sum()) for k in (0, 1, 2)}
    hist["3+"] = int((dm_ulp >= 3).sum())
    assert np.all(dm <= blk_bound + ulp), f"{what}: absmax off by up to {dm_ulp.max()} ulp"
    diff = got_codes != ref_codes
    n_diff = int(diff.sum())
    assert n_diff <= max(1, int(1e-4 * ref_codes.size)), f"{what}: {n_diff} of {ref_codes.size} codes differ"
    if n_diff:
        lv = O.NF4_LEVELS.astype(np.float64)
        mid = (lv[:-1] + lv[1:]) / 2
        rr, cc = np.nonzero(diff)
        for r, c in zip(rr, cc):
            a, b = int(got_codes[r, c]), int(ref_codes[r, c])
            assert abs(a - b) == 1, f"{what}: code jump {b}->{a} at {(r, c)}"
            assert c < cols
            M = float(ref_absmax[r, c // 64])
            dist = abs(float(vw[r, c]) - mid[min(a, b)] * M)
            assert dist <= ulp[r, c // 64], (
                f"{what}: code differs at {(r, c)} where the value is {dist / ulp[r, c // 64]:.2f} ulp from the boundary")
    return n_diff, int(dm_ulp.max()), hist
