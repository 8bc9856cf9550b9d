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


def check_merge(got_codes, got_absmax, ref_codes, ref_absmax, vw: np.ndarray, cols: int, what: str):
    """Merged codes: at most 0.01 % may differ from the oracle's, each by one
    level and only where the oracle's pre-quantisation value lies within one
    fp32 ulp (at the block scale's magnitude) of the decision boundary; scales
    within one ulp."""
    ulp = np.spacing(np.abs(ref_absmax).astype(np.float32)).astype(np.float64)
    assert np.all(np.abs(got_absmax.astype(np.float64) - ref_absmax.astype(np.float64)) <= ulp), f"{what}: absmax"
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
            boundary = mid[min(a, b)] * M
            assert abs(float(vw[r, c]) - boundary) <= 2 * float(ulp[r, c // 64]), f"{what}: not at a boundary {(r, c)}"
    return n_diff
