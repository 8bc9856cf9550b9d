"""The workspace-free forward, loqt_linear_fwd_static, against loqt_linear_fwd.

Who needs it: callers that are handed device tensors but may not allocate any
themselves - a plug-in inside a host framework that owns the allocator, code in
a serving loop where cudaMalloc's implicit device synchronisation is not
acceptable, a bare C program with no allocator at all.  For them the library
keeps the forward's scratch in a fixed 8 MiB array of its own.

This file is named so that pytest collects it last.  It calls the entry point
through the C ABI twice in a row with different inputs (the shared array still
holds the first call's intermediate when the second starts) and compares each
result with the ordinary entry point's on the same inputs, and with the CPU
oracle's forward.
"""
import numpy as np
import pytest
import torch

from oracle import loqt_oracle as O
from paper_2405_16528_b200 import binding as L
from paper_2405_16528_b200 import synth
from tests.gpu_util import MAX_REL, MEAN_REL, check_close, f32, from_dev_nf4

pytestmark = pytest.mark.gpu

STATIC_MAX = 8 * 1024 * 1024


def _layer(seed, out, inn, r, T):
    d = synth.make_layer(seed, "static", out, inn, r, 1e-2, T, device="cuda")
    return L.loqt_nf4_quantize(d["W"]), L.loqt_nf4_quantize(d["P"]), d["B"], d["x"]


def _compare(got, ref):
    g, r = got.float(), ref.float()
    err = (g - r).abs()
    assert torch.isfinite(g).all()
    assert (err.max() / r.abs().max()).item() <= MAX_REL
    assert (err.mean() / r.abs().mean()).item() <= MEAN_REL


def test_static_forward_matches_workspace_forward_twice():
    out, inn, r, T = 384, 320, 64, 200
    for call, (seed, s) in enumerate([(31, 1.0), (32, 0.5)]):
        Wq, Pq, B, x = _layer(seed, out, inn, r, T)
        ref = L.loqt_linear_fwd(Wq, Pq, B, s, x)
        y = torch.full((T, out), float("nan"), dtype=torch.bfloat16, device="cuda")
        if call == 0:
            # the first call on a device looks up the scratch array's address; let the context settle
            # before the free-memory readings below
            L.loqt_linear_fwd_static(Wq, Pq, B, s, x, y)
            y.fill_(float("nan"))
        torch.cuda.synchronize()
        before = torch.cuda.memory_allocated()
        free_before, _ = torch.cuda.mem_get_info()
        L.loqt_linear_fwd_static(Wq, Pq, B, s, x, y)
        torch.cuda.synchronize()
        free_after, _ = torch.cuda.mem_get_info()
        assert torch.cuda.memory_allocated() == before, "the static entry point must not allocate through torch"
        # the driver's own count of free device memory sees an allocation made inside the library too
        assert free_after >= free_before, f"device memory shrank by {free_before - free_after} bytes during the call"
        _compare(y, ref)
        assert torch.equal(y, ref), f"call {call}: same kernels, same inputs, different bits"
        oracle_y = O.loqt_forward(from_dev_nf4(Wq), from_dev_nf4(Pq), f32(B), s, f32(x), (out, inn, r))
        check_close(f32(y), oracle_y, f"static forward, call {call}")


def test_static_forward_rejects_oversized_problems():
    out, inn, r = 256, 256, 64
    Wq, Pq, B, x = _layer(33, out, inn, r, 8)
    T_big = STATIC_MAX // (64 * 2) + 1
    xb = torch.zeros((T_big, inn), dtype=torch.bfloat16, device="cuda")
    yb = torch.zeros((T_big, out), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(L.LoqtError, match="workspace"):
        L.loqt_linear_fwd_static(Wq, Pq, B, 1.0, xb, yb)
    # exactly at the limit is accepted
    T_ok = STATIC_MAX // (64 * 2)
    L.loqt_linear_fwd_static(Wq, Pq, B, 1.0, xb[:T_ok], yb[:T_ok])
    ref = L.loqt_linear_fwd(Wq, Pq, B, 1.0, xb[:T_ok])
    assert torch.equal(yb[:T_ok], ref)
