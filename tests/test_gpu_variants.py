"""GPU parity of every instantiation of the product kernel against the CPU oracle.

The library picks a tile shape per product with a cost model, so small test
shapes would only ever run the narrow single-CTA tiles, while the benchmark
sizes run 256-wide tiles, 256-row tiles and tcgen05 CTA pairs.  Here each of
the six tile shapes (columns x rows x pair) is forced in turn and the forward,
the backward and the merge are compared element by element with the oracle, on
shapes that are ragged in every dimension: out and in from the paper's MLP
widths 1376 / 2736 / 5461 (5461 is odd: a short last NF4 block, a row stride
that is not a multiple of 64), ranks 40 / 96 / 512, token counts that are not a
multiple of any tile height.  Together with the variant with and without NF4
staging this covers all twelve kernel instantiations; the library's launch
counters prove that the forced instantiation is the one that ran.
"""
import numpy as np
import pytest
import torch

from oracle import loqt_oracle as O
from paper_2405_16528_b200 import binding as L
from paper_2405_16528_b200 import synth
from tests.gpu_util import check_close, check_merge, f32, from_dev_nf4, merge_error_bound, padded, to_dev_nf4

pytestmark = pytest.mark.gpu

# (columns, rows, pair) of a tile; with nf4 in {0, 1} the twelve instantiations
TILES = [(128, 128, False), (128, 256, False), (256, 128, False), (256, 256, False), (256, 128, True), (256, 256, True)]
# (out, in, r, T)
SHAPES = [(1376, 5461, 96, 300), (5461, 1376, 40, 389), (2736, 640, 512, 200), (640, 2736, 512, 521)]


def _tile_id(t):
    return f"{t[0]}x{t[1]}{'pair' if t[2] else 'single'}"


_cache = {}


def _case(shape):
    """Inputs and oracle results of one shape (computed once, shared by all tiles)."""
    if shape in _cache:
        return _cache[shape]
    out, inn, r, T = shape
    s = 0.5
    d = synth.make_layer(50, ("variants",) + shape, out, inn, r, 1e-2, T)
    wq, pq = O.nf4_quantize(d["W"].numpy()), O.nf4_quantize(d["P"].numpy())
    host = {"wq": wq, "pq": pq, "B": f32(d["B"]), "x": f32(d["x"]), "dy": f32(d["dy"])}
    ref = {"y": O.loqt_forward(wq, pq, host["B"], s, host["x"], (out, inn, r))}
    ref["dx"], ref["dB"] = O.loqt_backward(wq, pq, host["B"], s, host["x"], host["dy"], (out, inn, r))
    ref["G"] = O.full_gradient(host["x"], host["dy"])
    ref["vw"] = O.loqt_merge_values(wq, pq, host["B"], s, (out, inn, r))
    ref["merged"] = O.nf4_quantize(ref["vw"])
    ref["bound"], _ = merge_error_bound(pq, host["B"], s, r, ref["merged"][1])
    _cache[shape] = (s, d, host, ref)
    return _cache[shape]


@pytest.fixture
def forced_tile(request):
    bn, rows, pair = request.param
    L.loqt_set_tile_override(bn, rows, pair)
    yield request.param
    L.loqt_set_tile_override(0)


def _counts(tile):
    bn, rows, pair = tile
    return L.loqt_variant_launches(bn, rows, pair, True), L.loqt_variant_launches(bn, rows, pair, False)


@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "x".join(map(str, s)))
@pytest.mark.parametrize("forced_tile", TILES, ids=_tile_id, indirect=True)
def test_forward_backward_merge_with_forced_tile(forced_tile, shape):
    out, inn, r, T = shape
    s, d, host, ref = _case(shape)
    Wq, Pq = to_dev_nf4(*host["wq"], inn), to_dev_nf4(*host["pq"], r)
    B, x, dy = padded(d["B"]), padded(d["x"]), padded(d["dy"])

    nf4_0, bf16_0 = _counts(forced_tile)
    y = padded(torch.zeros((T, out), dtype=torch.bfloat16))
    ws = L.new_workspace(L.loqt_workspace_bytes(L.LOQT_OP_BWD, out, inn, r, T))
    L.loqt_linear_fwd(Wq, Pq, B, s, x, y=y, ws=ws)
    L.loqt_device_status(ws)
    nf4_1, bf16_1 = _counts(forced_tile)
    # u = s x B^T ran the variant without NF4 staging, y the one with it
    assert nf4_1 == nf4_0 + 1 and bf16_1 == bf16_0 + 1, "the forced instantiation did not run"
    check_close(f32(y), ref["y"], f"y {shape} {_tile_id(forced_tile)}")

    dx = padded(torch.zeros((T, inn), dtype=torch.bfloat16))
    dB = torch.full((r, inn), 3.0, dtype=torch.float32, device="cuda")
    L.loqt_linear_bwd(Wq, Pq, B, s, x, dy, dx=dx, dB=dB, ws=ws)
    L.loqt_device_status(ws)
    nf4_2, bf16_2 = _counts(forced_tile)
    # dx dequantises W_q in its main loop; v = dy P-hat reads the factor staged as bf16 (the variant without NF4 staging)
    assert nf4_2 == nf4_1 + 1 and bf16_2 >= bf16_1 + 1, "v and dx did not run the forced instantiation"
    check_close(f32(dx), ref["dx"], f"dx {shape} {_tile_id(forced_tile)}")
    check_close(f32(dB), ref["dB"], f"dB {shape} {_tile_id(forced_tile)}")

    G = L.loqt_full_gradient(x, dy)
    check_close(f32(G), ref["G"], f"G^W {shape} {_tile_id(forced_tile)}")

    # the merge runs single 128-row tiles of either width; other forced shapes leave it on its own choice
    L.loqt_merge_requant(Wq, Pq, B, s)
    got_c, got_m = from_dev_nf4(Wq)
    check_merge(got_c, got_m, ref["merged"][0], ref["merged"][1], ref["vw"], inn, ref["bound"],
                f"merge {shape} {_tile_id(forced_tile)}")
    assert np.all(got_c[:, inn:] == 7)


RIGHT_SHAPE = (2736, 1376, 96, 300)


@pytest.mark.parametrize("forced_tile", TILES, ids=_tile_id, indirect=True)
def test_right_variant_with_forced_tile(forced_tile):
    out, inn, r, T = RIGHT_SHAPE
    s = 0.5
    key = ("right",) + RIGHT_SHAPE
    if key not in _cache:
        W = synth.normal(51, ("W", out, inn), (out, inn), 0.02)
        Q = synth.orthonormal(51, ("Q", inn, r), inn, r).T.contiguous()
        B = synth.normal(51, ("B", out, r), (out, r), 1e-2, torch.bfloat16)
        x = synth.normal(51, ("x", T, inn), (T, inn), 1.0, torch.bfloat16)
        dy = synth.normal(51, ("dy", T, out), (T, out), 1.0, torch.bfloat16)
        wq, qq = O.nf4_quantize(W.numpy()), O.nf4_quantize(Q.numpy())
        ref_y = O.loqt_forward_right(wq, qq, f32(B), s, f32(x), (out, inn, r))
        ref_dx, ref_dB = O.loqt_backward_right(wq, qq, f32(B), s, f32(x), f32(dy), (out, inn, r))
        _cache[key] = (wq, qq, B, x, dy, ref_y, ref_dx, ref_dB)
    wq, qq, B, x, dy, ref_y, ref_dx, ref_dB = _cache[key]
    Wq, Qq = to_dev_nf4(*wq, inn), to_dev_nf4(*qq, inn)
    Bd, xd, dyd = padded(B), padded(x), padded(dy)
    nf4_0, bf16_0 = _counts(forced_tile)
    y = L.loqt_linear_fwd_right(Wq, Qq, Bd, s, xd)
    nf4_1, bf16_1 = _counts(forced_tile)
    # y dequantises W_q inside the product; u multiplies the staged bf16 copy of the factor
    assert nf4_1 == nf4_0 + 1 and bf16_1 >= bf16_0 + 1, "u and y did not run the forced instantiation"
    check_close(f32(y), ref_y, f"right y {_tile_id(forced_tile)}")
    dx, dB = L.loqt_linear_bwd_right(Wq, Qq, Bd, s, xd, dyd)
    check_close(f32(dx), ref_dx, f"right dx {_tile_id(forced_tile)}")
    check_close(f32(dB), ref_dB, f"right dB {_tile_id(forced_tile)}")


def test_override_arguments():
    with pytest.raises(L.LoqtError, match="invalid"):
        L.loqt_set_tile_override(192, 128, False)
    with pytest.raises(L.LoqtError, match="unsupported"):
        L.loqt_set_tile_override(128, 128, True)
    L.loqt_set_tile_override(0)
