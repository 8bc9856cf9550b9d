"""ctypes binding of libloqt.so: argument marshalling only.

Every function here has the name and the argument order of the C entry point it
wraps (include/loqt.h); torch supplies device memory and the current stream,
all arithmetic runs in the library's CUDA kernels.  There is no fallback: if
the library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libloqt.so")

LOQT_OP_FWD, LOQT_OP_BWD, LOQT_OP_MERGE, LOQT_OP_MERGE_SPLIT, LOQT_OP_COMPENSATE, LOQT_OP_FULL_GRADIENT = 0, 1, 2, 3, 4, 5
LOQT_OP_FWD_RIGHT, LOQT_OP_BWD_RIGHT, LOQT_OP_MERGE_RIGHT, LOQT_OP_PROJECTION, LOQT_OP_COMPENSATE_RIGHT = 6, 7, 8, 9, 10
BLOCK = 64

EXPORTS = (
    "loqt_nf4_quantize", "loqt_nf4_dequantize", "loqt_linear_fwd", "loqt_linear_bwd",
    "loqt_merge_requant", "loqt_merge_requant_many", "loqt_merge_requant_split", "loqt_nf4_requantize",
    "loqt_compensated_init", "loqt_full_gradient", "loqt_adam_step",
    "loqt_linear_fwd_right", "loqt_linear_bwd_right", "loqt_merge_requant_right", "loqt_linear_fwd_static", "loqt_workspace_bytes",
    "loqt_device_status", "loqt_launch_count", "loqt_status_string",
    "loqt_set_tile_override", "loqt_variant_launches", "loqt_selftest_wait_timeout",
    "loqt_scales_workspace_bytes", "loqt_scales_double_quantize", "loqt_scales_double_dequantize",
    "loqt_nf4_dequantize_dq", "loqt_linear_fwd_dq", "loqt_linear_bwd_dq", "loqt_adam8_step", "loqt_projection", "loqt_projection_right", "loqt_compensated_init_right",
)


class LoqtError(RuntimeError):
    pass


class loqt_adam_params(ctypes.Structure):
    _fields_ = [
        ("lr", ctypes.c_float), ("beta1", ctypes.c_float), ("beta2", ctypes.c_float), ("eps", ctypes.c_float),
        ("weight_decay", ctypes.c_float), ("step", ctypes.c_int32),
    ]


class loqt_nf4_mat(ctypes.Structure):
    _fields_ = [
        ("codes", ctypes.c_void_p),
        ("absmax", ctypes.c_void_p),
        ("rows", ctypes.c_int32),
        ("cols", ctypes.c_int32),
        ("ld", ctypes.c_int32),
        ("block", ctypes.c_int32),
    ]


class loqt_adam8_state(ctypes.Structure):
    _fields_ = [("m8", ctypes.c_void_p), ("m_absmax", ctypes.c_void_p), ("v8", ctypes.c_void_p), ("v_absmax", ctypes.c_void_p)]


class loqt_dq_scales(ctypes.Structure):
    _fields_ = [("codes8", ctypes.c_void_p), ("c1", ctypes.c_void_p), ("offset", ctypes.c_void_p), ("n", ctypes.c_int64)]


_lib = None


def lib():
    """Loads libloqt.so (once).  Raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise LoqtError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2405_16528_b200.build`; "
            "there is no CPU or PyTorch fallback"
        )
    L = ctypes.CDLL(LIB_PATH)
    vp, i64, i32, f32, sz = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32, ctypes.c_float, ctypes.c_size_t
    M = loqt_nf4_mat
    L.loqt_nf4_quantize.argtypes = [vp, i64, M, vp]
    L.loqt_nf4_dequantize.argtypes = [M, vp, i64, ctypes.c_int, vp]
    L.loqt_linear_fwd.argtypes = [M, M, vp, i64, f32, vp, i64, i32, vp, i64, vp, sz, vp]
    L.loqt_linear_bwd.argtypes = [M, M, vp, i64, f32, vp, i64, vp, i64, i32, vp, i64, vp, i64, ctypes.c_int, vp, sz, vp]
    L.loqt_linear_fwd_static.argtypes = [M, M, vp, i64, f32, vp, i64, i32, vp, i64, ctypes.c_int, vp]
    L.loqt_linear_fwd_static.restype = ctypes.c_int
    L.loqt_merge_requant.argtypes = [M, M, vp, i64, f32, vp, sz, vp]
    L.loqt_merge_requant_split.argtypes = [M, M, vp, i64, f32, vp, sz, vp]
    L.loqt_nf4_requantize.argtypes = [vp, i64, f32, M, vp]
    L.loqt_compensated_init.argtypes = [vp, i64, vp, i64, i32, M, M, vp, i64, vp, sz, vp]
    L.loqt_compensated_init.restype = ctypes.c_int
    L.loqt_compensated_init_right.argtypes = L.loqt_compensated_init.argtypes
    L.loqt_compensated_init_right.restype = ctypes.c_int
    L.loqt_linear_fwd_right.argtypes = L.loqt_linear_fwd.argtypes
    L.loqt_linear_bwd_right.argtypes = L.loqt_linear_bwd.argtypes
    L.loqt_merge_requant_right.argtypes = L.loqt_merge_requant.argtypes
    for name in ("loqt_linear_fwd_right", "loqt_linear_bwd_right", "loqt_merge_requant_right"):
        getattr(L, name).restype = ctypes.c_int
    L.loqt_full_gradient.argtypes = [vp, i64, vp, i64, i32, i32, i32, vp, i64, ctypes.c_int, vp, sz, vp]
    L.loqt_full_gradient.restype = ctypes.c_int
    L.loqt_projection.argtypes = [vp, i64, i32, i32, i32, vp, i64, i32, vp, i64, vp, sz, vp]
    L.loqt_projection.restype = ctypes.c_int
    L.loqt_projection_right.argtypes = L.loqt_projection.argtypes
    L.loqt_projection_right.restype = ctypes.c_int
    L.loqt_adam_step.argtypes = [vp, i64, vp, i64, vp, vp, i64, i32, i32, loqt_adam_params, vp]
    L.loqt_adam_step.restype = ctypes.c_int
    L.loqt_merge_requant_many.argtypes = [i32, ctypes.POINTER(M), ctypes.POINTER(M), ctypes.POINTER(vp), ctypes.POINTER(i64), f32, vp, sz, vp]
    L.loqt_workspace_bytes.argtypes = [ctypes.c_int, i32, i32, i32, i32]
    L.loqt_workspace_bytes.restype = sz
    L.loqt_device_status.argtypes = [vp, vp]
    L.loqt_launch_count.argtypes = []
    L.loqt_launch_count.restype = ctypes.c_uint64
    L.loqt_set_tile_override.argtypes = [i32, i32, i32]
    L.loqt_set_tile_override.restype = ctypes.c_int
    L.loqt_variant_launches.argtypes = [i32, i32, i32, i32]
    L.loqt_variant_launches.restype = ctypes.c_uint64
    L.loqt_selftest_wait_timeout.argtypes = [vp, sz, ctypes.c_uint32, vp]
    L.loqt_selftest_wait_timeout.restype = ctypes.c_int
    D = loqt_dq_scales
    L.loqt_scales_workspace_bytes.argtypes = []
    L.loqt_scales_workspace_bytes.restype = sz
    L.loqt_scales_double_quantize.argtypes = [vp, D, vp, sz, vp]
    L.loqt_scales_double_dequantize.argtypes = [D, vp, vp]
    L.loqt_nf4_dequantize_dq.argtypes = [M, D, vp, i64, ctypes.c_int, vp]
    L.loqt_linear_fwd_dq.argtypes = [M, D, M, D, vp, i64, f32, vp, i64, i32, vp, i64, vp, sz, vp]
    L.loqt_linear_bwd_dq.argtypes = [M, D, M, D, vp, i64, f32, vp, i64, vp, i64, i32, vp, i64, vp, i64, ctypes.c_int, vp, sz, vp]
    for name in ("loqt_scales_double_quantize", "loqt_scales_double_dequantize", "loqt_nf4_dequantize_dq", "loqt_linear_fwd_dq",
                 "loqt_linear_bwd_dq"):
        getattr(L, name).restype = ctypes.c_int
    L.loqt_adam8_step.argtypes = [vp, i64, vp, i64, loqt_adam8_state, i32, i32, loqt_adam_params, vp]
    L.loqt_adam8_step.restype = ctypes.c_int
    L.loqt_status_string.argtypes = [ctypes.c_int]
    L.loqt_status_string.restype = ctypes.c_char_p
    for name in ("loqt_nf4_quantize", "loqt_nf4_dequantize", "loqt_linear_fwd", "loqt_linear_bwd",
                 "loqt_merge_requant", "loqt_merge_requant_many", "loqt_merge_requant_split", "loqt_nf4_requantize",
                 "loqt_device_status"):
        getattr(L, name).restype = ctypes.c_int
    _lib = L
    return L


def _check(st: int, what: str):
    if st != 0:
        raise LoqtError(f"{what} failed: {lib().loqt_status_string(st).decode()} (status {st})")


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _dev(t: torch.Tensor, dtype=None) -> int:
    if not t.is_cuda:
        raise LoqtError("the LoQT library works on CUDA tensors only")
    if dtype is not None and t.dtype != dtype:
        raise LoqtError(f"expected {dtype}, got {t.dtype}")
    if t.dim() == 2 and t.stride(1) != 1:
        raise LoqtError("matrices must be row-major with unit inner stride")
    return t.data_ptr()


@dataclass
class NF4Tensor:
    """Device storage of one NF4 matrix in the library's layout."""
    codes: torch.Tensor   # uint8 [rows, ld/2]
    absmax: torch.Tensor  # fp32  [rows, ld/64]
    rows: int
    cols: int

    @property
    def ld(self) -> int:
        return self.codes.shape[1] * 2

    def view(self) -> loqt_nf4_mat:
        return loqt_nf4_mat(self.codes.data_ptr(), self.absmax.data_ptr(), self.rows, self.cols, self.ld, BLOCK)

    @staticmethod
    def empty(rows: int, cols: int, device="cuda") -> "NF4Tensor":
        ld = (cols + BLOCK - 1) // BLOCK * BLOCK
        return NF4Tensor(
            torch.empty((rows, ld // 2), dtype=torch.uint8, device=device),
            torch.empty((rows, ld // BLOCK), dtype=torch.float32, device=device),
            rows, cols,
        )

    def clone(self) -> "NF4Tensor":
        return NF4Tensor(self.codes.clone(), self.absmax.clone(), self.rows, self.cols)

    def nbytes(self) -> int:
        return self.codes.numel() + 4 * self.absmax.numel()


def loqt_workspace_bytes(op: int, out: int, inn: int, r: int, T: int) -> int:
    return int(lib().loqt_workspace_bytes(op, out, inn, r, T))


def new_workspace(nbytes: int, device="cuda") -> torch.Tensor:
    """Zeroed uint8 workspace (the first word is the sticky device status)."""
    return torch.zeros((max(int(nbytes), 256),), dtype=torch.uint8, device=device)


def loqt_nf4_quantize(src: torch.Tensor, dst: NF4Tensor | None = None) -> NF4Tensor:
    rows, cols = src.shape
    dst = dst if dst is not None else NF4Tensor.empty(rows, cols, src.device)
    _check(lib().loqt_nf4_quantize(_dev(src, torch.float32), src.stride(0), dst.view(), _stream()), "loqt_nf4_quantize")
    return dst


def loqt_nf4_dequantize(src: NF4Tensor, dtype=torch.float32, dst: torch.Tensor | None = None) -> torch.Tensor:
    if dst is None:
        dst = torch.empty((src.rows, src.cols), dtype=dtype, device=src.codes.device)
    is_bf16 = {torch.float32: 0, torch.bfloat16: 1}[dst.dtype]
    _check(lib().loqt_nf4_dequantize(src.view(), _dev(dst), dst.stride(0), is_bf16, _stream()), "loqt_nf4_dequantize")
    return dst


def loqt_linear_fwd(Wq: NF4Tensor, Pq: NF4Tensor, B: torch.Tensor, s: float, x: torch.Tensor,
                    y: torch.Tensor | None = None, ws: torch.Tensor | None = None) -> torch.Tensor:
    T = x.shape[0]
    if y is None:
        y = torch.empty((T, Wq.rows), dtype=torch.bfloat16, device=x.device)
    if ws is None:
        ws = new_workspace(loqt_workspace_bytes(LOQT_OP_FWD, Wq.rows, Wq.cols, Pq.cols, T), x.device)
    _check(lib().loqt_linear_fwd(Wq.view(), Pq.view(), _dev(B, torch.bfloat16), B.stride(0), float(s),
                                 _dev(x, torch.bfloat16), x.stride(0), T, _dev(y, torch.bfloat16), y.stride(0),
                                 ws.data_ptr(), ws.numel(), _stream()), "loqt_linear_fwd")
    return y


def loqt_linear_fwd_static(Wq: NF4Tensor, Pq: NF4Tensor, B: torch.Tensor, s: float, x: torch.Tensor,
                           y: torch.Tensor, check_device_status: bool = True) -> torch.Tensor:
    """Forward through the entry point that needs no workspace: the caller passes
    only inputs and the output `y`; scratch is a fixed array inside the library."""
    T = x.shape[0]
    _check(lib().loqt_linear_fwd_static(Wq.view(), Pq.view(), _dev(B, torch.bfloat16), B.stride(0), float(s),
                                        _dev(x, torch.bfloat16), x.stride(0), T, _dev(y, torch.bfloat16), y.stride(0),
                                        int(bool(check_device_status)), _stream()), "loqt_linear_fwd_static")
    return y


def loqt_linear_bwd(Wq: NF4Tensor, Pq: NF4Tensor, B: torch.Tensor, s: float, x: torch.Tensor, dy: torch.Tensor,
                    dx: torch.Tensor | None = None, dB: torch.Tensor | None = None, accumulate_dB: bool = False,
                    ws: torch.Tensor | None = None, need_dx: bool = True):
    T = x.shape[0]
    if dx is None and need_dx:
        dx = torch.empty((T, Wq.cols), dtype=torch.bfloat16, device=x.device)
    if dB is None:
        dB = torch.zeros((Pq.cols, Wq.cols), dtype=torch.float32, device=x.device)
    if ws is None:
        ws = new_workspace(loqt_workspace_bytes(LOQT_OP_BWD, Wq.rows, Wq.cols, Pq.cols, T), x.device)
    _check(lib().loqt_linear_bwd(Wq.view(), Pq.view(), _dev(B, torch.bfloat16), B.stride(0), float(s),
                                 _dev(x, torch.bfloat16), x.stride(0), _dev(dy, torch.bfloat16), dy.stride(0), T,
                                 _dev(dx, torch.bfloat16) if dx is not None else None,
                                 dx.stride(0) if dx is not None else 0,
                                 _dev(dB, torch.float32), dB.stride(0), int(bool(accumulate_dB)),
                                 ws.data_ptr(), ws.numel(), _stream()), "loqt_linear_bwd")
    return dx, dB


def loqt_merge_requant(Wq: NF4Tensor, Pq: NF4Tensor, B: torch.Tensor, s: float, ws: torch.Tensor | None = None) -> NF4Tensor:
    if ws is None:
        ws = new_workspace(loqt_workspace_bytes(LOQT_OP_MERGE, Wq.rows, Wq.cols, Pq.cols, 0), B.device)
    _check(lib().loqt_merge_requant(Wq.view(), Pq.view(), _dev(B, torch.bfloat16), B.stride(0), float(s),
                                    ws.data_ptr(), ws.numel(), _stream()), "loqt_merge_requant")
    return Wq


def loqt_merge_requant_split(Wq: NF4Tensor, Pq: NF4Tensor, B: torch.Tensor, s: float,
                             ws: torch.Tensor | None = None) -> NF4Tensor:
    if ws is None:
        ws = new_workspace(loqt_workspace_bytes(LOQT_OP_MERGE_SPLIT, Wq.rows, Wq.cols, Pq.cols, 0), B.device)
    _check(lib().loqt_merge_requant_split(Wq.view(), Pq.view(), _dev(B, torch.bfloat16), B.stride(0), float(s),
                                          ws.data_ptr(), ws.numel(), _stream()), "loqt_merge_requant_split")
    return Wq


def loqt_nf4_requantize(delta: torch.Tensor, s: float, Wq: NF4Tensor) -> NF4Tensor:
    _check(lib().loqt_nf4_requantize(_dev(delta, torch.float32), delta.stride(0), float(s), Wq.view(), _stream()),
           "loqt_nf4_requantize")
    return Wq


def loqt_compensated_init(W: torch.Tensor, P: torch.Tensor, steps: int, ws: torch.Tensor | None = None):
    """Returns (Wq, Pq, B): Q_steps, q_NF4(P) and the bf16 factor B_steps."""
    out, inn = W.shape
    r = P.shape[1]
    Wq, Pq = NF4Tensor.empty(out, inn, W.device), NF4Tensor.empty(out, r, W.device)
    ldb = (inn + 7) // 8 * 8
    B = torch.empty((r, ldb), dtype=torch.bfloat16, device=W.device)[:, :inn]
    if ws is None:
        ws = new_workspace(loqt_workspace_bytes(LOQT_OP_COMPENSATE, out, inn, r, 0), W.device)
    _check(lib().loqt_compensated_init(_dev(W, torch.float32), W.stride(0), _dev(P, torch.float32), P.stride(0), int(steps),
                                       Wq.view(), Pq.view(), B.data_ptr(), B.stride(0), ws.data_ptr(), ws.numel(),
                                       _stream()), "loqt_compensated_init")
    loqt_device_status(ws)
    return Wq, Pq, B


def loqt_compensated_init_right(W: torch.Tensor, Q: torch.Tensor, steps: int, ws: torch.Tensor | None = None):
    """Right-side variant.  Returns (Wq, Qq, B): Q_steps, q_NF4(Q) (r x in) and the bf16 factor B_steps (out x r)."""
    out, inn = W.shape
    r = Q.shape[0]
    Wq, Qq = NF4Tensor.empty(out, inn, W.device), NF4Tensor.empty(r, inn, W.device)
    ldb = (r + 7) // 8 * 8
    B = torch.empty((out, ldb), dtype=torch.bfloat16, device=W.device)[:, :r]
    if ws is None:
        ws = new_workspace(loqt_workspace_bytes(LOQT_OP_COMPENSATE_RIGHT, out, inn, r, 0), W.device)
    _check(lib().loqt_compensated_init_right(_dev(W, torch.float32), W.stride(0), _dev(Q, torch.float32), Q.stride(0), int(steps),
                                             Wq.view(), Qq.view(), B.data_ptr(), B.stride(0), ws.data_ptr(), ws.numel(),
                                             _stream()), "loqt_compensated_init_right")
    loqt_device_status(ws)
    return Wq, Qq, B


def loqt_linear_fwd_right(Wq: NF4Tensor, Qq: NF4Tensor, B: torch.Tensor, s: float, x: torch.Tensor) -> torch.Tensor:
    """Right-side variant: y = x deq(W_q)^T + s (x deq(Q_q)^T) B^T; B is out x r."""
    T = x.shape[0]
    y = torch.empty((T, (Wq.rows + 7) // 8 * 8), dtype=torch.bfloat16, device=x.device)[:, : Wq.rows]
    ws = new_workspace(loqt_workspace_bytes(LOQT_OP_FWD_RIGHT, Wq.rows, Wq.cols, Qq.rows, T), x.device)
    _check(lib().loqt_linear_fwd_right(Wq.view(), Qq.view(), _dev(B, torch.bfloat16), B.stride(0), float(s),
                                       _dev(x, torch.bfloat16), x.stride(0), T, y.data_ptr(), y.stride(0),
                                       ws.data_ptr(), ws.numel(), _stream()), "loqt_linear_fwd_right")
    loqt_device_status(ws)
    return y


def loqt_linear_bwd_right(Wq: NF4Tensor, Qq: NF4Tensor, B: torch.Tensor, s: float, x: torch.Tensor, dy: torch.Tensor,
                          dB: torch.Tensor | None = None, accumulate_dB: bool = False):
    """Right-side variant: returns (dx [T, in] bf16, dB [out, r] fp32)."""
    T, r = x.shape[0], Qq.rows
    dx = torch.empty((T, (Wq.cols + 7) // 8 * 8), dtype=torch.bfloat16, device=x.device)[:, : Wq.cols]
    if dB is None:
        dB = torch.empty((Wq.rows, (r + 3) // 4 * 4), dtype=torch.float32, device=x.device)[:, :r]
    ws = new_workspace(loqt_workspace_bytes(LOQT_OP_BWD_RIGHT, Wq.rows, Wq.cols, r, T), x.device)
    _check(lib().loqt_linear_bwd_right(Wq.view(), Qq.view(), _dev(B, torch.bfloat16), B.stride(0), float(s),
                                       _dev(x, torch.bfloat16), x.stride(0), _dev(dy, torch.bfloat16), dy.stride(0), T,
                                       dx.data_ptr(), dx.stride(0), _dev(dB, torch.float32), dB.stride(0),
                                       int(accumulate_dB), ws.data_ptr(), ws.numel(), _stream()), "loqt_linear_bwd_right")
    loqt_device_status(ws)
    return dx, dB


def loqt_merge_requant_right(Wq: NF4Tensor, Qq: NF4Tensor, B: torch.Tensor, s: float) -> NF4Tensor:
    ws = new_workspace(loqt_workspace_bytes(LOQT_OP_MERGE_RIGHT, Wq.rows, Wq.cols, Qq.rows, 0), B.device)
    _check(lib().loqt_merge_requant_right(Wq.view(), Qq.view(), _dev(B, torch.bfloat16), B.stride(0), float(s),
                                          ws.data_ptr(), ws.numel(), _stream()), "loqt_merge_requant_right")
    loqt_device_status(ws)
    return Wq


def loqt_full_gradient(x: torch.Tensor, dy: torch.Tensor, G: torch.Tensor | None = None, accumulate: bool = False,
                       ws: torch.Tensor | None = None) -> torch.Tensor:
    """G^W = dy^T x (fp32 [out, in])."""
    T, inn = x.shape
    out = dy.shape[1]
    if G is None:
        ld = (inn + 3) // 4 * 4
        G = torch.empty((out, ld), dtype=torch.float32, device=x.device)[:, :inn]
    if ws is None:
        ws = new_workspace(loqt_workspace_bytes(LOQT_OP_FULL_GRADIENT, out, inn, 0, T), x.device)
    _check(lib().loqt_full_gradient(_dev(x, torch.bfloat16), x.stride(0), _dev(dy, torch.bfloat16), dy.stride(0), T, out, inn,
                                    _dev(G, torch.float32), G.stride(0), int(accumulate), ws.data_ptr(), ws.numel(),
                                    _stream()), "loqt_full_gradient")
    return G


def loqt_projection(G: torch.Tensor, Omega: torch.Tensor, iters: int, P: torch.Tensor | None = None,
                    ws: torch.Tensor | None = None) -> torch.Tensor:
    """P (fp32 [out, r], orthonormal columns) spanning approximately the r leading left singular vectors of
    G (fp32 [out, in]) by `iters` rounds of subspace iteration started from Omega (bf16 [in, r])."""
    out, inn = G.shape
    r = Omega.shape[1]
    if P is None:
        P = torch.empty((out, r), dtype=torch.float32, device=G.device)
    if ws is None:
        ws = new_workspace(loqt_workspace_bytes(LOQT_OP_PROJECTION, out, inn, r, 0), G.device)
    _check(lib().loqt_projection(_dev(G, torch.float32), G.stride(0), out, inn, r, _dev(Omega, torch.bfloat16), Omega.stride(0),
                                 int(iters), _dev(P, torch.float32), P.stride(0), ws.data_ptr(), ws.numel(), _stream()),
           "loqt_projection")
    return P


def loqt_projection_right(G: torch.Tensor, Omega: torch.Tensor, iters: int, Q: torch.Tensor | None = None,
                          ws: torch.Tensor | None = None) -> torch.Tensor:
    """Q (fp32 [r, in], orthonormal rows) spanning approximately the r leading right singular vectors of
    G (fp32 [out, in]) by `iters` rounds of subspace iteration started from Omega (bf16 [out, r])."""
    out, inn = G.shape
    r = Omega.shape[1]
    if Q is None:
        Q = torch.empty((r, inn), dtype=torch.float32, device=G.device)
    if ws is None:
        ws = new_workspace(loqt_workspace_bytes(LOQT_OP_PROJECTION, out, inn, r, 0), G.device)
    _check(lib().loqt_projection_right(_dev(G, torch.float32), G.stride(0), out, inn, r, _dev(Omega, torch.bfloat16),
                                       Omega.stride(0), int(iters), _dev(Q, torch.float32), Q.stride(0), ws.data_ptr(),
                                       ws.numel(), _stream()), "loqt_projection_right")
    return Q


def loqt_adam_step(B: torch.Tensor, dB: torch.Tensor, m: torch.Tensor, v: torch.Tensor, step: int, lr: float,
                   beta1: float = 0.9, beta2: float = 0.999, eps: float = 1e-8, weight_decay: float = 0.0) -> None:
    """In-place optimiser step on B (bf16) and its bf16 moments m, v from the fp32 gradient dB."""
    if m.shape != B.shape or v.shape != B.shape or m.stride(0) != v.stride(0):
        raise LoqtError("B, m and v must have the same shape, m and v the same row stride")
    hp = loqt_adam_params(lr, beta1, beta2, eps, weight_decay, int(step))
    _check(lib().loqt_adam_step(_dev(B, torch.bfloat16), B.stride(0), _dev(dB, torch.float32), dB.stride(0),
                                _dev(m, torch.bfloat16), _dev(v, torch.bfloat16), m.stride(0), B.shape[0], B.shape[1], hp,
                                _stream()), "loqt_adam_step")


@dataclass
class DQScales:
    """Device storage of the doubly quantised block scales of one NF4 matrix."""
    codes8: torch.Tensor  # uint8 [n]
    c1: torch.Tensor      # fp32 [ceil(n / 256)]
    offset: torch.Tensor  # fp32 [1]

    def view(self) -> loqt_dq_scales:
        return loqt_dq_scales(self.codes8.data_ptr(), self.c1.data_ptr(), self.offset.data_ptr(), self.codes8.numel())

    @staticmethod
    def empty(n: int, device="cuda") -> "DQScales":
        return DQScales(torch.empty((n,), dtype=torch.uint8, device=device),
                        torch.empty(((n + 255) // 256,), dtype=torch.float32, device=device),
                        torch.empty((1,), dtype=torch.float32, device=device))


def loqt_scales_double_quantize(absmax: torch.Tensor, dst: DQScales | None = None) -> DQScales:
    """Doubly quantises the fp32 block scales of a matrix (contiguous, row-major)."""
    if not absmax.is_contiguous():
        raise LoqtError("the scales must be contiguous")
    dst = dst if dst is not None else DQScales.empty(absmax.numel(), absmax.device)
    ws = new_workspace(int(lib().loqt_scales_workspace_bytes()), absmax.device)
    _check(lib().loqt_scales_double_quantize(_dev(absmax, torch.float32), dst.view(), ws.data_ptr(), ws.numel(), _stream()),
           "loqt_scales_double_quantize")
    return dst


def loqt_scales_double_dequantize(src: DQScales, shape) -> torch.Tensor:
    out = torch.empty(shape, dtype=torch.float32, device=src.codes8.device)
    _check(lib().loqt_scales_double_dequantize(src.view(), out.data_ptr(), _stream()), "loqt_scales_double_dequantize")
    return out


def _codes_only(q: NF4Tensor) -> loqt_nf4_mat:
    return loqt_nf4_mat(q.codes.data_ptr(), None, q.rows, q.cols, q.ld, BLOCK)


def loqt_nf4_dequantize_dq(src: NF4Tensor, dq: DQScales, dtype=torch.float32) -> torch.Tensor:
    dst = torch.empty((src.rows, src.cols), dtype=dtype, device=src.codes.device)
    is_bf16 = {torch.float32: 0, torch.bfloat16: 1}[dtype]
    _check(lib().loqt_nf4_dequantize_dq(_codes_only(src), dq.view(), _dev(dst), dst.stride(0), is_bf16, _stream()),
           "loqt_nf4_dequantize_dq")
    return dst


def loqt_linear_fwd_dq(Wq: NF4Tensor, Wdq: DQScales, Pq: NF4Tensor, Pdq: DQScales, B: torch.Tensor, s: float, x: torch.Tensor,
                       y: torch.Tensor | None = None) -> torch.Tensor:
    T = x.shape[0]
    if y is None:
        y = torch.empty((T, (Wq.rows + 7) // 8 * 8), dtype=torch.bfloat16, device=x.device)[:, : Wq.rows]
    ws = new_workspace(loqt_workspace_bytes(LOQT_OP_FWD, Wq.rows, Wq.cols, Pq.cols, T), x.device)
    _check(lib().loqt_linear_fwd_dq(_codes_only(Wq), Wdq.view(), _codes_only(Pq), Pdq.view(), _dev(B, torch.bfloat16), B.stride(0),
                                    float(s), _dev(x, torch.bfloat16), x.stride(0), T, _dev(y, torch.bfloat16), y.stride(0),
                                    ws.data_ptr(), ws.numel(), _stream()), "loqt_linear_fwd_dq")
    loqt_device_status(ws)
    return y


def loqt_linear_bwd_dq(Wq: NF4Tensor, Wdq: DQScales, Pq: NF4Tensor, Pdq: DQScales, B: torch.Tensor, s: float, x: torch.Tensor,
                       dy: torch.Tensor):
    T = x.shape[0]
    dx = torch.empty((T, (Wq.cols + 7) // 8 * 8), dtype=torch.bfloat16, device=x.device)[:, : Wq.cols]
    dB = torch.empty((Pq.cols, (Wq.cols + 3) // 4 * 4), dtype=torch.float32, device=x.device)[:, : Wq.cols]
    ws = new_workspace(loqt_workspace_bytes(LOQT_OP_BWD, Wq.rows, Wq.cols, Pq.cols, T), x.device)
    _check(lib().loqt_linear_bwd_dq(_codes_only(Wq), Wdq.view(), _codes_only(Pq), Pdq.view(), _dev(B, torch.bfloat16), B.stride(0),
                                    float(s), _dev(x, torch.bfloat16), x.stride(0), _dev(dy, torch.bfloat16), dy.stride(0), T,
                                    dx.data_ptr(), dx.stride(0), dB.data_ptr(), dB.stride(0), 0, ws.data_ptr(), ws.numel(),
                                    _stream()), "loqt_linear_bwd_dq")
    loqt_device_status(ws)
    return dx, dB


def loqt_adam8_step(B: torch.Tensor, dB: torch.Tensor, m8: torch.Tensor, m_absmax: torch.Tensor, v8: torch.Tensor,
                    v_absmax: torch.Tensor, step: int, lr: float, beta1: float = 0.9, beta2: float = 0.999, eps: float = 1e-8,
                    weight_decay: float = 0.0) -> None:
    """In-place optimiser step on B (bf16) with 8-bit block-wise quantised moments
    (m8, v8: uint8 [r * in]; m_absmax, v_absmax: fp32 [ceil(r * in / 2048)])."""
    n = B.shape[0] * B.shape[1]
    if m8.numel() != n or v8.numel() != n or m_absmax.numel() != (n + 2047) // 2048 or v_absmax.numel() != (n + 2047) // 2048:
        raise LoqtError("moment buffers do not match the shape of B")
    hp = loqt_adam_params(lr, beta1, beta2, eps, weight_decay, int(step))
    st = loqt_adam8_state(_dev(m8, torch.uint8), _dev(m_absmax, torch.float32), _dev(v8, torch.uint8), _dev(v_absmax, torch.float32))
    _check(lib().loqt_adam8_step(_dev(B, torch.bfloat16), B.stride(0), _dev(dB, torch.float32), dB.stride(0), st,
                                 B.shape[0], B.shape[1], hp, _stream()), "loqt_adam8_step")


def merge_many_workspace_bytes(Wqs, Pqs, group: int = 8) -> int:
    """Workspace that lets loqt_merge_requant_many stage `group` matrices ahead
    (the status block plus `group` scratch slots of the largest matrix)."""
    if not Wqs:
        return 256
    need = max(loqt_workspace_bytes(LOQT_OP_MERGE, w.rows, w.cols, p.cols, 0) for w, p in zip(Wqs, Pqs))
    return 256 + max(1, min(group, len(Wqs))) * (need - 256)


def loqt_merge_requant_many(Wqs, Pqs, Bs, s: float, ws: torch.Tensor | None = None):
    n = len(Wqs)
    if ws is None:
        ws = new_workspace(merge_many_workspace_bytes(Wqs, Pqs), Bs[0].device)
    aW = (loqt_nf4_mat * n)(*[w.view() for w in Wqs])
    aP = (loqt_nf4_mat * n)(*[p.view() for p in Pqs])
    aB = (ctypes.c_void_p * n)(*[_dev(b, torch.bfloat16) for b in Bs])
    aL = (ctypes.c_int64 * n)(*[b.stride(0) for b in Bs])
    _check(lib().loqt_merge_requant_many(n, aW, aP, aB, aL, float(s), ws.data_ptr(), ws.numel(), _stream()),
           "loqt_merge_requant_many")
    return Wqs


def loqt_device_status(ws: torch.Tensor) -> None:
    _check(lib().loqt_device_status(ws.data_ptr(), _stream()), "device status")


def loqt_launch_count() -> int:
    return int(lib().loqt_launch_count())


def loqt_set_tile_override(bn: int, rows: int = 128, pair: bool = False) -> None:
    """Forces a tile shape for later products (bn = 0: automatic again)."""
    _check(lib().loqt_set_tile_override(int(bn), int(rows), int(bool(pair))), "loqt_set_tile_override")


def loqt_variant_launches(bn: int, rows: int, pair: bool, nf4: bool) -> int:
    return int(lib().loqt_variant_launches(int(bn), int(rows), int(bool(pair)), int(bool(nf4))))


def loqt_selftest_wait_timeout(ws: torch.Tensor, limit_us: int = 1000) -> None:
    """Launches the wait self-test; the outcome is read with loqt_device_status(ws)."""
    _check(lib().loqt_selftest_wait_timeout(ws.data_ptr(), ws.numel(), int(limit_us), _stream()),
           "loqt_selftest_wait_timeout")
