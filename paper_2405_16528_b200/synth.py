"""Seeded synthetic inputs shaped like the paper's Llama-style layers.

Holds no arithmetic of the method itself: it only draws random matrices.  Both
the tests (which feed the same tensors to the CPU oracle and to the CUDA
library) and the benchmark use it.

Shapes follow the paper's hyper-parameter table (hidden / intermediate size,
rank) and its sequence length of 256; the value distributions are
W ~ N(0, 0.02^2), P = an orthonormal out x r matrix (what the top-r left
singular vectors of a gradient look like), B ~ N(0, sigma_B^2), and
activations / output gradients ~ N(0, 1).
"""
from __future__ import annotations

import hashlib
from dataclasses import dataclass

import torch


def tensor_seed(seed: int, *names) -> int:
    """Stable 63-bit seed derived from (seed, names...)."""
    h = hashlib.blake2b(repr((int(seed),) + tuple(str(n) for n in names)).encode(), digest_size=8)
    return int.from_bytes(h.digest(), "little") & 0x7FFFFFFFFFFFFFFF


def _gen(seed, names, device):
    g = torch.Generator(device=device)
    g.manual_seed(tensor_seed(seed, *names))
    return g


def normal(seed, names, shape, sigma=1.0, dtype=torch.float32, device="cpu"):
    """N(0, sigma^2) tensor, drawn in fp32 then rounded to `dtype`."""
    g = _gen(seed, names, device)
    t = torch.randn(shape, generator=g, device=device, dtype=torch.float32) * float(sigma)
    return t.to(dtype)


def orthonormal(seed, names, rows, cols, device="cpu"):
    """fp32 rows x cols matrix with orthonormal columns: the Q factor (sign-fixed
    so that diag(R) > 0) of a Gaussian matrix."""
    g = _gen(seed, names, device)
    a = torch.randn((rows, cols), generator=g, device=device, dtype=torch.float32)
    wide = torch.float64 if torch.device(device).type == "cpu" else torch.float32
    q, r = torch.linalg.qr(a.to(wide), mode="reduced")
    q = q * torch.sign(torch.diagonal(r)).unsqueeze(0)
    return q.to(torch.float32).contiguous()


def lowrank_gradient(seed, names, out, inn, r, tail=0.5, noise=1e-3, device="cpu"):
    """fp32 out x in matrix shaped like a layer's full-rank gradient: a dominant
    part of rank r (singular values spread linearly over [1, 2]), a tail of
    min(out, in) - r further directions (singular values from `tail` down to a
    tenth of it) and dense Gaussian noise of standard deviation `noise`.
    Singular vectors are Q factors of Gaussian matrices.  Drawn in float64."""
    g = _gen(seed, names, "cpu")
    k = min(out, inn)
    U, _ = torch.linalg.qr(torch.randn((out, k), generator=g, dtype=torch.float64))
    V, _ = torch.linalg.qr(torch.randn((inn, k), generator=g, dtype=torch.float64))
    sv = torch.cat([torch.linspace(2.0, 1.0, r, dtype=torch.float64),
                    float(tail) * torch.linspace(1.0, 0.1, k - r, dtype=torch.float64)])
    G = (U * sv) @ V.T + float(noise) * torch.randn((out, inn), generator=g, dtype=torch.float64)
    return G.to(torch.float32).to(device)


@dataclass(frozen=True)
class LayerSet:
    """One benchmark / parity configuration: the distinct projection shapes of a
    decoder layer, how often each occurs per layer, and the layer count."""
    name: str
    hidden: int
    mlp: int
    layers: int
    r: int
    T: int
    sigma_B: float
    single: bool = False  # a single square matrix instead of a layer set

    def shapes(self):
        """[(label, out, in, count per layer)]"""
        if self.single:
            return [("w", self.hidden, self.hidden, 1)]
        return [
            ("attn_qkvo", self.hidden, self.hidden, 4),
            ("mlp_gate_up", self.mlp, self.hidden, 2),
            ("mlp_down", self.hidden, self.mlp, 1),
        ]

    def matrices(self):
        return sum(c for _, _, _, c in self.shapes()) * self.layers


CONFIGS = [
    LayerSet("single-256", 256, 256, 1, 32, 512, 1e-3, single=True),
    LayerSet("llama-60m", 512, 1376, 8, 128, 4096, 1e-3),
    LayerSet("llama-350m", 1024, 2736, 24, 256, 4096, 1e-3),
    LayerSet("llama-1b", 2048, 5461, 24, 512, 8192, 1e-2),
    LayerSet("llama-7b", 4096, 11008, 32, 1024, 4096, 1e-3),
]


def fwd_bwd_flops(out: int, inn: int, r: int, T: int) -> int:
    """Algorithmic flops of one factored forward + backward:
    main products (y, dx) 4*T*in*out, low-rank products (u, u->y, v, v->dx, dB)
    2*T*r*(3*in + 2*out)."""
    return 4 * T * inn * out + 2 * T * r * (3 * inn + 2 * out)


def nf4_bytes(rows: int, cols: int) -> int:
    ld = (cols + 63) // 64 * 64
    return rows * ld // 2 + rows * (ld // 64) * 4


def merge_bytes(out: int, inn: int, r: int) -> int:
    """Algorithmic bytes of one merge: read + write W_q, read P_q, read bf16 B."""
    return 2 * nf4_bytes(out, inn) + nf4_bytes(out, r) + r * inn * 2


def make_layer(seed, label, out, inn, r, sigma_B, T=None, device="cpu"):
    """The tensors of one LoQT linear: fp32 W and P (to be NF4-quantised by the
    caller), bf16 B, and - when T is given - bf16 x and dy."""
    d = {
        "W": normal(seed, (label, "W"), (out, inn), 0.02, torch.float32, device),
        "P": orthonormal(seed, (label, "P"), out, r, device),
        "B": normal(seed, (label, "B"), (r, inn), sigma_B, torch.bfloat16, device),
    }
    if T is not None:
        d["x"] = normal(seed, (label, "x"), (T, inn), 1.0, torch.bfloat16, device)
        d["dy"] = normal(seed, (label, "dy"), (T, out), 1.0, torch.bfloat16, device)
    return d
