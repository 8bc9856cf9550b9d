"""CPU oracle for the LoQT quantized low-rank linear layer (arXiv 2405.16528).

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, obviously-correct
statement of what the GPU library must compute.  It is imported by the tests,
by the smoke check and by the benchmark's CPU-baseline leg, and by nothing
else; the product path never routes through it.  It shares no code, table or
helper with the CUDA sources: the NF4 level table below is this file's own
copy.

Everything is numpy.  Floating-point contractions run in float64 (numpy's
matmul serves as the library primitive); no blocking, fusion or reordering is
applied beyond what the definitions state.

Conventions (PyTorch nn.Linear style: W is out x in):

    W_q : NF4 codes + one fp32 absmax per block of 64 consecutive elements of
          a row (Section 5.1 "Neural Network Quantization and NF4")
    P_q : NF4, out x r        B : r x in (16-bit)        s : scalar (Alg. 1)
    W_eff = deq(W_q) + s * deq(P_q) @ B          (Section 2, Alg. 1 merge line)

Parity pins (tests/test_oracle_*.py): level table vs. the closed-form quantile
construction; quantiser vs. pure-Python brute force, exact round trip of the
16 levels, +-1 at the block maximum, idempotence; bf16 rounding vs. torch's
conversion; forward/backward vs. the dense W_eff route, torch fp64 autograd and
central finite differences; merge vs. zero-B identity and the dense product.
No function here is "parity unpinned".
"""
from __future__ import annotations

import numpy as np

BLOCK = 64  # Section 5.1: the block length of the NF4 quantiser

# NF4 levels q_1..q_16 (ascending).  The paper defers to QLoRA for the values
# (Section 5.1); these are the 16 fp32 numbers published there: 8 positive and
# 7 negative equal-probability N(0,1) quantiles plus an exact zero, divided by
# the largest.  tests/test_oracle_nf4.py rebuilds them from that closed form.
NF4_LEVELS = np.array(
    [
        -1.0,
        -0.6961928009986877,
        -0.5250730514526367,
        -0.39491748809814453,
        -0.28444138169288635,
        -0.18477343022823334,
        -0.09105003625154495,
        0.0,
        0.07958029955625534,
        0.16093020141124725,
        0.24611230194568634,
        0.33791524171829224,
        0.44070982933044434,
        0.5626170039176941,
        0.7229568362236023,
        1.0,
    ],
    dtype=np.float32,
)
ZERO_CODE = 7  # index of the exact 0.0 level; used for padding and all-zero blocks


# ----------------------------------------------------------------------------
# bf16 helpers (the 16-bit format of B, x, dy and of the dequantised operands)
# ----------------------------------------------------------------------------
def bf16_round(a: np.ndarray) -> np.ndarray:
    """Round fp32 values to the nearest bf16 (ties to even); returns fp32 holding
    bf16-representable values.  bf16 keeps the top 16 bits of an fp32."""
    a32 = np.ascontiguousarray(a, dtype=np.float32)
    u = a32.view(np.uint32).astype(np.uint64)
    lsb = (u >> np.uint64(16)) & np.uint64(1)
    r = ((u + np.uint64(0x7FFF) + lsb) >> np.uint64(16)) << np.uint64(16)
    return (r & np.uint64(0xFFFFFFFF)).astype(np.uint32).view(np.float32).reshape(a32.shape)


# ----------------------------------------------------------------------------
# Storage layout (ABI-visible, not arithmetic): rows padded to a multiple of 64
# ----------------------------------------------------------------------------
def padded_cols(cols: int) -> int:
    return (cols + BLOCK - 1) // BLOCK * BLOCK


def pack_codes(codes: np.ndarray) -> np.ndarray:
    """[rows, ld] codes 0..15 -> [rows, ld/2] bytes; element 2j is the low nibble
    of byte j, element 2j+1 the high nibble."""
    c = codes.astype(np.uint8)
    return (c[:, 0::2] | (c[:, 1::2] << 4)).astype(np.uint8)


def unpack_codes(packed: np.ndarray) -> np.ndarray:
    rows, half = packed.shape
    out = np.empty((rows, half * 2), dtype=np.uint8)
    out[:, 0::2] = packed & 0x0F
    out[:, 1::2] = packed >> 4
    return out


# ----------------------------------------------------------------------------
# NF4 quantise / dequantise  (Section 5.1, the four displayed equations)
# ----------------------------------------------------------------------------
def nf4_quantize(w: np.ndarray):
    """q_NF4 applied to a 2-D fp32 matrix.

    Blocks are 64 consecutive elements along a row; a row whose length is not a
    multiple of 64 ends in a short block whose scale is taken over its real
    elements, and the storage is padded with the zero level.

    Per block: M = max |w| (fp32, exact).  Per element: n = w / M rounded to
    fp32 (so the block's largest-magnitude element maps to exactly +-1), and
    the code is argmin_i |n - q_i| over the 16 levels, evaluated in float64,
    first index on ties.  A block of zeros gets M = 0 and the zero level.

    Returns (codes uint8 [rows, ld] with values 0..15, absmax fp32 [rows, ld/64]).
    """
    w = np.asarray(w)
    assert w.ndim == 2 and w.dtype == np.float32
    rows, cols = w.shape
    ld = padded_cols(cols)
    nb = ld // BLOCK
    codes = np.full((rows, ld), ZERO_CODE, dtype=np.uint8)
    absmax = np.zeros((rows, nb), dtype=np.float32)
    levels64 = NF4_LEVELS.astype(np.float64)
    for b in range(nb):
        c0, c1 = b * BLOCK, min((b + 1) * BLOCK, cols)
        blk = w[:, c0:c1]
        m = np.max(np.abs(blk), axis=1).astype(np.float32)
        absmax[:, b] = m
        nz = m > 0
        if not np.any(nz):
            continue
        with np.errstate(divide="ignore", invalid="ignore"):
            n = (blk / m[:, None]).astype(np.float32)  # fp32 IEEE division
        dist = np.abs(n.astype(np.float64)[:, :, None] - levels64[None, None, :])
        idx = np.argmin(dist, axis=2).astype(np.uint8)  # first occurrence on ties
        idx[~nz, :] = ZERO_CODE
        codes[:, c0:c1] = idx
    return codes, absmax


def nf4_dequantize(codes: np.ndarray, absmax: np.ndarray, cols: int | None = None) -> np.ndarray:
    """q_NF4^{-1}: w = M_beta * q[code], one fp32 multiply.  Returns fp32 [rows, cols]."""
    rows, ld = codes.shape
    cols = ld if cols is None else cols
    m = np.repeat(absmax.astype(np.float32), BLOCK, axis=1)[:, :ld]
    w = (m * NF4_LEVELS[codes]).astype(np.float32)
    return w[:, :cols]


def nf4_dequantize_bf16(codes, absmax, cols=None) -> np.ndarray:
    """The 16-bit operand the matrix products see (Section 2.4: W_BF16, P_BF16):
    the fp32 dequantised value rounded once to bf16."""
    return bf16_round(nf4_dequantize(codes, absmax, cols))


# ----------------------------------------------------------------------------
# Forward, backward  (Section 2, "Equivalence of Gradient Updates"; Alg. 1)
# ----------------------------------------------------------------------------
def _operands(wq, pq, B, out_in_r):
    out, inn, r = out_in_r
    W = nf4_dequantize_bf16(wq[0], wq[1], inn).astype(np.float64)  # out x in
    P = nf4_dequantize_bf16(pq[0], pq[1], r).astype(np.float64)  # out x r
    Bm = np.asarray(B, dtype=np.float64)
    assert W.shape == (out, inn) and P.shape == (out, r) and Bm.shape == (r, inn)
    return W, P, Bm


def loqt_forward(wq, pq, B, s, x, shape):
    """y = x W^T + s (x B^T) P^T with W = deq(W_q), P = deq(P_q); float64, the
    factored order the method states.  `wq`, `pq` are (codes, absmax) pairs,
    `shape` = (out, in, r).  x is T x in (bf16-representable values)."""
    W, P, Bm = _operands(wq, pq, B, shape)
    x = np.asarray(x, dtype=np.float64)
    u = x @ Bm.T  # T x r
    return x @ W.T + float(s) * (u @ P.T)


def loqt_backward(wq, pq, B, s, x, dy, shape):
    """Gradients of L = <y, dy>:  v = dy P;  dx = dy W + s v B;
    dB = s v^T x  (= s P^T G^W with G^W = dy^T x).  W and P are frozen, so no
    other gradient exists.  Returns (dx [T, in], dB [r, in]) in float64."""
    W, P, Bm = _operands(wq, pq, B, shape)
    x = np.asarray(x, dtype=np.float64)
    dy = np.asarray(dy, dtype=np.float64)
    v = dy @ P  # T x r
    dx = dy @ W + float(s) * (v @ Bm)
    dB = float(s) * (v.T @ x)
    return dx, dB


# ----------------------------------------------------------------------------
# Periodic merge + requantise  (Section 2.4; Alg. 1 merge line; Section 2.5)
# ----------------------------------------------------------------------------
def loqt_merge_values(wq, pq, B, s, shape) -> np.ndarray:
    """The fp32 matrix handed to the quantiser at a merge:
    fl32( deq32(W_q) + s * P_BF16 @ B ), the sum formed in float64 and rounded
    once.  The quantiser's input is 32-bit (Section 5.1), so W enters with its
    unrounded fp32 dequantised value; P enters as the 16-bit matmul operand."""
    out, inn, r = shape
    W32 = nf4_dequantize(wq[0], wq[1], inn).astype(np.float64)
    P = nf4_dequantize_bf16(pq[0], pq[1], r).astype(np.float64)
    delta = P @ np.asarray(B, dtype=np.float64)
    return (W32 + float(s) * delta).astype(np.float32)


def loqt_merge_requant(wq, pq, B, s, shape):
    """W_q <- q_NF4( deq(W_q) + s deq(P_q) B ).  Returns (codes, absmax)."""
    return nf4_quantize(loqt_merge_values(wq, pq, B, s, shape))


def nf4_requantize(wq, delta, s, cols):
    """The requantising half of the merge with the product already formed
    (Section 2.4; Algorithm 1, merge line; quantiser of Section 5.1):
    W_q <- q_NF4( fl32( deq32(W_q) + s * delta ) ) for an fp32 matrix `delta`
    ([rows, cols]); the sum is formed in float64 and rounded once.  Returns
    (codes, absmax)."""
    W32 = nf4_dequantize(wq[0], wq[1], cols).astype(np.float64)
    d = np.asarray(delta, dtype=np.float32).astype(np.float64)
    return nf4_quantize((W32 + float(s) * d).astype(np.float32))


def loqt_compensate(W, P, steps, B0=None):
    """Error-compensated initialisation of (Q, B) for a fixed projection P
    (Section 2.5 "Compensating for Quantization Errors"; Algorithm 2, the loop
    over compensation steps; appendix "Choice of Quantization Method": B =
    P^+ (W - Q)).  Alternating minimisation of || Q + P B - W ||:

        B_0 = 0
        for c = 1..steps:   Q_c = q_NF4( W - P B_{c-1} )
                            B_c = P^+ ( W - deq(Q_c) )

    P has orthonormal columns, so P^+ = P^T.  Precisions follow the hot path:
    W and W - P B are 32-bit (the quantiser's input), P, the residual
    W - deq(Q_c) and B enter the matrix products as 16-bit operands (one rounding
    each), sums in float64.

    W: fp32 [out, in]; P: fp32 [out, r].  Returns ((codes, absmax) of Q_steps,
    B_steps as fp32 holding bf16 values [r, in]).  B0 (bf16 values, [r, in])
    replaces the zero start of Algorithm 2, so that a test can check one step
    from any state."""
    W = np.asarray(W, dtype=np.float32)
    out, inn = W.shape
    Pb = bf16_round(np.asarray(P, dtype=np.float32)).astype(np.float64)
    W64 = W.astype(np.float64)
    B = np.zeros((Pb.shape[1], inn), dtype=np.float32) if B0 is None else bf16_round(np.asarray(B0, dtype=np.float32))
    q = None
    for _ in range(int(steps)):
        what = (W64 - Pb @ B.astype(np.float64)).astype(np.float32)
        q = nf4_quantize(what)
        resid = bf16_round((W - nf4_dequantize(q[0], q[1], inn)).astype(np.float32))
        B = bf16_round((Pb.T @ resid.astype(np.float64)).astype(np.float32))
    return q, B


def adam_step(B, g, m, v, step, lr, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0):
    """One optimiser step on the trainable factor, B <- B - rho(G^B) (Algorithm 1,
    the update line; Section 2.1: rho is Adam; hyper-parameter tables: AdamW,
    optimiser states in BF16).  Adam as published by Kingma & Ba (Algorithm 1
    there) with the decoupled weight decay of Loshchilov & Hutter:

        m <- beta1 m + (1 - beta1) g          v <- beta2 v + (1 - beta2) g^2
        mhat = m / (1 - beta1^t)              vhat = v / (1 - beta2^t)
        B <- B - lr ( mhat / (sqrt(vhat) + eps) + weight_decay B )

    B, m, v hold bf16 values, g is fp32; everything is evaluated in float64 and
    B, m, v are rounded to bf16 once at the end.  Returns (B, m, v) as fp32 arrays
    holding bf16 values."""
    B64 = np.asarray(B, dtype=np.float64)
    g64 = np.asarray(g, dtype=np.float32).astype(np.float64)
    m64 = beta1 * np.asarray(m, dtype=np.float64) + (1.0 - beta1) * g64
    v64 = beta2 * np.asarray(v, dtype=np.float64) + (1.0 - beta2) * g64 * g64
    mhat = m64 / (1.0 - beta1 ** step)
    vhat = v64 / (1.0 - beta2 ** step)
    Bn = B64 - lr * (mhat / (np.sqrt(vhat) + eps) + weight_decay * B64)
    return bf16_round(Bn.astype(np.float32)), bf16_round(m64.astype(np.float32)), bf16_round(v64.astype(np.float32))


def full_gradient(x, dy):
    """G^W = dy^T x, the full-rank gradient of the layer's weight (out x in) that is
    formed only at merge steps to find the next projection (Section 2.1, the
    gradient G^W of Eq. for W's update; Algorithm 1, the line that computes G^W
    before Initialize; Algorithm 2 takes its SVD).  Sums in float64."""
    return np.asarray(dy, dtype=np.float64).T @ np.asarray(x, dtype=np.float64)


# ----------------------------------------------------------------------------
# Right-side variant  (Section 2.1, the one-sided projection equation and the
# paragraph after it: a matrix taller than wide is projected from the right,
# G Q, and the adapter derivation carries over with Q^T).  The adapter sits on
# the input side:
#     W = deq(W_q) + s B deq(Q_q),   B out x r trainable (bf16),   Q r x in frozen NF4.
# ----------------------------------------------------------------------------
def _operands_right(wq, qq, B, out_in_r):
    out, inn, r = out_in_r
    W = nf4_dequantize_bf16(wq[0], wq[1], inn).astype(np.float64)  # out x in
    Q = nf4_dequantize_bf16(qq[0], qq[1], inn).astype(np.float64)  # r x in
    Bm = np.asarray(B, dtype=np.float64)
    assert W.shape == (out, inn) and Q.shape == (r, inn) and Bm.shape == (out, r)
    return W, Q, Bm


def loqt_forward_right(wq, qq, B, s, x, shape):
    """y = x W^T + s (x Q^T) B^T, float64, factored order."""
    W, Q, Bm = _operands_right(wq, qq, B, shape)
    x = np.asarray(x, dtype=np.float64)
    return x @ W.T + float(s) * ((x @ Q.T) @ Bm.T)


def loqt_backward_right(wq, qq, B, s, x, dy, shape):
    """Gradients of L = <y, dy>:  dx = dy W + s (dy B) Q;  dB = s dy^T (x Q^T)
    (= s G^W Q^T with G^W = dy^T x).  Returns (dx [T, in], dB [out, r])."""
    W, Q, Bm = _operands_right(wq, qq, B, shape)
    x = np.asarray(x, dtype=np.float64)
    dy = np.asarray(dy, dtype=np.float64)
    dx = dy @ W + float(s) * ((dy @ Bm) @ Q)
    dB = float(s) * (dy.T @ (x @ Q.T))
    return dx, dB


def loqt_compensate_right(W, Q, steps, B0=None):
    """Error-compensated initialisation for the right-side variant (Section 2.5 and
    Algorithm 2's loop, carried over to the right-side factorisation W = Q_w + B Q of
    Section 2.1): alternating minimisation of || Q_w + B Q - W || for a fixed Q with
    orthonormal rows,

        B_0 = 0;  for c = 1..steps:  Q_c = q_NF4( W - B_{c-1} Q ),  B_c = ( W - deq(Q_c) ) Q^+

    with Q^+ = Q^T.  Precisions as in loqt_compensate: W and W - B Q are 32-bit, Q, the
    residual and B enter the products as 16-bit operands, sums in float64.
    W: fp32 [out, in]; Q: fp32 [r, in].  Returns ((codes, absmax) of Q_steps, B_steps as
    fp32 holding bf16 values [out, r])."""
    W = np.asarray(W, dtype=np.float32)
    out, inn = W.shape
    Qb = bf16_round(np.asarray(Q, dtype=np.float32)).astype(np.float64)
    W64 = W.astype(np.float64)
    B = np.zeros((out, Qb.shape[0]), dtype=np.float32) if B0 is None else bf16_round(np.asarray(B0, dtype=np.float32))
    q = None
    for _ in range(int(steps)):
        what = (W64 - B.astype(np.float64) @ Qb).astype(np.float32)
        q = nf4_quantize(what)
        resid = bf16_round((W - nf4_dequantize(q[0], q[1], inn)).astype(np.float32))
        B = bf16_round((resid.astype(np.float64) @ Qb.T).astype(np.float32))
    return q, B


def loqt_merge_values_right(wq, qq, B, s, shape) -> np.ndarray:
    """fl32( deq32(W_q) + s * B @ Q_BF16 ): the quantiser's input at a merge."""
    out, inn, r = shape
    W32 = nf4_dequantize(wq[0], wq[1], inn).astype(np.float64)
    Q = nf4_dequantize_bf16(qq[0], qq[1], inn).astype(np.float64)
    return (W32 + float(s) * (np.asarray(B, dtype=np.float64) @ Q)).astype(np.float32)


# ----------------------------------------------------------------------------
# Double quantisation of the block scales  (Section 2.4: the quantisation state
# is itself quantised, following QLoRA)
#
# The paper gives no parameters; the reading taken is QLoRA's description of
# its "double quantization": the fp32 block scales c2 (one per 64 weights) are
# centred by subtracting their mean, cut into blocks of 256, and each block is
# quantised symmetrically to an 8-bit float with one fp32 scale c1 per block.
# The 8-bit float is taken to be the OCP FP8 E4M3 format (1 sign, 4 exponent, 3
# mantissa bits, bias 7, subnormals, largest finite value 448, no infinities),
# scaled so that 448 stands for the block's largest centred scale.  Storage per
# weight: 4 bits of code + 8/64 bits of scale code + 32/(64*256) bits of c1
# = 4.127 bits, against 4.5 with fp32 scales.
# ----------------------------------------------------------------------------
DQ_BLOCK = 256        # first-level scales per second-level block
E4M3_MAX = 448.0


def e4m3_decode(code: np.ndarray) -> np.ndarray:
    """Value of an FP8 E4M3 bit pattern (OCP 8-bit floating point specification):
    sign s, exponent e (4 bits, bias 7), mantissa m (3 bits);
    e = 0: (-1)^s 2^-6 (m / 8);  otherwise (-1)^s 2^(e-7) (1 + m / 8);
    e = 15, m = 7 is NaN.  Returns float64."""
    c = np.asarray(code, dtype=np.uint8).astype(np.int64)
    s = np.where(c & 0x80, -1.0, 1.0)
    e = (c >> 3) & 0xF
    m = (c & 0x7).astype(np.float64)
    val = np.where(e == 0, 2.0 ** -6 * (m / 8.0), 2.0 ** (e - 7).astype(np.float64) * (1.0 + m / 8.0))
    val = np.where((e == 15) & (m == 7), np.nan, val)
    return s * val


def e4m3_encode(x: np.ndarray) -> np.ndarray:
    """Nearest E4M3 value of each |x| <= 448 (round to nearest, ties to the even
    mantissa), by search over the 254 finite bit patterns; +0 for zeros of either sign."""
    x = np.asarray(x, dtype=np.float64)
    codes = np.array([c for c in range(256) if (c & 0x7F) != 0x7F and c != 0x80], dtype=np.uint8)  # finite, one zero
    vals = e4m3_decode(codes)
    order = np.argsort(vals, kind="stable")
    codes, vals = codes[order], vals[order]
    hi = np.clip(np.searchsorted(vals, x, side="left"), 1, len(vals) - 1)
    lo = hi - 1
    d_lo, d_hi = np.abs(x - vals[lo]), np.abs(vals[hi] - x)
    pick_hi = (d_hi < d_lo) | ((d_hi == d_lo) & ((codes[hi] & 1) == 0))   # tie: even mantissa bit pattern
    out = np.where(pick_hi, codes[hi], codes[lo]).astype(np.uint8)
    return out


def dq_quantize_absmax(absmax: np.ndarray, offset=None):
    """Double quantisation of the fp32 block scales of one matrix.

    absmax: fp32, any shape; taken in row-major order as one sequence c2[0..n).
    offset: the mean of c2 rounded to fp32 (computed here in float64 unless given;
            any nearby value is a valid encoding parameter, so a caller may pass
            the one another implementation chose).
    Per block of 256 consecutive scales: d = fl32(c2 - offset); m = max |d|;
    code = E4M3( fl32( fl32(d / m) * 448 ) ), +0 when m = 0; the stored second-level
    scale is c1 = fl32(m / 448), the value one E4M3 unit stands for.
    Returns (codes uint8 [n], c1 fp32 [ceil(n / 256)], offset fp32 scalar)."""
    c2 = np.ascontiguousarray(absmax, dtype=np.float32).reshape(-1)
    n = c2.size
    if offset is None:
        offset = np.float32(np.mean(c2.astype(np.float64))) if n else np.float32(0.0)
    offset = np.float32(offset)
    nb = (n + DQ_BLOCK - 1) // DQ_BLOCK
    codes = np.zeros(n, dtype=np.uint8)
    c1 = np.zeros(nb, dtype=np.float32)
    d = (c2 - offset).astype(np.float32)
    for b in range(nb):
        blk = d[b * DQ_BLOCK : (b + 1) * DQ_BLOCK]
        m = np.float32(np.max(np.abs(blk)))
        c1[b] = np.float32(m / np.float32(E4M3_MAX))
        if m > 0:
            t = ((blk / m).astype(np.float32) * np.float32(E4M3_MAX)).astype(np.float32)
            codes[b * DQ_BLOCK : b * DQ_BLOCK + blk.size] = e4m3_encode(t)
    return codes, c1, offset


def dq_dequantize_absmax(codes: np.ndarray, c1: np.ndarray, offset, shape=None) -> np.ndarray:
    """The scales the layer works with after double quantisation:
    c2' = fl32( fl32( E4M3(code) * c1 ) + offset ), two fp32 roundings."""
    codes = np.asarray(codes, dtype=np.uint8).reshape(-1)
    q = e4m3_decode(codes).astype(np.float32)
    scale = np.repeat(np.asarray(c1, dtype=np.float32), DQ_BLOCK)[: codes.size]
    out = ((q * scale).astype(np.float32) + np.float32(offset)).astype(np.float32)
    return out if shape is None else out.reshape(shape)


def dq_bits_per_weight() -> float:
    """Storage of a doubly quantised NF4 matrix per weight, in bits."""
    return 4.0 + 8.0 / BLOCK + 32.0 / (BLOCK * DQ_BLOCK)


# ----------------------------------------------------------------------------
# 8-bit optimiser states  (the paper trains B with "8-bit Adam", citing Dettmers et
# al., "8-bit Optimizers via Block-wise Quantization": Section 3.2 memory
# comparison, the 13B run and the continued-pretraining appendix)
#
# The paper gives no formulas; the reading taken is that publication's scheme:
# the two Adam moments are stored as 8-bit codes, quantised block-wise (blocks of
# 2048 consecutive elements, one fp32 scale = the block's largest magnitude), in
# the "dynamic tree" data type - a sign bit, then a run of zero bits whose length
# E is a base-10 exponent, an indicator bit, and the remaining f bits a linear
# fraction - with the sign bit turned into one more fraction bit for the
# non-negative second moment.  The fraction's grid inside a decade is this
# file's reading: magnitude(E, j) = 10^-E * (0.1 + 0.9 * (j + 1) / 2^f), j = 0 ..
# 2^f - 1, so that a decade's largest value is 10^-E itself and its smallest lies
# just above the decade below; code 0 is zero.  Read as an integer, the magnitude
# bits are then 2^f + j: magnitudes ascend with the code.
# An optimiser step dequantises the moments, updates in 32-bit arithmetic, and
# quantises them again.
# ----------------------------------------------------------------------------
OPT8_BLOCK = 2048


def dyn8_codebook(signed: bool) -> np.ndarray:
    """Magnitudes of the 8-bit dynamic data type as fp32, indexed by the magnitude
    bits (7 of them when a sign bit is kept, else 8): 128 or 256 ascending values."""
    bits = 7 if signed else 8
    c = np.zeros(1 << bits, dtype=np.float64)
    for f in range(bits):
        E = bits - 1 - f
        for j in range(1 << f):
            c[(1 << f) + j] = (0.1 + 0.9 * (j + 1) / float(1 << f)) * (10.0 ** -E)
    return c.astype(np.float32)


def dyn8_quantize(x: np.ndarray, signed: bool):
    """Block-wise quantisation of a flat fp32 array to the 8-bit dynamic type.
    Per block of 2048: M = max |x|; n = fl32(x / M); the magnitude index is the
    number of midpoints between neighbouring magnitudes that |n| exceeds (so the
    nearest magnitude, the smaller one on a tie); the sign goes to bit 7 (signed
    type, never set for a zero magnitude).  Returns (codes uint8 [n], absmax fp32)."""
    x = np.ascontiguousarray(x, dtype=np.float32).reshape(-1)
    n_el = x.size
    nb = (n_el + OPT8_BLOCK - 1) // OPT8_BLOCK
    c = dyn8_codebook(signed).astype(np.float64)
    mid = (c[:-1] + c[1:]) / 2.0
    codes = np.zeros(n_el, dtype=np.uint8)
    absmax = np.zeros(nb, dtype=np.float32)
    for b in range(nb):
        blk = x[b * OPT8_BLOCK : (b + 1) * OPT8_BLOCK]
        M = np.float32(np.max(np.abs(blk)))
        absmax[b] = M
        if not M > 0:
            continue
        n = (blk / M).astype(np.float32).astype(np.float64)
        idx = np.searchsorted(mid, np.abs(n), side="left").astype(np.uint8)  # count of midpoints strictly below |n|
        if signed:
            idx = np.where((n < 0) & (idx > 0), idx | 0x80, idx).astype(np.uint8)
        codes[b * OPT8_BLOCK : b * OPT8_BLOCK + blk.size] = idx
    return codes, absmax


def dyn8_dequantize(codes: np.ndarray, absmax: np.ndarray, signed: bool) -> np.ndarray:
    """x' = fl32( magnitude[code] * M ), negated when the sign bit is set."""
    codes = np.asarray(codes, dtype=np.uint8).reshape(-1)
    c = dyn8_codebook(signed)
    M = np.repeat(np.asarray(absmax, dtype=np.float32), OPT8_BLOCK)[: codes.size]
    if signed:
        mag = (c[codes & 0x7F] * M).astype(np.float32)
        return np.where(codes & 0x80, -mag, mag).astype(np.float32)
    return (c[codes] * M).astype(np.float32)


def adam8_step(B, g, m8, m_absmax, v8, v_absmax, step, lr, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0):
    """One Adam step on B (see adam_step) with the moments held in 8 bits: they are
    dequantised, updated with the gradient, used for the step on B, and quantised
    again.  B: bf16 values [r, in]; g: fp32 [r, in]; m8, v8: uint8 [r * in] codes of
    the row-major flattened moments with one fp32 scale per 2048 elements.
    Evaluated in float64 from the fp32 dequantised moments; B is rounded once to
    bf16, the new moments once to fp32 before quantisation.
    Returns (B, m8, m_absmax, v8, v_absmax)."""
    shape = np.asarray(B).shape
    m = dyn8_dequantize(m8, m_absmax, True).astype(np.float64).reshape(shape)
    v = dyn8_dequantize(v8, v_absmax, False).astype(np.float64).reshape(shape)
    B64 = np.asarray(B, dtype=np.float64)
    g64 = np.asarray(g, dtype=np.float32).astype(np.float64)
    m64 = beta1 * m + (1.0 - beta1) * g64
    v64 = beta2 * v + (1.0 - beta2) * g64 * g64
    mhat = m64 / (1.0 - beta1 ** step)
    vhat = v64 / (1.0 - beta2 ** step)
    Bn = B64 - lr * (mhat / (np.sqrt(vhat) + eps) + weight_decay * B64)
    mq = dyn8_quantize(m64.astype(np.float32).reshape(-1), True)
    vq = dyn8_quantize(v64.astype(np.float32).reshape(-1), False)
    return bf16_round(Bn.astype(np.float32)), mq[0], mq[1], vq[0], vq[1]


# ----------------------------------------------------------------------------
# The projection P from the full-rank gradient  (Section 2, first paragraph, and
# Algorithm 2, the SVD lines: P = the first r columns of U in G^W = U S V^T)
# ----------------------------------------------------------------------------
def top_r_left_subspace(G: np.ndarray, r: int) -> np.ndarray:
    """The definition: the r left singular vectors of G with the largest singular
    values, as the columns of an out x r matrix (numpy's SVD, float64).  Only the
    spanned subspace is unique (signs, and rotations inside groups of equal
    singular values, are not)."""
    U, _, _ = np.linalg.svd(np.asarray(G, dtype=np.float64), full_matrices=False)
    return U[:, :r]


def subspace_iteration(G: np.ndarray, Omega: np.ndarray, iters: int) -> np.ndarray:
    """An approximation of that subspace by randomised subspace iteration (Halko,
    Martinsson and Tropp, "Finding structure with randomness", Algorithm 4.4),
    the route a GPU takes because it consists of matrix products and the
    orthonormalisation of tall thin matrices:

        Q = orth(G Omega);  repeat iters times:  Z = orth(G^T Q);  Q = orth(G Z)

    Omega: in x r test matrix (the random numbers are an input).  orth() is the Q
    factor of numpy's QR.  float64 throughout.  Returns Q, out x r with orthonormal
    columns; its span tends to the top-r left singular subspace as iters grows, at
    the rate (sigma_{r+1} / sigma_r)^(2 iters + 1)."""
    G = np.asarray(G, dtype=np.float64)
    Q, _ = np.linalg.qr(G @ np.asarray(Omega, dtype=np.float64))
    for _ in range(int(iters)):
        Z, _ = np.linalg.qr(G.T @ Q)
        Q, _ = np.linalg.qr(G @ Z)
    return Q


def top_r_right_subspace(G: np.ndarray, r: int) -> np.ndarray:
    """The right-side counterpart (Section 2.1: a matrix with more rows than columns is
    projected from the right): the r right singular vectors of G with the largest singular
    values, as the rows of an r x in matrix (numpy's SVD, float64)."""
    _, _, Vt = np.linalg.svd(np.asarray(G, dtype=np.float64), full_matrices=False)
    return Vt[:r, :]


def subspace_iteration_right(G: np.ndarray, Omega: np.ndarray, iters: int) -> np.ndarray:
    """Randomised subspace iteration for the right singular subspace:

        Q = orth(G^T Omega);  repeat iters times:  Z = orth(G Q);  Q = orth(G^T Z)

    Omega: out x r test matrix.  Returns Q^T, r x in with orthonormal rows."""
    G = np.asarray(G, dtype=np.float64)
    Q, _ = np.linalg.qr(G.T @ np.asarray(Omega, dtype=np.float64))
    for _ in range(int(iters)):
        Z, _ = np.linalg.qr(G @ Q)
        Q, _ = np.linalg.qr(G.T @ Z)
    return Q.T


def subspace_sines(P: np.ndarray, Q: np.ndarray) -> np.ndarray:
    """Sines of the principal angles between the column spaces of P and Q (both
    with orthonormal columns): the singular values of (I - P P^T) Q."""
    P = np.asarray(P, dtype=np.float64)
    Q = np.asarray(Q, dtype=np.float64)
    return np.linalg.svd(Q - P @ (P.T @ Q), compute_uv=False)
