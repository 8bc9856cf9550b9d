#!/usr/bin/env python
"""Benchmark of the LoQT quantized low-rank linear hot path on B200.

One step = one pass of the whole hot path over one batch of synthetic input:
forward + backward of every projection matrix of a Llama-shaped layer set, then
one merge + requantise of all of them.  Prints one JSON line (rank 0).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config 0..4]
  python bench.py --impl reference ...      # times the CPU oracle instead

With N > 1 (launched by torch.distributed.run) every rank runs an independent
replica of the layer set (the path has no exchange step); the reported value is
the sum over ranks divided by the slowest rank's time.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "LoQT linear fwd+bwd TFLOP/s & % bf16 tensor peak; merge_requant GB/s % HBM"


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {
            "hbm_gbs": float(p["hbm_gbs"]),
            "bf16_tflops": float(p["bf16_tflops"]),
            "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
            "source": "measured",
        }
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# --------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while a region runs."""

    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        try:
            rows = [l.strip().split(", ") for l in open(self.path) if l.strip()]
            os.unlink(self.path)
            sm = sorted(float(r[1]) for r in rows if len(r) >= 9)
            if sm:
                out["sm_mhz"] = sm[len(sm) // 2]
                out["sm_max_mhz"] = float(rows[0][2])
                out["power_w_max"] = max(float(r[3]) for r in rows if len(r) >= 9)
                names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
                for i, n in enumerate(names):
                    if any(r[5 + i].strip().lower() == "active" for r in rows if len(r) >= 9):
                        out["reasons"].append(n)
                out["samples"] = len(sm)
        except Exception:
            pass
        return out


# --------------------------------------------------------------------------- workload
def build_model(cfg, seed, device):
    """All projection matrices of the layer set, quantised on the device, plus
    per-matrix activations.  Returns a list of dicts (one per matrix)."""
    import torch

    from paper_2405_16528_b200 import binding as L
    from paper_2405_16528_b200 import synth

    mats = []
    for layer in range(cfg.layers):
        for label, out, inn, count in cfg.shapes():
            for j in range(count):
                name = (cfg.name, layer, label, j)
                W = synth.normal(seed, name + ("W",), (out, inn), 0.02, torch.float32, device)
                P = synth.orthonormal(seed, name + ("P",), out, cfg.r, device)
                m = {
                    "out": out, "in": inn, "label": label,
                    "Wq": L.loqt_nf4_quantize(W), "Pq": L.loqt_nf4_quantize(P),
                    "B": synth.normal(seed, name + ("B",), (cfg.r, inn), cfg.sigma_B, torch.bfloat16, device),
                    "x": synth.normal(seed, name + ("x",), (cfg.T, inn), 1.0, torch.bfloat16, device),
                    "dy": synth.normal(seed, name + ("dy",), (cfg.T, out), 1.0, torch.bfloat16, device),
                }
                del W, P
                mats.append(m)
    return mats


def pad8(n):
    return (n + 7) // 8 * 8


def alloc_outputs(cfg, mats, device):
    """Output buffers shared by all matrices of a shape (overwritten every call)."""
    import torch

    from paper_2405_16528_b200 import binding as L

    bufs = {}
    ws_bytes = 256
    for m in mats:
        key = (m["out"], m["in"])
        if key not in bufs:
            bufs[key] = {
                "y": torch.empty((cfg.T, pad8(m["out"])), dtype=torch.bfloat16, device=device)[:, : m["out"]],
                "dx": torch.empty((cfg.T, pad8(m["in"])), dtype=torch.bfloat16, device=device)[:, : m["in"]],
                "dB": torch.empty((cfg.r, m["in"]), dtype=torch.float32, device=device),
            }
        ws_bytes = max(ws_bytes, L.loqt_workspace_bytes(L.LOQT_OP_FWD, m["out"], m["in"], cfg.r, cfg.T),
                       L.loqt_workspace_bytes(L.LOQT_OP_BWD, m["out"], m["in"], cfg.r, cfg.T),
                       256 + min(8, len(mats)) * (L.loqt_workspace_bytes(L.LOQT_OP_MERGE, m["out"], m["in"], cfg.r, 0) - 256))
    return bufs, L.new_workspace(ws_bytes, device)


def pad_rows(t):
    """Row stride a multiple of 8 elements (16 bytes), as the library requires."""
    import torch

    rows, cols = t.shape
    if cols % 8 == 0:
        return t
    buf = torch.zeros((rows, pad8(cols)), dtype=t.dtype, device=t.device)
    buf[:, :cols] = t
    return buf[:, :cols]


def time_nf4_kernels(device, peaks, rows=16384, cols=8192, iters=10):
    """The streaming kernels on a matrix whose every stream exceeds twice the L2
    (fp32 source 537 MB, bf16 output 268 MB; an output of about the L2 size runs
    at half speed even for a plain fill):
    achieved GB/s on their algorithmic bytes (quantise 4 + 0.5625 B/element,
    dequantise to bf16 0.5625 + 2 B/element, requantise 4 + 1.125 B/element) against
    the measured HBM copy rate."""
    import torch

    from paper_2405_16528_b200 import binding as L

    w = torch.randn((rows, cols), device=device, dtype=torch.float32) * 0.02
    q = L.NF4Tensor.empty(rows, cols, device)
    out = torch.empty((rows, cols), device=device, dtype=torch.bfloat16)

    def timed(fn):
        for _ in range(3):
            fn()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(iters):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / iters

    n = rows * cols
    ms_q = timed(lambda: L.loqt_nf4_quantize(w, q))
    ms_d = timed(lambda: L.loqt_nf4_dequantize(q, dst=out))
    # the streaming half of the two-pass merge: W_q <- q(deq(W_q) + delta), 4 + 2 * 0.5625 B/element
    w.mul_(0.05)
    ms_r = timed(lambda: L.loqt_nf4_requantize(w, 1.0, q))
    gq = n * 4.5625 / (ms_q * 1e-3) / 1e9
    gd = n * 2.5625 / (ms_d * 1e-3) / 1e9
    gr = n * 5.125 / (ms_r * 1e-3) / 1e9
    return {
        "shape": [rows, cols],
        "quantize_gb_s": round(gq, 1), "quantize_pct_hbm": round(100 * gq / peaks["hbm_gbs"], 1),
        "dequantize_bf16_gb_s": round(gd, 1), "dequantize_pct_hbm": round(100 * gd / peaks["hbm_gbs"], 1),
        "requantize_gb_s": round(gr, 1), "requantize_pct_hbm": round(100 * gr / peaks["hbm_gbs"], 1),
        "of": peaks["source"],
    }


def time_adam_step(device, peaks, rows=16384, cols=8192, iters=10):
    """The fused optimiser step on a factor larger than L2: 4 (gradient) + 3 x (2 + 2)
    (B and the two bf16 moments, read and written) = 16 bytes per element."""
    import torch

    from paper_2405_16528_b200 import binding as L

    B = torch.randn((rows, cols), device=device, dtype=torch.float32).mul_(1e-2).to(torch.bfloat16)
    g = torch.randn((rows, cols), device=device, dtype=torch.float32).mul_(1e-3)
    m, v = torch.zeros_like(B), torch.zeros_like(B)
    for step in range(1, 4):
        L.loqt_adam_step(B, g, m, v, step, 1e-3)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(iters):
        L.loqt_adam_step(B, g, m, v, 4 + i, 1e-3)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / iters
    gbs = rows * cols * 16 / (ms * 1e-3) / 1e9
    return {"shape": [rows, cols], "ms": round(ms, 4), "gb_s": round(gbs, 1), "pct_hbm": round(100 * gbs / peaks["hbm_gbs"], 1),
            "of": peaks["source"]}


def time_compensated_init(device, peaks, cfg, seed, steps=5, iters=5):
    """Error-compensated initialisation (Section 2.5) of one matrix of the
    configuration's first shape: `steps` rounds of quantise + residual, B = P^T residual
    and W - P B.  Flops counted: (2 steps - 1) products of 2 out in r."""
    import torch

    from paper_2405_16528_b200 import binding as L
    from paper_2405_16528_b200 import synth

    _, out, inn, _ = next(iter(cfg.shapes()))
    r = cfg.r
    W = synth.normal(seed, ("ci", "W"), (out, inn), 0.02, torch.float32, device)
    P = synth.orthonormal(seed, ("ci", "P"), out, r, device)
    ws = L.new_workspace(L.loqt_workspace_bytes(L.LOQT_OP_COMPENSATE, out, inn, r, 0), device)
    for _ in range(2):
        L.loqt_compensated_init(W, P, steps, ws=ws)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        L.loqt_compensated_init(W, P, steps, ws=ws)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / iters
    flops = (2 * steps - 1) * 2.0 * out * inn * r
    tf = flops / (ms * 1e-3) / 1e12
    return {
        "shape": [out, inn], "r": r, "steps": steps, "ms": round(ms, 4), "tflops": round(tf, 1),
        "pct_bf16_peak_burst": round(100 * tf / peaks["bf16_tflops"], 1), "of": peaks["source"],
    }


def time_projection(device, peaks, cfg, seed, iters=2, reps=3):
    """The projection step (Algorithm 2, SVD lines) for one matrix of the configuration's first shape:
    randomised subspace iteration with `iters` rounds from a Gaussian test matrix.  Work counted: the
    2 iters + 1 products of 2 out in r flops (tensor cores) and, per orthonormalisation, m r^2 (Gram, lower
    half) + r^3 / 3 (Cholesky) + m r^2 (triangular solve) double-precision flops."""
    import torch

    from paper_2405_16528_b200 import binding as L
    from paper_2405_16528_b200 import synth

    _, out, inn, _ = next(iter(cfg.shapes()))
    r = cfg.r
    G = synth.normal(seed, ("pj", "G"), (out, inn), 1.0, torch.float32, device)
    Om = synth.normal(seed, ("pj", "Omega"), (inn, r), 1.0, torch.bfloat16, device)
    P = torch.empty((out, r), dtype=torch.float32, device=device)
    ws = L.new_workspace(L.loqt_workspace_bytes(L.LOQT_OP_PROJECTION, out, inn, r, 0), device)
    for _ in range(2):
        L.loqt_projection(G, Om, iters, P=P, ws=ws)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        L.loqt_projection(G, Om, iters, P=P, ws=ws)
    e1.record()
    torch.cuda.synchronize()
    L.loqt_device_status(ws)
    ms = e0.elapsed_time(e1) / reps
    f64 = sum(2.0 * m * r * r + r ** 3 / 3.0 for m in [out] + [inn, out] * iters)
    return {"shape": [out, inn], "r": r, "iters": iters, "ms": round(ms, 3),
            "product_tflops_bf16": round((2 * iters + 1) * 2.0 * out * inn * r / 1e12, 4),
            "orth_gflops_f64": round(f64 / 1e9, 2), "orth_f64_tflops_if_all_time": round(f64 / (ms * 1e-3) / 1e12, 2)}


def run_per_shape(args):
    """Diagnostic: median time of forward, backward and merge for one matrix of
    each distinct shape of the configuration, L2 flushed between calls."""
    import torch

    from paper_2405_16528_b200 import binding as L
    from paper_2405_16528_b200 import build, synth

    build.build()
    torch.cuda.set_device(0)
    cfg = synth.CONFIGS[args.config]
    r, T = cfg.r, cfg.T
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")

    def timeit(fn, n=7):
        ts = []
        for i in range(n + 2):
            flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            torch.cuda.synchronize()
            if i >= 2:
                ts.append(e0.elapsed_time(e1))
        return sorted(ts)[len(ts) // 2]

    res = {}
    for _, out, inn, _ in cfg.shapes():
        d = synth.make_layer(args.seed, ("shape", out, inn), out, inn, r, cfg.sigma_B, T, device="cuda")
        Wq, Pq = L.loqt_nf4_quantize(d["W"]), L.loqt_nf4_quantize(d["P"])
        B, x, dy = pad_rows(d["B"]), pad_rows(d["x"]), pad_rows(d["dy"])
        y = torch.empty((T, pad8(out)), dtype=torch.bfloat16, device="cuda")[:, :out]
        dx = torch.empty((T, pad8(inn)), dtype=torch.bfloat16, device="cuda")[:, :inn]
        dB = torch.empty((r, inn), dtype=torch.float32, device="cuda")
        ws = L.new_workspace(max(L.loqt_workspace_bytes(L.LOQT_OP_BWD, out, inn, r, T),
                                 L.loqt_workspace_bytes(L.LOQT_OP_MERGE_SPLIT, out, inn, r, 0)))
        tf = timeit(lambda: L.loqt_linear_fwd(Wq, Pq, B, 1.0, x, y=y, ws=ws))
        tb = timeit(lambda: L.loqt_linear_bwd(Wq, Pq, B, 1.0, x, dy, dx=dx, dB=dB, ws=ws))
        Wc = Wq.clone()
        tm = timeit(lambda: L.loqt_merge_requant(Wc, Pq, B, 1.0, ws=ws))
        ts = timeit(lambda: L.loqt_merge_requant_split(Wc, Pq, B, 1.0, ws=ws))
        # the streaming half alone: read delta (fp32) + codes + scales, write codes + scales
        delta = torch.randn((out, Wq.ld), dtype=torch.float32, device="cuda")[:, :inn] * 1e-3
        tr = timeit(lambda: L.loqt_nf4_requantize(delta, 1.0, Wc))
        requant_bytes = out * inn * 4 + 2 * synth.nf4_bytes(out, inn)
        right = {}
        if out > inn:
            # the right-side variant the paper prescribes for tall matrices: Q is r x in, B out x r
            Qq = L.loqt_nf4_quantize(synth.orthonormal(args.seed, ("Q", out, inn), inn, r, "cuda").T.contiguous())
            Br = synth.normal(args.seed, ("Br", out, inn), (out, r), cfg.sigma_B, torch.bfloat16, "cuda")
            trf = timeit(lambda: L.loqt_linear_fwd_right(Wq, Qq, Br, 1.0, x))
            trb = timeit(lambda: L.loqt_linear_bwd_right(Wq, Qq, Br, 1.0, x, dy))
            trm = timeit(lambda: L.loqt_merge_requant_right(Wc, Qq, Br, 1.0))
            flops_r = 4.0 * T * inn * out + 2.0 * T * r * (2 * inn + 3 * out)
            right = {"right_fwd_ms": round(trf, 4), "right_bwd_ms": round(trb, 4), "right_merge_ms": round(trm, 4),
                     "right_fwdbwd_tflops": round(flops_r / (trf + trb) / 1e9, 1)}
        L.loqt_device_status(ws)
        res[f"{out}x{inn}"] = {
            "fwd_ms": round(tf, 4), "bwd_ms": round(tb, 4), "merge_ms": round(tm, 4), "merge_split_ms": round(ts, 4),
            "fwdbwd_tflops": round(synth.fwd_bwd_flops(out, inn, r, T) / (tf + tb) / 1e9, 1),
            "merge_gb_s": round(synth.merge_bytes(out, inn, r) / tm / 1e6, 1),
            "requant_stage_ms": round(tr, 4), "requant_stage_gb_s": round(requant_bytes / tr / 1e6, 1),
            **right,
        }
    print(json.dumps({"per_shape": res, "config": cfg.name}), flush=True)


def measure_config(args, ci, rank, world, local_rank, dist, device, e2e=True):
    """Builds the layer set of configuration `ci` on this rank's GPU, runs W warm-up
    steps and K timed steps (fwd+bwd of every matrix, then one merge of all), and
    returns the timings (max over ranks) with the clocks sampled meanwhile."""
    import torch

    from paper_2405_16528_b200 import binding as L
    from paper_2405_16528_b200 import synth

    cfg = synth.CONFIGS[ci]
    if args.layers > 0:
        import dataclasses

        cfg = dataclasses.replace(cfg, layers=args.layers, name=f"{cfg.name}[{args.layers} layer(s)]")
    s = 1.0
    mats = build_model(cfg, args.seed + rank, device)
    for m in mats:
        for k in ("B", "x", "dy"):
            m[k] = pad_rows(m[k])
    bufs, ws = alloc_outputs(cfg, mats, device)
    flops_step = sum(synth.fwd_bwd_flops(m["out"], m["in"], cfg.r, cfg.T) for m in mats)
    merge_bytes_step = sum(synth.merge_bytes(m["out"], m["in"], cfg.r) for m in mats)
    merge_flops_step = sum(2 * m["out"] * m["in"] * cfg.r for m in mats)

    def fwd_bwd():
        for m in mats:
            b = bufs[(m["out"], m["in"])]
            L.loqt_linear_fwd(m["Wq"], m["Pq"], m["B"], s, m["x"], y=b["y"], ws=ws)
            L.loqt_linear_bwd(m["Wq"], m["Pq"], m["B"], s, m["x"], m["dy"], dx=b["dx"], dB=b["dB"], ws=ws)

    Wqs, Pqs, Bs = [m["Wq"] for m in mats], [m["Pq"] for m in mats], [m["B"] for m in mats]

    def merge():
        L.loqt_merge_requant_many(Wqs, Pqs, Bs, s, ws=ws)

    def sync():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(args.warmup):
        fwd_bwd()
        merge()
    sync()
    L.loqt_device_status(ws)

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    launches0 = L.loqt_launch_count()
    sync()
    t_wall0 = time.perf_counter()
    for k in range(args.steps):
        ev[k][0].record()
        fwd_bwd()
        ev[k][1].record()
        merge()
        ev[k][2].record()
    sync()
    t_wall = time.perf_counter() - t_wall0
    launches = L.loqt_launch_count() - launches0
    clocks = sampler.stop() if rank == 0 else None
    L.loqt_device_status(ws)

    ms_fb = sum(e[0].elapsed_time(e[1]) for e in ev) / args.steps
    ms_mg = sum(e[1].elapsed_time(e[2]) for e in ev) / args.steps
    ms_step = sum(e[0].elapsed_time(e[2]) for e in ev) / args.steps

    # ---- end to end through the public API with HOST buffers: every step the activations x and the
    # output gradients dy of every matrix come from pinned host memory, the gradient of the trained
    # factor goes back to the host, and the merge of all matrices closes the step.  y and dx stay on
    # the device (in a training step they feed the neighbouring layers there).
    ms_e2e, h2d, d2h, e2e_steps = 0.0, 0, 0, 0
    if e2e:
        e2e_steps = max(1, min(args.steps, 2))
        shapes = {}
        for m in mats:
            key = (m["out"], m["in"])
            if key not in shapes:
                shapes[key] = {
                    "hx": torch.empty((cfg.T, m["x"].stride(0)), dtype=torch.bfloat16).pin_memory(),
                    "hdy": torch.empty((cfg.T, m["dy"].stride(0)), dtype=torch.bfloat16).pin_memory(),
                    "hdB": torch.empty((cfg.r, m["in"]), dtype=torch.float32).pin_memory(),
                    "dxin": torch.empty((cfg.T, m["x"].stride(0)), dtype=torch.bfloat16, device=device),
                    "ddy": torch.empty((cfg.T, m["dy"].stride(0)), dtype=torch.bfloat16, device=device),
                }
                shapes[key]["hx"].normal_()
                shapes[key]["hdy"].normal_()
        for m in mats:
            sh = shapes[(m["out"], m["in"])]
            h2d += sh["hx"].numel() * 2 + sh["hdy"].numel() * 2
            d2h += sh["hdB"].numel() * 4

        # Copies and kernels run on three streams: the activations of the next matrix arrive
        # (copy stream, two staging slots per shape) while the current one is computed, and dB
        # leaves (second copy stream, two dB buffers per shape) while the next one is computed.
        main = torch.cuda.current_stream()
        s_in, s_out = torch.cuda.Stream(device=device), torch.cuda.Stream(device=device)
        for sh in shapes.values():
            sh["slots"] = [
                {"dxin": torch.empty_like(sh["dxin"]), "ddy": torch.empty_like(sh["ddy"]),
                 "dB": torch.empty((cfg.r, sh["hdB"].shape[1]), dtype=torch.float32, device=device),
                 "free": None, "drained": None}
                for _ in range(2)]
            sh["next"] = 0

        def e2e_step():
            for m in mats:
                sh = shapes[(m["out"], m["in"])]
                b = bufs[(m["out"], m["in"])]
                slot = sh["slots"][sh["next"]]
                sh["next"] ^= 1
                with torch.cuda.stream(s_in):
                    if slot["free"] is not None:
                        s_in.wait_event(slot["free"])      # the kernels that last read this slot are done
                    slot["dxin"].copy_(sh["hx"], non_blocking=True)
                    slot["ddy"].copy_(sh["hdy"], non_blocking=True)
                    arrived = torch.cuda.Event()
                    arrived.record(s_in)
                main.wait_event(arrived)
                if slot["drained"] is not None:
                    main.wait_event(slot["drained"])       # this slot's previous dB has left
                xin = slot["dxin"][:, : m["in"]]
                dyin = slot["ddy"][:, : m["out"]]
                L.loqt_linear_fwd(m["Wq"], m["Pq"], m["B"], s, xin, y=b["y"], ws=ws)
                L.loqt_linear_bwd(m["Wq"], m["Pq"], m["B"], s, xin, dyin, dx=b["dx"], dB=slot["dB"], ws=ws)
                slot["free"] = torch.cuda.Event()
                slot["free"].record(main)
                with torch.cuda.stream(s_out):
                    s_out.wait_event(slot["free"])
                    sh["hdB"].copy_(slot["dB"], non_blocking=True)
                    slot["drained"] = torch.cuda.Event()
                    slot["drained"].record(s_out)
            merge()
            main.wait_stream(s_out)
            main.wait_stream(s_in)

        e2e_step()
        sync()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(e2e_steps):
            e2e_step()
        e1.record()
        sync()
        ms_e2e = e0.elapsed_time(e1) / e2e_steps
        del shapes

    times = torch.tensor([ms_fb, ms_mg, ms_step, ms_e2e], dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(times, op=dist.ReduceOp.MAX)
    ms_fb, ms_mg, ms_step, ms_e2e = [float(v) for v in times.cpu()]
    out = {
        "cfg": cfg, "n_mats": len(mats), "flops_step": flops_step, "merge_bytes_step": merge_bytes_step,
        "merge_flops_step": merge_flops_step, "ms_fb": ms_fb, "ms_mg": ms_mg, "ms_step": ms_step, "ms_e2e": ms_e2e,
        "h2d": h2d, "d2h": d2h, "e2e_steps": e2e_steps, "launches": int(launches), "clocks": clocks, "t_wall": t_wall, "s": s,
    }
    del mats, bufs, ws, Wqs, Pqs, Bs
    torch.cuda.empty_cache()
    return out


def merge_report(m, world, peaks):
    """The merge of one measured configuration: GB/s on its algorithmic bytes (read and
    write W_q, read P_q, read B), the TFLOP/s of its product, and the share of the roof
    that binds it, max(tensor time, HBM time)."""
    gbs = world * m["merge_bytes_step"] / (m["ms_mg"] * 1e-3) / 1e9
    tf = world * m["merge_flops_step"] / (m["ms_mg"] * 1e-3) / 1e12
    t_tensor = m["merge_flops_step"] / (peaks["bf16_tflops_sustained"] * 1e12)
    t_hbm = m["merge_bytes_step"] / (peaks["hbm_gbs"] * 1e9)
    return {
        "ms": round(m["ms_mg"], 3),
        "gb_s": round(gbs, 1),
        "pct_hbm": round(100 * gbs / world / peaks["hbm_gbs"], 2),
        "gemm_tflops": round(tf, 1),
        "binding_roof": "tensor" if t_tensor >= t_hbm else "hbm",
        "pct_of_binding_roof": round(100 * max(t_tensor, t_hbm) / (m["ms_mg"] * 1e-3), 2),
        "bytes_per_step": m["merge_bytes_step"],
    }


# DRAM read + write bytes of the forward/backward launches (u, y, v, dx, dB) of ONE attention-shaped
# matrix, from the ncu capture summarised in profiles/ (None where no capture of the current kernels exists).
NCU_TRAFFIC = {
    4: {"bytes": 285.3e6,
        "of": "sum of dram__bytes_read + dram__bytes_write over the five product launches (u, y, v, dx, dB) of one 4096x4096 matrix, "
              "r=1024, T=4096 (profiles/loqt_gemm_kernel_llama7b_attention.md); algorithmic bytes of the same launches 338.4e6"},
    3: {"bytes": 215.1e6,
        "of": "the same for one 2048x2048 matrix, r=512, T=8192 (profiles/loqt_gemm_kernel_llama1b_attention.md); algorithmic 293e6"},
}


def run_ours(args, rank, world, local_rank):
    import torch

    from paper_2405_16528_b200 import binding as L
    from paper_2405_16528_b200 import build, synth

    build.build()
    L.lib()  # fails loudly when the CUDA library is missing
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod

        dist = dist_mod
        dist.init_process_group("nccl", device_id=device)

    main = measure_config(args, args.config, rank, world, local_rank, dist, device)
    # the second spec shape set (Llama-1B: odd MLP width 5461, r = 512, T = 8192) in the same run
    extra = {}
    for ci in args.also:
        if ci != args.config:
            extra[ci] = measure_config(args, ci, rank, world, local_rank, dist, device, e2e=False)

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peaks = load_peaks()
    cfg = main["cfg"]
    nf4 = time_nf4_kernels(device, peaks)
    nf4_large = time_nf4_kernels(device, peaks, rows=65536, cols=8192, iters=5)
    comp = time_compensated_init(device, peaks, cfg, args.seed)
    adam = time_adam_step(device, peaks)
    proj = time_projection(device, peaks, cfg, args.seed)
    tflops = world * main["flops_step"] / (main["ms_fb"] * 1e-3) / 1e12
    per_gpu_tflops = tflops / world
    traffic = NCU_TRAFFIC.get(args.config, {"bytes": None, "of": "no capture for this configuration"})
    result = {
        "metric": METRIC,
        "value": round(tflops, 2),
        "unit": "TFLOP/s (fwd+bwd, algorithmic flops of the factored layer)",
        "n_gpus": world,
        "steps": args.steps,
        "warmup": args.warmup,
        "ms_per_step": round(main["ms_step"], 3),
        "ms_fwd_bwd": round(main["ms_fb"], 3),
        "ms_merge": round(main["ms_mg"], 3),
        "higher_is_better": True,
        "scaling": "weak",
        "vs_baseline": None,
        "dtype": "bf16 x bf16 -> fp32 (NF4 weights)",
        "data": "synthetic",
        "config": {
            "workload": f"configs[{args.config}] {cfg.name}: {main['n_mats']} projection matrices, r={cfg.r}, T={cfg.T}",
            "step": "fwd+bwd of every matrix, then merge_requant of all",
            "l2": "inputs larger than L2: every matrix has its own weights and activations",
            "replicas": world,
            "s": main["s"],
        },
        "pct_bf16_peak": {
            "burst": round(100 * per_gpu_tflops / peaks["bf16_tflops"], 2),
            "sustained": round(100 * per_gpu_tflops / peaks["bf16_tflops_sustained"], 2),
            "of": peaks["source"],
        },
        "merge_requant": merge_report(main, world, peaks),
        "roofline": {
            "kernel": "loqt_gemm_kernel (fused NF4-dequant tcgen05 GEMM; all fwd+bwd launches)",
            "bound": "tensor",
            "achieved": round(per_gpu_tflops, 2),
            "peak": peaks["bf16_tflops_sustained"],
            "unit": "TFLOP/s",
            "frac": round(per_gpu_tflops / peaks["bf16_tflops_sustained"], 4),
            "peak_kind": f"sustained, of {peaks['source']}",
            "traffic": traffic["bytes"],
            "traffic_of": traffic["of"],
        },
        "e2e": {
            "value": round(world * main["flops_step"] / (main["ms_e2e"] * 1e-3) / 1e12, 2),
            "unit": "TFLOP/s",
            "h2d_bytes_per_step": main["h2d"],
            "d2h_bytes_per_step": main["d2h"],
            "steps": main["e2e_steps"],
            "region": "H2D of x and dy of every matrix from pinned memory, fwd, bwd, D2H of dB, then the merge of all matrices; copies on their own streams, overlapped with the kernels",
            "left_out": "y and dx are not copied back: they stay on the device for the neighbouring layers",
        },
        "configs": {},
        "nf4_stream": nf4,
        "nf4_stream_large": nf4_large,
        "compensated_init": comp,
        "adam_step": adam,
        "projection": proj,
        "gpu_launches": main["launches"],
        "clocks": main["clocks"],
        "wall_s_timed": round(main["t_wall"], 3),
    }
    for ci, m in extra.items():
        tf = m["flops_step"] / (m["ms_fb"] * 1e-3) / 1e12  # per GPU
        result["configs"][str(ci)] = {
            "workload": f"configs[{ci}] {m['cfg'].name}: {m['n_mats']} projection matrices, r={m['cfg'].r}, T={m['cfg'].T}",
            "tflops": round(world * tf, 2),
            "ms_fwd_bwd": round(m["ms_fb"], 3),
            "pct_bf16_peak": {"burst": round(100 * tf / peaks["bf16_tflops"], 2),
                              "sustained": round(100 * tf / peaks["bf16_tflops_sustained"], 2), "of": peaks["source"]},
            "merge_requant": merge_report(m, world, peaks),
            "gpu_launches": m["launches"],
            "clocks": m["clocks"],
            "roofline_traffic": NCU_TRAFFIC.get(ci, {"bytes": None})["bytes"],
        }
    if not args.no_cpu_baseline and world == 1:
        result["cpu_baseline"] = cpu_baseline(cfg, args.seed)
    print(json.dumps(result), flush=True)
    if dist is not None:
        dist.destroy_process_group()


# --------------------------------------------------------------------------- oracle timing
def oracle_sample(cfg, seed, T_sample, shapes=None):
    """Forward + backward of one matrix per listed (out, in) shape of `cfg`
    (default: the attention shape) through the CPU oracle on T_sample tokens.
    Returns (seconds, algorithmic flops)."""
    import torch

    from oracle import loqt_oracle as O
    from paper_2405_16528_b200 import synth

    shapes = shapes or [(cfg.hidden, cfg.hidden)]
    dt = 0.0
    flops = 0
    for out, inn in shapes:
        d = synth.make_layer(seed, ("cpu", out, inn), out, inn, cfg.r, cfg.sigma_B, T_sample)
        wq, pq = O.nf4_quantize(d["W"].numpy()), O.nf4_quantize(d["P"].numpy())
        f = lambda t: t.to(torch.float32).numpy()
        B, x, dy = f(d["B"]), f(d["x"]), f(d["dy"])
        t0 = time.perf_counter()
        O.loqt_forward(wq, pq, B, 1.0, x, (out, inn, cfg.r))
        O.loqt_backward(wq, pq, B, 1.0, x, dy, (out, inn, cfg.r))
        dt += time.perf_counter() - t0
        flops += synth.fwd_bwd_flops(out, inn, cfg.r, T_sample)
    return dt, flops


def blas_threads():
    try:
        from threadpoolctl import threadpool_info

        n = [p.get("num_threads", 0) for p in threadpool_info() if p.get("user_api") == "blas"]
        if n:
            return max(n)
    except Exception:
        pass
    return os.cpu_count() or 1


def cpu_baseline(cfg, seed):
    shapes = [(o, i) for _, o, i, _ in cfg.shapes()]
    dt, flops = oracle_sample(cfg, seed, cfg.T, shapes)
    return {
        "value": round(flops / dt / 1e12, 5),
        "unit": "TFLOP/s",
        "cores": blas_threads(),
        "kind": "oracle",
        "sample": f"fwd+bwd of one matrix of each of the {len(shapes)} distinct shapes of a layer, all {cfg.T} tokens, fp64, {dt:.2f} s",
    }


def run_reference(args, rank, world):
    if rank != 0:
        return
    from paper_2405_16528_b200 import synth

    cfg = synth.CONFIGS[args.config]
    T_sample = min(cfg.T, 512)
    for _ in range(args.warmup):
        oracle_sample(cfg, args.seed, T_sample)
    tot_t = tot_f = 0.0
    for _ in range(args.steps):
        dt, fl = oracle_sample(cfg, args.seed, T_sample)
        tot_t += dt
        tot_f += fl
    val = tot_f / tot_t / 1e12
    sample = f"per step: fwd+bwd of one {cfg.hidden}x{cfg.hidden} r={cfg.r} matrix on {T_sample} of {cfg.T} tokens, fp64"
    print(json.dumps({
        "impl": "reference",
        "metric": METRIC,
        "value": round(val, 5),
        "unit": "TFLOP/s (fwd+bwd, algorithmic flops of the factored layer)",
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": round(1e3 * tot_t / args.steps, 3),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"configs[{args.config}] {cfg.name} (bounded sample)", "sample": sample},
        "cpu_baseline": {"value": round(val, 5), "unit": "TFLOP/s", "cores": blas_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": round(val, 5), "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=4)
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--layers", type=int, default=0, help="override the layer count (small cases for profiling)")
    ap.add_argument("--also", type=int, nargs="*", default=[3],
                    help="further configurations measured (fwd+bwd and merge) after the main one, reported under \"configs\"")
    ap.add_argument("--per-shape", action="store_true", help="diagnostic: time one matrix of each distinct shape and exit")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.per_shape:
        if rank == 0:
            run_per_shape(args)
    elif args.impl == "reference":
        run_reference(args, rank, world)
    else:
        run_ours(args, rank, world, local_rank)


if __name__ == "__main__":
    main()
