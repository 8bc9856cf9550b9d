"""The N > 1 path of bench.py on CPU: two gloo ranks, each an independent
replica; the reported time is the maximum over ranks and the value sums the
ranks' work (weak scaling, no data-path collective)."""
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

SCRIPT = textwrap.dedent(
    """
    import os, sys, json
    import torch, torch.distributed as dist
    sys.path.insert(0, %r)
    from paper_2405_16528_b200 import synth
    dist.init_process_group("gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    cfg = synth.CONFIGS[0]
    # every rank owns a replica with its own seed: different tensors, same shapes
    w = synth.normal(rank, ("W",), (cfg.hidden, cfg.hidden), 0.02)
    digest = torch.tensor([float(w.double().sum())], dtype=torch.float64)
    gathered = [torch.zeros_like(digest) for _ in range(world)]
    dist.all_gather(gathered, digest)
    ms = torch.tensor([10.0 + 5.0 * rank], dtype=torch.float64)   # this rank's step time
    dist.all_reduce(ms, op=dist.ReduceOp.MAX)
    flops = sum(synth.fwd_bwd_flops(o, i, cfg.r, cfg.T) * c for _, o, i, c in cfg.shapes()) * cfg.layers
    if rank == 0:
        print(json.dumps({"ms": float(ms), "value": world * flops / (float(ms) * 1e-3) / 1e12,
                          "distinct": len({float(g) for g in gathered}), "flops": flops}))
    dist.barrier()
    dist.destroy_process_group()
    """
)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_gloo_ranks_reduce_like_bench(tmp_path):
    script = tmp_path / "ranks.py"
    script.write_text(SCRIPT % ROOT)
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
           "--master-addr", "127.0.0.1", "--master-port", str(_free_port()), str(script)]
    res = subprocess.run(cmd, capture_output=True, text=True, timeout=300)
    assert res.returncode == 0, res.stderr[-2000:]
    import json

    line = [l for l in res.stdout.splitlines() if l.startswith("{")][-1]
    out = json.loads(line)
    assert out["ms"] == 15.0                      # the slower rank sets the time
    assert out["distinct"] == 2                   # replicas are independent
    assert abs(out["value"] - 2 * out["flops"] / 15e-3 / 1e12) < 1e-9


def test_reference_arm_runs_on_rank0_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "0",
                          "--steps", "1", "--warmup", "0"], capture_output=True, text=True, env=env, timeout=300)
    assert res.returncode == 0 and res.stdout.strip() == ""
    env = dict(os.environ, RANK="0", WORLD_SIZE="2", LOCAL_RANK="0")
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "0",
                          "--steps", "1", "--warmup", "0"], capture_output=True, text=True, env=env, timeout=300)
    import json

    out = json.loads(res.stdout.strip().splitlines()[-1])
    assert out["impl"] == "reference" and out["n_gpus"] == 2 and out["e2e"]["h2d_bytes_per_step"] == 0
