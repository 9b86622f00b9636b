"""Multi-GPU layout of the benchmark, checked on CPU with two gloo ranks: the path has no data
exchange (heads and projections are independent), so every rank quantizes its own layer from
its own seed and the only collectives are the barrier and the max-over-ranks time."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys, json
    import numpy as np
    import torch
    import torch.distributed as dist
    sys.path.insert(0, os.environ["TB_ROOT"])
    import bench, tb_inputs
    dist.init_process_group("gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    cfg, proj = bench.workload("tiny")
    W, G, Xb = bench.gen_inputs(cfg, proj, seed=rank, n_tok=256)
    # every rank owns an independent problem: different seeds give different data
    digest = torch.tensor([float(np.abs(W).sum()), float(Xb.astype(np.float64).sum())], dtype=torch.float64)
    gathered = [torch.zeros_like(digest) for _ in range(world)]
    dist.all_gather(gathered, digest)
    # max over ranks of the per-rank time, as bench.py reports it
    t = torch.tensor([10.0 + rank], dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.barrier()
    if rank == 0:
        print(json.dumps({"world": world, "distinct": bool((gathered[0] != gathered[1]).all()),
                          "max_ms": float(t.item()), "value": proj.d_out * world / (float(t.item()) * 1e-3)}))
    dist.destroy_process_group()
""")


def test_two_ranks_own_independent_layers(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, TB_ROOT=ROOT, MASTER_ADDR="127.0.0.1")
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
                          "--master-addr", "127.0.0.1", "--master-port", "29611", str(script)],
                         capture_output=True, text=True, env=env, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    import json
    line = [l for l in out.stdout.splitlines() if l.startswith("{")][-1]
    rec = json.loads(line)
    assert rec["world"] == 2 and rec["distinct"]
    assert rec["max_ms"] == 11.0                      # the slower rank defines the step time
    assert abs(rec["value"] - 256 * 2 / 11e-3) < 1e-6  # whole-job throughput = all ranks' rows / max time


def test_launch_count_formula_is_positive_and_scales():
    import bench
    cfg, proj = bench.workload("l2_7b_q")
    a = bench.count_launches(cfg, proj, 262144)
    assert 100 < a < 2000
