"""Multi-GPU layout of the benchmark, checked on CPU with two gloo ranks: the path has no data
exchange (heads and projections are independent), so every rank quantizes its own layer from
its own seed and the only collectives are the barrier and the max-over-ranks time.  The ranks run
bench.py's own sharding logic (seed per rank, whole-job value from the slowest rank) and its
reference arm under torchrun; the CUDA arm itself must refuse to run without a GPU."""
import json
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
    cfg = tb_inputs.CONFIGS["l3_8b_block"]
    seed = bench.rank_seed(rank)
    # every rank owns an independent layer: the weights and the activation recipe follow its seed
    W = tb_inputs.weight(seed, 64, 128)
    X = tb_inputs.heavy_tail_device(tb_inputs.HeavyTailRecipe(128, seed=seed), 512, torch.device("cpu"), seed)
    digest = torch.tensor([float(np.abs(W).sum()), float(X.float().abs().sum())], dtype=torch.float64)
    gathered = [torch.zeros_like(digest) for _ in range(world)]
    dist.all_gather(gathered, digest)
    # max over ranks of the per-rank step time, then the whole-job value, as bench.main forms them
    t = torch.tensor([10.0 + rank], dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.barrier()
    if rank == 0:
        print(json.dumps({"world": world, "distinct": bool((gathered[0] != gathered[1]).all()),
                          "max_ms": float(t.item()), "value": bench.aggregate_value(cfg, world, float(t.item())),
                          "rows": bench.out_channels(cfg)}))
    dist.destroy_process_group()
""")


def _torchrun(args, port, timeout=600):
    env = dict(os.environ, TB_ROOT=ROOT, MASTER_ADDR="127.0.0.1")
    return subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
                           "--master-addr", "127.0.0.1", "--master-port", str(port)] + args,
                          capture_output=True, text=True, env=env, timeout=timeout, cwd=ROOT)


def test_two_ranks_own_independent_layers(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    out = _torchrun([str(script)], 29611, 300)
    assert out.returncode == 0, out.stderr[-2000:]
    rec = json.loads([ln for ln in out.stdout.splitlines() if ln.startswith("{")][-1])
    assert rec["world"] == 2 and rec["distinct"]
    assert rec["max_ms"] == 11.0                       # the slower rank defines the step time
    assert rec["rows"] == 4096 + 1024 + 1024 + 4096    # q, k, v, o of the GQA block
    assert abs(rec["value"] - rec["rows"] * 2 / 11e-3) < 1e-6   # all ranks' rows / the slowest rank's time


def test_reference_arm_under_torchrun_prints_one_line_from_rank_zero():
    """bench.py --impl reference launched as the driver launches it for N = 2: rank 0 times the oracle
    and prints the line, the other rank exits 0 without work."""
    out = _torchrun(["bench.py", "--gpus", "2", "--impl", "reference", "--workload", "tiny", "--steps", "1",
                     "--warmup", "3"], 29613)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    rec = json.loads(lines[0])
    assert rec["impl"] == "reference" and rec["n_gpus"] == 2 and rec["config"]["workload"] == "tiny"
    assert rec["cpu_baseline"]["kind"] == "oracle" and rec["cpu_baseline"]["cores"] >= 1
    assert rec["value"] > 0 and rec["e2e"]["h2d_bytes_per_step"] == 0 and rec["higher_is_better"] is True


def test_cuda_arm_refuses_to_run_without_a_gpu():
    import torch
    if torch.cuda.is_available():
        return
    out = subprocess.run([sys.executable, "bench.py", "--workload", "tiny", "--steps", "1"], capture_output=True,
                         text=True, cwd=ROOT, timeout=300)
    assert out.returncode != 0 and "no CPU path" in out.stderr


def test_work_counts_of_the_configurations():
    """The algorithmic counts the roofline fractions are formed from."""
    import bench
    import tb_inputs
    c = tb_inputs.CONFIGS["l2_7b_q"]
    assert bench.sweep_flops(c) == 4096 * 4096.0 ** 2
    assert bench.loop_flops(c) == 4096 * 4096.0 ** 2 + 16.0 * 4096 * 4096 * 129 + 4096 * 4096 * 96.0
    b = tb_inputs.CONFIGS["l2_70b_block"]
    assert bench.out_channels(b) == 8192 + 1024 + 1024 + 8192
    assert bench.hessian_flops(b, 1000) == 1000 * 8192 * 8193.0 * 10
    r = tb_inputs.CONFIGS["l2_7b_block"]
    # with R: q, k, o sweeps count twice (the P term), v (one H_in per head) once
    assert bench.sweep_flops(r) == (2 * 3 + 1) * 4096 * 4096.0 ** 2
