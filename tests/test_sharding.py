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


# --------------------------------------------------------------------------- head- and token-sharded projection
def test_shard_ranges_cover_everything_once():
    from paper_2602_04929_b200.sharded import shard_heads, shard_tokens
    for n_tok, world in [(262144, 8), (20000, 3), (2048, 4), (5, 2), (6144, 2)]:
        cuts = [shard_tokens(n_tok, world, r) for r in range(world)]
        assert cuts[0][0] == 0 and cuts[-1][1] == n_tok
        assert all(a[1] == b[0] for a, b in zip(cuts, cuts[1:]))
        assert all(t0 % 2048 == 0 for t0, t1 in cuts if t1 > t0)    # non-empty slices start on accumulation runs
        sizes = [b - a for a, b in cuts]
        assert max(sizes) - min(sizes) < 2 * 2048        # one run of difference plus the ragged last run
    for n_heads, world in [(32, 8), (8, 3), (2, 4), (64, 1)]:
        cuts = [shard_heads(n_heads, world, r) for r in range(world)]
        assert cuts[0][0] == 0 and cuts[-1][1] == n_heads
        assert all(a[1] == b[0] for a, b in zip(cuts, cuts[1:]))
        assert max(b - a for a, b in cuts) - min(b - a for a, b in cuts) <= 1


SHARDED_WORKER = textwrap.dedent("""
    import os, sys, json
    import torch
    import torch.distributed as dist
    sys.path.insert(0, os.environ["TB_ROOT"])
    import tb_inputs
    from paper_2602_04929_b200 import sharded

    class FakeOps:
        '''CPU stand-ins with the calling convention of the library calls (float64, so that the
        all-reduced sums equal the single-process sums to rounding): only the plumbing is under test.'''
        def accumulate(self, X, Xfp, alpha):
            Xd = X.double()
            H = Xd.T @ Xd
            R = None if Xfp is None else alpha * (Xd - Xfp.double()).T @ Xd
            return H, R
        def finalize(self, H, R, n, damp):
            H /= n
            Hsum = H.clone()
            H += damp * torch.diag(H).mean() * torch.eye(H.shape[0], dtype=H.dtype)
            if R is not None:
                R /= n
            return Hsum
        def factor(self, H):
            if H.dim() == 3:
                return torch.stack([self.factor(h) for h in H])
            return torch.linalg.cholesky(torch.linalg.inv(H)).T.contiguous()
        def correction(self, R, U):
            T = R @ U.T
            return torch.triu(T, 1) @ U, T @ U
        def build_hout(self, G, Hsum, n_heads, d_head, damp):
            Gd = G.double().reshape(n_heads, d_head, -1)
            return torch.stack([g @ Hsum @ g.T + damp * torch.eye(d_head, dtype=torch.float64) for g in Gd])
        def quantize(self, kw, W, H, U, Hout, Uout, R, P, C):
            # any deterministic function of exactly the arguments a rank must hold
            heads, dh = kw["n_heads"], kw["d_head"]
            Wd = W.double().reshape(heads, dh, -1)
            s = (Wd.abs().amax(dim=2, keepdim=True) / 3.0) * (1.0 + 0.01 * torch.diag(U).mean())
            if Uout is not None:
                s = s * (1.0 + 0.01 * torch.diagonal(Uout, dim1=1, dim2=2).mean(dim=1).reshape(heads, 1, 1))
            if C is not None:
                s = s * (1.0 + 0.01 * C.abs().mean())
            codes = torch.clamp(torch.round(Wd / s) + 2, 0, 3)
            w_hat = (s * (codes - 2)).reshape(heads * dh, -1)
            loss = ((w_hat.reshape(heads, dh, -1) - Wd) @ H * (w_hat.reshape(heads, dh, -1) - Wd)).sum(dim=(1, 2))
            ng = 1
            return (codes.reshape(heads * dh, -1).to(torch.uint8), s.reshape(heads * dh, ng).float(),
                    torch.full((heads * dh, ng), 2, dtype=torch.int32), w_hat.float(), loss)

    dist.init_process_group("gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    d, H, dh, n_tok = 32, 3, 4, 6144 + 100          # 3 heads on 2 ranks: 2 + 1; ragged token count
    W = torch.from_numpy(tb_inputs.weight(7, H * dh, d))
    G = torch.from_numpy(tb_inputs.weight(7, H * dh, d, tid=tb_inputs.T_WPARTNER))
    rec = tb_inputs.DeviationRecipe(tb_inputs.HeavyTailRecipe(d, seed=7))
    X, Xfp = (torch.from_numpy(a) for a in rec.chunk(0, n_tok))
    t0, t1 = sharded.shard_tokens(n_tok, world, rank)
    out = sharded.quantize_projection_sharded(W, X[t0:t1], n_tok, H, dh, 2, 0, 2, G=G, Xfp_local=Xfp[t0:t1],
                                              ops=FakeOps())
    # the same through the world-size-1 path on all tokens (no process group involved in the arithmetic)
    ops = FakeOps()
    Hf, Rf = ops.accumulate(X, Xfp, 0.25)
    Hsum = ops.finalize(Hf, Rf, n_tok, 0.01)
    U = ops.factor(Hf); P, C = ops.correction(Rf, U)
    Ho = ops.build_hout(G, Hsum, H, dh, 0.01); Uo = ops.factor(Ho)
    ref = ops.quantize(dict(n_heads=H, d_head=dh), W, Hf, U, Ho, Uo, Rf, P, C)
    ok = (torch.equal(out.codes, ref[0]) and torch.allclose(out.scales, ref[1], rtol=1e-6)
          and torch.equal(out.zeros, ref[2]) and torch.allclose(out.w_hat, ref[3], rtol=1e-6)
          and torch.allclose(out.loss, ref[4], rtol=1e-9))
    shapes = [tuple(out.codes.shape), tuple(out.scales.shape), tuple(out.loss.shape)]
    # every rank holds the same gathered result
    digest = torch.tensor([float(out.w_hat.double().sum()), float(out.loss.sum())], dtype=torch.float64)
    both = [torch.zeros_like(digest) for _ in range(world)]
    dist.all_gather(both, digest)
    if rank == 0:
        print(json.dumps({"ok": bool(ok), "shapes": shapes, "same_on_all_ranks": bool(torch.equal(both[0], both[1])),
                          "tokens": [t0, t1]}))
    dist.destroy_process_group()
""")


def test_head_and_token_sharded_projection_on_two_gloo_ranks(tmp_path):
    """The sharded path's plumbing on CPU: token slices, the all-reduce of the statistics, the head
    ranges (3 heads on 2 ranks), the padded all-gather and its order, against the unsharded call of
    the same stand-in arithmetic."""
    script = tmp_path / "sharded_worker.py"
    script.write_text(SHARDED_WORKER)
    out = _torchrun([str(script)], 29615, 300)
    assert out.returncode == 0, out.stderr[-3000:]
    rec = json.loads([ln for ln in out.stdout.splitlines() if ln.startswith("{")][-1])
    assert rec["ok"] and rec["same_on_all_ranks"]
    assert rec["shapes"] == [[12, 32], [12, 1], [3]]
    assert rec["tokens"] == [0, 4096]


def test_sharded_path_needs_the_cuda_library_by_default():
    """Without `ops` the sharded path calls the library, which refuses CPU tensors."""
    import pytest
    import torch
    from paper_2602_04929_b200 import sharded
    with pytest.raises(ValueError):
        sharded.quantize_projection_sharded(torch.zeros(8, 128), torch.zeros((2048, 128), dtype=torch.bfloat16), 2048,
                                            2, 4, 2, 0, 2)
