#!/usr/bin/env python
"""Benchmark of the TurboBoA quantizer path on B200.

One "step" quantizes one projection from its calibration activations: Hessian
accumulation and finalisation, H_out construction, both inverse Cholesky
factors, then the out-channel-group loop, the scale refinement and the loss.
The default workload is the Llama-2-7B-shaped q_proj (W 4096 x 4096, 128 x 2048
synthetic heavy-tailed tokens in bf16, 32 heads x 128, INT2, column groups of
128, out-block 32, adaptive grid + coordinate descent).

    python bench.py --gpus 1 --steps 5 --warmup 3
    python -m torch.distributed.run --nproc-per-node N ... bench.py --gpus N ...
    python bench.py --impl reference        # the float64 CPU oracle on the host cores

Prints ONE JSON line on rank 0.  With N > 1 every rank quantizes its own layer
(independent problems, no collective on the data path): weak scaling.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import tb_inputs  # noqa: E402

METRIC = "out_channels_quantized_per_s"
UNIT = "out-channels/s"
DAMP = 0.01
FLAGS_ADAPT, FLAGS_CD = 1, 2
# FP64 FMA peak of the CUDA cores: 148 SMs x 64 FP64 lanes x 2 flop x 1.965 GHz (TFLOP/s)
FP64_ALU_PEAK_TFLOPS = 148 * 64 * 2 * 1.965e9 / 1e12
# FP32 FMA peak: 148 SMs x 128 lanes x 2 x 1.965 GHz
FP32_ALU_PEAK_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12
# dram__bytes_read.sum + dram__bytes_write.sum per launch, from the ncu captures summarised under
# profiles/ (full-size workload, one launch each); filled in when a capture of the current kernel exists
NCU_TRAFFIC = {
    ("l2_7b_q", "k_sweep_rows"): 80.0e6,   # 69.4 MB read + 8.8-11.5 MB written per launch (4 launches per layer)
    ("l2_7b_q", "k_grid_tri"): 35.0e6,     # read per launch (4 launches per layer); nothing written to DRAM
    ("l2_7b_q", "k_syrk_tc"): 6.367e9,     # 6.271 GB read + 0.096 GB written, one launch per layer; X itself is 2.15 GB
}


def workload(name: str):
    cfg = tb_inputs.CONFIGS[name]
    proj = cfg.projections[0]
    return cfg, proj


def gen_inputs(cfg, proj, seed: int, n_tok: int):
    """Host-side synthetic inputs: W, partner projection G (W_K), X as bf16 bit patterns."""
    W = tb_inputs.weight(seed, proj.d_out, proj.d_in)
    G = tb_inputs.weight(seed, proj.d_out, proj.d_in, tid=tb_inputs.T_WPARTNER) if proj.partner else None
    rec = tb_inputs.HeavyTailRecipe(proj.d_in, seed=seed)
    Xb = np.empty((n_tok, proj.d_in), np.uint16)
    step = 4096
    for t0 in range(0, n_tok, step):
        n = min(step, n_tok - t0)
        Xb[t0:t0 + n] = tb_inputs.to_bf16_bits(rec.chunk(t0, n, bf16=False))
    return W, G, Xb


class ClockSampler:
    """nvidia-smi clocks and throttle reasons, sampled while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "50",
                 "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for nm, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def count_launches(cfg, proj, n_tok: int, with_loss=True, cd_iters=1) -> int:
    """Kernel launches of one step of this library (torch's own fill / reduce kernels not counted),
    from the launch loops of the library for a shared H_in without the propagated-error term."""
    d, dh, H = proj.d_in, proj.d_head, proj.n_heads
    has_hout = bool(proj.partner)
    g = cfg.out_block if has_hout else dh
    S = dh // g

    def factor(dd, n_batch=1):
        panels = -(-dd // 64)
        dp = 64 << max(0, (panels - 1).bit_length())
        G = min(512, dp)                                 # the inverse goes block by block of G columns
        n = 1 + panels + max(0, panels - 2)              # reverse, panels, trailing updates (from the panel after the next on)
        s = 64
        while s < G:                                     # inside a block: both products of every level
            n += (dp // G) * 2 * (1 if G // (2 * s) == 1 else n_batch)
            s *= 2
        n += dp // G                                     # 64 x 64 diagonal inverses, one launch per block
        while s < dp:                                    # above: first product (in row pieces when large), second product
            n += (dp // (2 * s)) * ((-(-s // 768) if s > 1024 else 1) + 1)
            s *= 2
        return n + 1                                     # reverse

    d_out = proj.d_out
    seg = cfg.quant_group or d
    ng = d // seg
    n = 1 + 1 + 2                                       # tensor-core accumulate, mirror, finalize (2)
    if has_hout:
        hout_tensor = d_out % 8 == 0 and d % 32 == 0    # G Hsum as a split-bf16 tensor-core product
        n += (3 if hout_tensor else 1) + 2              # (two splits +) product, per-head Gram, combine
    n += factor(d) + (factor(dh, H) if has_hout else 0)
    n += 1 + (1 if has_hout and S > 1 else 0)           # widen, compensation matrices
    n += (S if cfg.adaptive else 1) + S                 # grid search, one sweep launch per step
    n += 2 * (S - 1) if has_hout else 0                 # residual + compensation GEMM
    if cfg.cd:
        # rows per batch: whole heads (or blocks of 128 rows) whose blockwise products fit 4 GiB
        unit_rows = dh if has_hout else 1
        rows = max(1, (4 << 30) // (ng * d * 8 * unit_rows)) * unit_rows
        rows = min(rows, d_out)
        if not has_hout and rows > 128:
            rows = rows // 128 * 128
        batches = -(-d_out // rows)
        yw_tensor = seg % 64 == 0 and rows % 8 == 0 and d_out % 8 == 0 and (dh % 8 == 0 or rows == d_out)
        dm_tensor = yw_tensor and d % 32 == 0
        per_batch = (3 if yw_tensor else 1) - (1 if yw_tensor else 0)   # transpose + product (the split of H_in is once)
        per_batch += 2 if dm_tensor else 1                               # (split of Q - W +) product with H_in
        if has_hout:
            csize = 8
            while csize > 1 and (ng % csize or (rows // dh) * csize > 148):
                csize //= 2
            by_cols = ng <= 32 and (ng // csize) * seg <= 1024 and seg % 2 == 0 and d % 2 == 0 and d * 4 <= 48 * 1024
            per_batch += (1 if by_cols else 0) + 3 * cd_iters            # row statistics; then G, cluster pass, refresh
        else:
            per_batch += 2 * cd_iters                                    # the two row kernels
        n += 1 + (1 if yw_tensor else 0) + batches * per_batch           # prep, split of H_in
    n += 1                                              # dequant
    if with_loss:
        n += 1 + (0 if cfg.cd else 1) + (1 if has_hout else 0) + 2      # prep, (Z product), (H_out Z), partial sums, reduction
    return n


def run_reference(args, cfg, proj, rank, world):
    """The float64 CPU oracle, as it stands, on a bounded sample: one head of the workload
    per step (heads are independent).  Rank 0 only."""
    if rank != 0:
        return
    import oracle
    d, dh = proj.d_in, proj.d_head
    n_tok = 4096
    import oracle.problems as pu
    prob = pu.make_problem(0, d, 1, dh, n_tok, hout="proj" if proj.partner else None)
    flags = (FLAGS_ADAPT if cfg.adaptive else 0) | (FLAGS_CD if cfg.cd else 0)
    od = pu.oracle_desc(prob, cfg.bits, cfg.quant_group, cfg.out_block, flags)

    def step():
        oracle.quantize_layer(od, prob["W"], prob["Hin"][0], prob["Uin"][0], prob["Hout"], prob["Uout"])

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = (time.perf_counter() - t0) / max(args.steps, 1)
    value = dh / dt
    cores = oracle.num_threads()
    sample = (f"group loop + scale refinement of 1 head ({dh} out-channels) of the {proj.d_out}x{d} layer per "
              f"step; Hessian ({n_tok} tokens) and factors computed once outside the timed steps")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": cfg.name, "d_out": proj.d_out, "d_in": d, "bits": cfg.bits,
                       "quant_group": cfg.quant_group, "out_block": cfg.out_block},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def cpu_baseline(cfg, proj, budget_s: float = 20.0):
    """Oracle timed on the host cores on a bounded sample of the same workload."""
    import oracle
    import oracle.problems as pu
    d, dh = proj.d_in, proj.d_head
    prob = pu.make_problem(0, d, 1, dh, 4096, hout="proj" if proj.partner else None)
    flags = (FLAGS_ADAPT if cfg.adaptive else 0) | (FLAGS_CD if cfg.cd else 0)
    od = pu.oracle_desc(prob, cfg.bits, cfg.quant_group, cfg.out_block, flags)
    t0 = time.perf_counter()
    oracle.quantize_layer(od, prob["W"], prob["Hin"][0], prob["Uin"][0], prob["Hout"], prob["Uout"])
    dt = time.perf_counter() - t0
    return {"value": dh / dt, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"group loop + scale refinement of 1 of {proj.n_heads} heads ({dh} out-channels), "
                      f"{dt:.1f} s; Hessian accumulation and factorisation not included"}


def report_configs(args):
    """Times tb_quantize_layer on every projection of the five configurations (device-resident
    inputs; Hessians from 16384 synthetic tokens, which changes no shape) and prints one JSON
    line per projection: seconds per layer, out-channels/s of the whole call and of the group
    loop (grid + sweep + compensation), and the loop's fraction of the FP64 peak."""
    import torch
    import paper_2602_04929_b200 as tb
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    n_tok = args.tokens or 16384
    only = set(args.only.split(",")) if args.only else None
    for name, cfg in tb_inputs.CONFIGS.items():
        if only and name not in only:
            continue
        d = cfg.d_model
        cache = {}

        def hessian(tag, with_r):
            if tag in cache:
                return cache[tag]
            rec = tb_inputs.HeavyTailRecipe(d, seed=0, tid_shift=0 if tag == "attn" else 1)
            if name == "tiny":
                X = torch.from_numpy(tb_inputs.activations_gaussian(0, cfg.n_tok, d)).to(dev)
                Xfp = None
            elif with_r:
                xs, xf = tb_inputs.DeviationRecipe(rec).chunk(0, n_tok)
                X = torch.from_numpy(xs).to(dev).to(torch.bfloat16)
                Xfp = torch.from_numpy(xf).to(dev).to(torch.bfloat16)
            else:
                X = torch.from_numpy(rec.chunk(0, n_tok)).to(dev).to(torch.bfloat16)
                Xfp = None
            H = torch.zeros((d, d), dtype=torch.float32, device=dev)
            tb.tb_accumulate_hessian(H, X)
            R = None
            if Xfp is not None:
                R = torch.zeros((d, d), dtype=torch.float32, device=dev)
                tb.tb_accumulate_cross(R, X, Xfp, cfg.alpha)
            Hsum = torch.empty_like(H)
            tb.tb_finalize_hessian(H, R, X.shape[0], cfg.damp, Hsum_out=Hsum)
            U, info = tb.tb_factor(H)
            assert int(info.max().item()) == 0
            P = C = None
            if R is not None:
                P, C = tb.tb_prepare_correction(R, U)
            cache[tag] = (H, Hsum, U, R, P, C)
            return cache[tag]

        def hessian_per_head(n_heads):
            """Value projection (Table 1): one H_in per head from X-bar_h = A_h X with the synthetic causal
            decay of tb_inputs; no propagated-error term on this projection (there is no X-bar of the
            full-precision path in the recipe)."""
            if "v" in cache:
                return cache["v"]
            rec = tb_inputs.HeavyTailRecipe(d, seed=0)
            Xh = rec.chunk(0, n_tok)
            Hs = torch.empty((n_heads, d, d), dtype=torch.float32, device=dev)
            for h in range(n_heads):
                Xb = torch.from_numpy(tb_inputs.causal_decay_mix(Xh, tb_inputs.decay_rate(h), 2048)).to(dev).to(torch.bfloat16)
                Hs[h].zero_()
                tb.tb_accumulate_hessian(Hs[h], Xb)
                tb.tb_finalize_hessian(Hs[h], None, n_tok, cfg.damp)
            Us, info = tb.tb_factor(Hs)
            assert int(info.max().item()) == 0
            cache["v"] = (Hs, None, Us, None, None, None)
            return cache["v"]

        for proj in cfg.projections:
            per_head = proj.name == "v" and name != "tiny"
            if per_head:
                H, Hsum, U, R, P, C = hessian_per_head(proj.n_heads)
            else:
                H, Hsum, U, R, P, C = hessian("o" if proj.name == "o" else "attn", cfg.with_r)
            W = torch.from_numpy(tb_inputs.weight(0, proj.d_out, proj.d_in, tid=tb_inputs.T_W + (hash(proj.name) % 3))).to(dev)
            Hout = Uout = None
            if name == "tiny":
                Hout = torch.from_numpy(tb_inputs.spd_matrix(0, proj.d_head)[None]).to(dev)
            elif proj.partner in ("k", "q"):
                gh = cfg.n_kv_heads if proj.partner == "k" else cfg.n_q_heads
                G = torch.from_numpy(tb_inputs.weight(0, gh * cfg.d_head, d, tid=tb_inputs.T_WPARTNER)).to(dev)
                Hout = tb.tb_build_hout(G, Hsum, proj.n_heads, proj.d_head, cfg.damp)
            elif proj.partner == "o":
                G = torch.from_numpy(tb_inputs.weight(0, cfg.n_q_heads * cfg.d_head, d, tid=tb_inputs.T_WOUT)).to(dev)
                Hout = tb.tb_build_hout(G, None, proj.n_heads, proj.d_head, cfg.damp)
            if Hout is not None:
                Uout, info = tb.tb_factor(Hout)
                assert int(info.max().item()) == 0
            blocks = [cfg.out_block] if name != "l2_70b_block" or proj.name != "q" else [1, 8, 32, 64, 128]
            for g in blocks:
                flags = (FLAGS_ADAPT if cfg.adaptive else 0) | (FLAGS_CD if cfg.cd else 0)
                desc = tb.layer_desc(proj.d_out, proj.d_in, proj.n_heads, proj.d_head, cfg.bits, cfg.quant_group,
                                     g if Hout is not None else proj.d_head, n_hin=proj.n_heads if per_head else 1,
                                     flags=flags)
                ws = torch.empty(tb.tb_quantize_layer_workspace(desc, R is not None, True), dtype=torch.uint8, device=dev)
                res = None
                for rep in range(3):
                    if rep == 1:
                        tb.tb_profile_enable(True)
                        torch.cuda.synchronize()
                        t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
                        t0.record()
                    res = tb.tb_quantize_layer(desc, W, H, U, Hout, Uout, R, P, C, ws=ws, out=res)
                t1.record()
                torch.cuda.synchronize()
                ms = t0.elapsed_time(t1) / 2
                q = {k: v / 2 for k, v in tb.tb_profile_read().items()}
                tb.tb_profile_enable(False)
                loop_ms = q["grid"] + q["sweep"] + q["compensation"]
                seg = cfg.quant_group or proj.d_in
                S = proj.d_head // g if Hout is not None else 1
                # algorithmic FP64 work of the loop: sweep d_in^2 per row (twice with the P term), the symmetric
                # quadratic forms of the grid search, and with R the W0 C product of every step but the last
                fl = (1 + (R is not None)) * proj.d_out * proj.d_in ** 2 + 16.0 * proj.d_out * proj.d_in * (seg + 1) + \
                    (2.0 * proj.d_out * proj.d_in ** 2 * (S - 1) / S if (R is not None and S > 1) else 0.0)
                print(json.dumps({"config": name, "projection": proj.name, "shape": [proj.d_out, proj.d_in],
                                  "heads": proj.n_heads, "n_hin": proj.n_heads if per_head else 1, "out_block": g, "bits": cfg.bits,
                                  "with_r": R is not None,
                                  "adaptive": cfg.adaptive, "cd": cfg.cd, "ms_per_layer": ms,
                                  "out_channels_per_s": proj.d_out / (ms * 1e-3), "phases_ms": q, "loop_ms": loop_ms,
                                  "loop_out_channels_per_s": proj.d_out / (loop_ms * 1e-3),
                                  "loop_tflops": fl / (loop_ms * 1e-3) / 1e12,
                                  "loop_frac_of_fp64_peak": fl / (loop_ms * 1e-3) / 1e12 / FP64_ALU_PEAK_TFLOPS,
                                  "device_error_flag": tb.tb_device_error_flag()}), flush=True)
                del ws
        del cache
        torch.cuda.empty_cache()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--report-configs", action="store_true",
                    help="time tb_quantize_layer on every projection of the five configurations")
    ap.add_argument("--only", default="", help="comma-separated config names for --report-configs")
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="l2_7b_q")
    ap.add_argument("--tokens", type=int, default=0, help="override the token count (default: the config's)")
    ap.add_argument("--heads", type=int, default=0,
                    help="keep only this many heads of the projection (small captures under a profiler)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.report_configs:
        report_configs(args)
        return

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    cfg, proj = workload(args.workload)
    if args.heads and proj.partner:
        import dataclasses
        proj = dataclasses.replace(proj, n_heads=args.heads, d_out=args.heads * proj.d_head)
    if args.impl == "reference":
        run_reference(args, cfg, proj, rank, world)
        return

    import torch
    import paper_2602_04929_b200 as tb
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the quantizer has no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    tb.load()

    n_tok = args.tokens or cfg.n_tok
    d, d_out, H, dh = proj.d_in, proj.d_out, proj.n_heads, proj.d_head
    flags = (FLAGS_ADAPT if cfg.adaptive else 0) | (FLAGS_CD if cfg.cd else 0)
    desc = tb.layer_desc(d_out, d, H, dh, cfg.bits, cfg.quant_group, cfg.out_block, flags=flags)
    ng = desc.n_groups

    W_h, G_h, Xb_h = gen_inputs(cfg, proj, seed=rank, n_tok=n_tok)
    W = torch.from_numpy(W_h).to(dev)
    G = torch.from_numpy(G_h).to(dev) if G_h is not None else None
    X = torch.from_numpy(Xb_h.view(np.int16)).to(dev).view(torch.bfloat16)
    g_heads = H if G is not None else 0

    lib = tb.load()
    Hin = torch.empty((d, d), dtype=torch.float32, device=dev)
    Hsum = torch.empty_like(Hin)
    out = tb.QuantizeResult(
        codes=torch.empty((d_out, d), dtype=torch.uint8, device=dev),
        scales=torch.empty((d_out, ng), dtype=torch.float32, device=dev),
        zeros=torch.empty((d_out, ng), dtype=torch.int32, device=dev),
        cand=torch.empty((d_out, ng), dtype=torch.uint8, device=dev),
        w_hat=torch.empty((d_out, d), dtype=torch.float32, device=dev),
        loss=torch.empty(H, dtype=torch.float64, device=dev),
        stats=torch.zeros(8, dtype=torch.int64, device=dev))
    ws = torch.empty(tb.tb_quantize_layer_workspace(desc, False, True), dtype=torch.uint8, device=dev)

    phases = {}

    def ev():
        e = torch.cuda.Event(enable_timing=True)
        e.record()
        return e

    # H_out and its factor depend on the Hessian only, like the factor of H_in: they run on a second
    # stream next to it (the factor of H_in is a chain of small launches that leaves SMs idle)
    side = torch.cuda.Stream(device=dev) if G is not None else None

    def step(record=None):
        marks = [("start", ev())] if record is not None else None
        Hin.zero_()
        tb.tb_accumulate_hessian(Hin, X)
        tb.tb_finalize_hessian(Hin, None, n_tok, DAMP, Hsum_out=Hsum)
        if marks is not None:
            marks.append(("hessian", ev()))
        Hout = Uout = None
        if G is not None:
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                Hout = tb.tb_build_hout(G, Hsum, H, dh, DAMP)
                Uout, info_out = tb.tb_factor(Hout)
        Uin, info_in = tb.tb_factor(Hin)
        if G is not None:
            torch.cuda.current_stream().wait_stream(side)
        if marks is not None:
            marks.append(("factor", ev()))
        tb.tb_quantize_layer(desc, W, Hin, Uin, Hout, Uout, ws=ws, out=out)
        if marks is not None:
            marks.append(("quantize", ev()))
            record.append(marks)
        return info_in

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()

    for _ in range(args.warmup):
        info = step()
    torch.cuda.synchronize()
    assert int(info.max().item()) == 0, "H_in was not positive definite"

    sampler = ClockSampler(local_rank)
    tb.tb_profile_enable(True)
    rec = []
    barrier()
    torch.cuda.synchronize()
    sampler.start()
    e0 = ev()
    for _ in range(args.steps):
        step(rec)
    e1 = ev()
    torch.cuda.synchronize()
    barrier()
    clocks = sampler.stop()
    total_ms = e0.elapsed_time(e1)
    q_ms = tb.tb_profile_read()
    tb.tb_profile_enable(False)
    for marks in rec:
        for (_, a), (nm, b) in zip(marks[:-1], marks[1:]):
            phases[nm] = phases.get(nm, 0.0) + a.elapsed_time(b)
    K = max(args.steps, 1)
    phases = {k: v / K for k, v in phases.items()}
    q_ms = {k: v / K for k, v in q_ms.items()}
    ms_per_step = total_ms / K
    if world > 1:
        import torch.distributed as dist
        t = torch.tensor([ms_per_step], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms_per_step = float(t.item())

    # ---- end to end from pinned host buffers through the C ABI ----
    e2e = None
    if not args.no_e2e:
        Wp = torch.from_numpy(W_h).pin_memory()
        Xp = torch.from_numpy(Xb_h.view(np.int16)).pin_memory()
        Gp = torch.from_numpy(G_h).pin_memory() if G_h is not None else None
        outs = {"codes": torch.empty((d_out, d), dtype=torch.uint8).pin_memory(),
                "scales": torch.empty((d_out, ng), dtype=torch.float32).pin_memory(),
                "zeros": torch.empty((d_out, ng), dtype=torch.int32).pin_memory(),
                "w_hat": torch.empty((d_out, d), dtype=torch.float32).pin_memory(),
                "loss": torch.empty(H, dtype=torch.float64).pin_memory()}
        hws = torch.empty(tb.tb_quantize_from_host_workspace(desc, n_tok, g_heads), dtype=torch.uint8, device=dev)
        tb.tb_quantize_from_host(desc, Wp, Xp, Gp, DAMP, DAMP, outs, hws)  # warm-up
        n_e2e = min(K, 3)
        barrier()
        torch.cuda.synchronize()
        a = ev()
        for _ in range(n_e2e):
            tb.tb_quantize_from_host(desc, Wp, Xp, Gp, DAMP, DAMP, outs, hws)
        b = ev()
        torch.cuda.synchronize()
        e2e_ms = a.elapsed_time(b) / n_e2e
        if world > 1:
            import torch.distributed as dist
            t = torch.tensor([e2e_ms], dtype=torch.float64, device=dev)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            e2e_ms = float(t.item())
        h2d = Wp.numel() * 4 + Xp.numel() * 2 + (Gp.numel() * 4 if Gp is not None else 0)
        d2h = sum(v.numel() * v.element_size() for v in outs.values())
        e2e = {"value": d_out * world / (e2e_ms * 1e-3), "unit": UNIT, "ms_per_step": e2e_ms, "steps": n_e2e,
               "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h)}
        assert np.array_equal(outs["codes"].numpy(), out.codes.cpu().numpy()), "host and device paths disagree"

    if rank != 0:
        if world > 1:
            import torch.distributed as dist
            dist.destroy_process_group()
        return

    # ---- rooflines (algorithmic work / measured phase time) ----
    peaks = {}
    try:
        peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
    except OSError:
        pass
    bf16_peak = float(peaks.get("bf16_tflops", 1590.0))
    bf16_kind = "measured cuBLAS bf16 burst (MEASURED_PEAKS.json)" if peaks else "fallback 1.59 PFLOP/s"
    seg = cfg.quant_group or d
    has_hout = G is not None
    # issued tensor-core work of the Hessian: 128 x 256 tiles on or below the diagonal
    m_blocks = -(-d // 128)
    syrk_tiles = sum(mi // 2 + 1 for mi in range(m_blocks))
    fl = {
        "hessian": 2.0 * 128 * 256 * n_tok * syrk_tiles,
        "sweep": 1.0 * d_out * d * d,                             # d_in^2 flop per out-channel
        # e H e^T of a symmetric H: seg (seg + 1) / 2 products and as many additions per candidate and group
        "grid": 16.0 * d_out * d * (seg + 1),
        # Cholesky of the reversed matrix (d^3 / 3) and the triangular inverse (d^3 / 3), for H_in and per head for H_out
        "factor": (2.0 / 3.0) * d ** 3 + ((2.0 / 3.0) * dh ** 3 * H if has_hout else 0.0),
    }
    fp64_kind = "FP64 FMA / FP64 tensor pipe, 148 SM x 64 lanes x 2 x 1.965 GHz"
    roof_all = {}
    times = {}
    if phases.get("hessian"):
        times["hessian"] = phases["hessian"]
        roof_all["hessian"] = {"kernel": "k_syrk_tc (+ zero, mirror, finalize)", "bound": "tensor",
                               "achieved": fl["hessian"] / (phases["hessian"] * 1e-3) / 1e12, "peak": bf16_peak,
                               "unit": "TFLOP/s", "peak_kind": bf16_kind}
    names = {"sweep": "k_sweep_rows", "grid": "k_grid_tri"}
    for nm in ("sweep", "grid"):
        if q_ms.get(nm):
            times[nm] = q_ms[nm]
            roof_all[nm] = {"kernel": names[nm], "bound": "alu", "achieved": fl[nm] / (q_ms[nm] * 1e-3) / 1e12,
                            "peak": FP64_ALU_PEAK_TFLOPS, "unit": "TFLOP/s", "peak_kind": fp64_kind}
    if phases.get("factor"):
        roof_all["factor"] = {"kernel": "k_chol_panel + FP64 GEMM engine (trailing updates, recursive-doubling inverse); "
                                        "the H_out build and its factor run beside it on a second stream",
                              "bound": "alu", "achieved": fl["factor"] / (phases["factor"] * 1e-3) / 1e12,
                              "peak": FP64_ALU_PEAK_TFLOPS, "unit": "TFLOP/s", "peak_kind": fp64_kind}
    # DRAM traffic per launch from the committed ncu captures (profiles/), bytes; None where no capture applies
    traffic = {"sweep": NCU_TRAFFIC.get((cfg.name, "k_sweep_rows")), "grid": NCU_TRAFFIC.get((cfg.name, "k_grid_tri")),
               "hessian": NCU_TRAFFIC.get((cfg.name, "k_syrk_tc"))}
    for k, v in roof_all.items():
        v["frac"] = v["achieved"] / v["peak"]
        v["traffic"] = traffic.get(k) if not args.heads and not args.tokens else None
    # the single kernel with the largest share of the step (the Hessian product, the column sweep or the grid search)
    dominant = max(times, key=times.get) if times else None
    roofline = dict(roof_all.get(dominant, {}))
    loop_ms = q_ms.get("grid", 0.0) + q_ms.get("sweep", 0.0) + q_ms.get("compensation", 0.0)
    loop_fl = fl["sweep"] + fl["grid"] + (1.0 * d_out * d * (dh - cfg.out_block) if has_hout else 0.0)

    line = {
        "metric": METRIC, "value": d_out * world / (ms_per_step * 1e-3), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": cfg.name, "d_out": d_out, "d_in": d, "n_heads": H, "d_head": dh,
                   "tokens": n_tok, "x_dtype": "bf16", "bits": cfg.bits, "quant_group": cfg.quant_group,
                   "out_block": cfg.out_block, "adaptive_grid": cfg.adaptive, "cd_refine": cfg.cd,
                   "l2": "inputs larger than L2 (activations %.1f GiB)" % (n_tok * d * 2 / 2 ** 30)},
        "seconds_per_layer": ms_per_step * 1e-3,
        "phases_ms": dict(phases, **{"quantize/" + k: v for k, v in q_ms.items()}),
        "loop_ms": loop_ms,
        "loop_out_channels_per_s": d_out / (loop_ms * 1e-3) if loop_ms else None,
        "loop_roofline": {"bound": "alu", "achieved": loop_fl / (loop_ms * 1e-3) / 1e12 if loop_ms else None,
                          "peak": FP64_ALU_PEAK_TFLOPS, "unit": "TFLOP/s",
                          "frac": loop_fl / (loop_ms * 1e-3) / 1e12 / FP64_ALU_PEAK_TFLOPS if loop_ms else None},
        "clocks": clocks, "gpu_launches": count_launches(cfg, proj, n_tok) * args.steps,
        "roofline": roofline, "rooflines": roof_all,
    }
    if e2e is not None:
        line["e2e"] = e2e
    if world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(cfg, proj)
    print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
