#!/usr/bin/env python
"""Benchmark of the TurboBoA quantizer path on B200.

One "step" quantizes one attention layer from its calibration activations through ONE call of the
C ABI (tb_attention_layer): Hessians of the attention input, of every key/value head's
attention-weighted input (the value projection's own H_in, Table 1) and of the output projection's
input; the out-channel Hessians of Table 1; every inverse Cholesky factor; then Algorithm 1's
out-channel-group loop (and, where the configuration has them, the scale refinement and the
propagated-error terms) for W_Q, W_K, W_V and W_O.  The default workload is the largest of the five
configurations, the Llama-2-70B-shaped block (q/o 8192 x 8192, k/v 1024 x 8192, 64 heads, 8 key/value
heads, 128 x 2048 synthetic bf16 tokens, INT2, column groups of 128, out-block 32).  The other four
configurations are measured in the same run and carried in the line's `configs` array.

    python bench.py --gpus 1 --steps 8 --warmup 3
    python -m torch.distributed.run --nproc-per-node N ... bench.py --gpus N ...
    python bench.py --impl reference        # the float64 CPU oracle on the host cores

Prints ONE JSON line on rank 0.  With N > 1 every rank quantizes its own layer (independent
problems, no collective on the data path): weak scaling.
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
FLAGS_ADAPT, FLAGS_CD = 1, 2
DEFAULT_WORKLOAD = "l2_70b_block"
# FP64 FMA peak of the CUDA cores: 148 SMs x 64 FP64 lanes x 2 flop x 1.965 GHz (TFLOP/s)
FP64_ALU_PEAK_TFLOPS = 148 * 64 * 2 * 1.965e9 / 1e12
# FP32 FMA rate measured on this GPU by a register-resident FFMA loop (profiles/fp64_peak_microbench.md)
FP32_FFMA_MEASURED_TFLOPS = 71.5
FP64_KIND = "FP64 FMA / FP64 tensor pipe, 148 SM x 64 lanes x 2 x 1.965 GHz"
# dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu captures summarised under
# profiles/ (bytes), keyed by (workload, kernel); absent where the kernel has changed since its capture
# (the mean over the launches of that kernel in one layer; the Hessian kernel's figure holds for the
# default 262 144 tokens only)
NCU_TRAFFIC = {
    ("l2_70b_block", "k_sweep_rows"): 759.0e6,     # 13 launches per layer, 9.9 GB in all
    ("l2_70b_block", "k_grid_tri"): 314.1e6,       # 4 launches per layer
    ("l2_70b_block", "k_syrk_tc"): 55.2e9,         # 10 launches per layer (pair form, 66 pairs), 49.4 .. 58.7 GB read each
    ("l2_7b_q", "k_sweep_rows"): 77.9e6,           # 4 launches per layer
    ("l2_7b_q", "k_grid_tri"): 34.9e6,             # 4 launches per layer
    ("l2_7b_q", "k_syrk_tc"): 6.91e9,
}
NCU_TRAFFIC_TOKENS = 262144


# --------------------------------------------------------------------------------------------
# configurations
# --------------------------------------------------------------------------------------------

def config_flags(cfg) -> int:
    return (FLAGS_ADAPT if cfg.adaptive else 0) | (FLAGS_CD if cfg.cd else 0)


def is_block(cfg) -> bool:
    return len(cfg.projections) == 4


def config_summary(cfg, n_tok) -> dict:
    return {"workload": cfg.name, "tokens": n_tok, "x_dtype": "bf16", "bits": cfg.bits, "quant_group": cfg.quant_group,
            "out_block": cfg.out_block, "adaptive_grid": cfg.adaptive, "cd_refine": cfg.cd,
            "propagated_error": cfg.with_r,
            "projections": {p.name: [p.d_out, p.d_in] for p in cfg.projections},
            "n_q_heads": cfg.n_q_heads, "n_kv_heads": cfg.n_kv_heads, "d_head": cfg.d_head}


def out_channels(cfg) -> int:
    return sum(p.d_out for p in cfg.projections)


def proj_with_r(cfg, p) -> bool:
    """The value projection of a block has one H_in per head and runs without the propagated-error term."""
    return cfg.with_r and not (p.name == "v" and is_block(cfg))


def loop_flops(cfg) -> float:
    """Algorithmic FP64 work of the out-channel-group loop of every projection: the sweep's d_in^2 per
    row (twice with the P term), the symmetric quadratic forms of the grid search
    (n_cand d_in (group + 1) per row), the joint compensation ((d_head - g) d_in per row) and, with R,
    the W0 C product of every step but the last (2 d_in^2 per row)."""
    total = 0.0
    for p in cfg.projections:
        has_hout = p.partner is not None or cfg.name == "tiny"
        g = cfg.out_block if has_hout else p.d_head
        S = p.d_head // g
        seg = cfg.quant_group or p.d_in
        total += (2 if proj_with_r(cfg, p) else 1) * p.d_out * float(p.d_in) ** 2
        total += 16.0 * p.d_out * p.d_in * (seg + 1)
        if has_hout:
            total += 1.0 * p.d_out * p.d_in * (p.d_head - g)
        if proj_with_r(cfg, p) and S > 1:
            total += 2.0 * p.d_out * float(p.d_in) ** 2 * (S - 1) / S
    return total


def sweep_flops(cfg) -> float:
    return sum((2 if proj_with_r(cfg, p) else 1) * p.d_out * float(p.d_in) ** 2 for p in cfg.projections)


def hessian_flops(cfg, n_tok) -> float:
    """Algorithmic work of the Hessian accumulations: n_tok d (d + 1) per symmetric Hessian (each
    product of the lower triangle once, multiply and add)."""
    if is_block(cfg):
        d, dq = cfg.d_model, cfg.n_q_heads * cfg.d_head
        return n_tok * d * (d + 1.0) * (1 + cfg.n_kv_heads) + n_tok * dq * (dq + 1.0)
    d = cfg.projections[0].d_in
    return n_tok * d * (d + 1.0)


def factor_flops(cfg) -> float:
    """Cholesky of the reversed matrix (d^3 / 3) plus the triangular inverse (d^3 / 3) per matrix."""
    if is_block(cfg):
        d, dq, dh = cfg.d_model, cfg.n_q_heads * cfg.d_head, cfg.d_head
        return ((2.0 / 3.0) * d ** 3 * (1 + cfg.n_kv_heads) + (2.0 / 3.0) * dq ** 3 +
                (2.0 / 3.0) * dh ** 3 * (cfg.n_q_heads + 2 * cfg.n_kv_heads))
    p = cfg.projections[0]
    return (2.0 / 3.0) * p.d_in ** 3 + (2.0 / 3.0) * p.d_head ** 3 * p.n_heads


# --------------------------------------------------------------------------------------------
# clocks
# --------------------------------------------------------------------------------------------

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
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
                pw.append(float(parts[2]))
            except ValueError:
                continue
            for nm, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(pw) if pw else None, "samples": len(sm), "reasons": sorted(reasons)}


def ev():
    import torch
    e = torch.cuda.Event(enable_timing=True)
    e.record()
    return e


# --------------------------------------------------------------------------------------------
# a whole attention layer through tb_attention_layer
# --------------------------------------------------------------------------------------------

class LayerProblem:
    """Device-resident synthetic inputs of one attention layer of `cfg` and its result buffers."""

    def __init__(self, cfg, n_tok, dev, seed):
        import torch
        import paper_2602_04929_b200 as tb
        self.cfg, self.n_tok, self.dev = cfg, n_tok, dev
        d, hq, hkv, dh = cfg.d_model, cfg.n_q_heads, cfg.n_kv_heads, cfg.d_head
        dq = hq * dh

        def t(a):
            return torch.from_numpy(a).to(dev)

        self.W = [t(tb_inputs.weight(seed, dq, d)), t(tb_inputs.weight(seed, hkv * dh, d, tid=tb_inputs.T_WPARTNER)),
                  t(tb_inputs.weight(seed + 1000, hkv * dh, d)), t(tb_inputs.weight(seed, d, dq, tid=tb_inputs.T_WOUT))]
        rec = tb_inputs.HeavyTailRecipe(d, seed=seed)
        rec_o = tb_inputs.HeavyTailRecipe(dq, seed=seed, tid_shift=1)
        self.X_fp = self.X_o_fp = None
        if cfg.with_r:
            self.X_fp = tb_inputs.heavy_tail_device(rec, n_tok, dev, seed)
            self.X = tb_inputs.deviation_device(tb_inputs.DeviationRecipe(rec), self.X_fp, seed)
            self.X_o_fp = tb_inputs.heavy_tail_device(rec_o, n_tok, dev, seed)
            self.X_o = tb_inputs.deviation_device(tb_inputs.DeviationRecipe(rec_o), self.X_o_fp, seed)
        else:
            self.X = tb_inputs.heavy_tail_device(rec, n_tok, dev, seed)
            self.X_o = tb_inputs.heavy_tail_device(rec_o, n_tok, dev, seed)
        # the value projection's attention-weighted inputs A_h X, one per key/value head
        self.X_v = torch.empty((hkv, n_tok, d), dtype=torch.bfloat16, device=dev)
        for h in range(hkv):
            self.X_v[h] = tb_inputs.causal_decay_mix_device(self.X, tb_inputs.decay_rate(h), cfg.seq_len)
        self.desc = tb.attention_desc(d, hq, hkv, dh, cfg.bits, cfg.quant_group, cfg.out_block, n_tok,
                                      flags=config_flags(cfg), damp=cfg.damp, alpha=cfg.alpha, on_host=False, concurrent=True)
        self.outs = tb.attention_outputs(self.desc, device=dev)
        self.n_info = tb.tb_attention_layer_info_count(self.desc, True)
        self.info = torch.zeros(self.n_info, dtype=torch.int32, device=dev)
        self.io = tb.attention_io(self.desc, self.X, self.X_o, self.W, self.outs, X_fp=self.X_fp, X_v=self.X_v,
                                  X_o_fp=self.X_o_fp, info=self.info)
        self.ws = torch.empty(tb.tb_attention_layer_workspace(self.desc, self.io), dtype=torch.uint8, device=dev)
        self.activation_bytes = sum(x.numel() * 2 for x in (self.X, self.X_fp, self.X_v, self.X_o, self.X_o_fp)
                                    if x is not None)

    def step(self, concurrent=True):
        import paper_2602_04929_b200 as tb
        self.desc.concurrent = int(concurrent)
        self.desc.on_host = 0
        tb.tb_attention_layer(self.desc, self.io, self.ws)

    def host_copies(self):
        """Pinned host copies of every input, and pinned result buffers, for the host-buffer call."""
        import paper_2602_04929_b200 as tb

        def pin(x):
            return None if x is None else x.cpu().pin_memory()

        self.desc.on_host, self.desc.concurrent = 1, 1
        houts = tb.attention_outputs(self.desc, device=None, pin=True)
        hX, hXo, hW = pin(self.X), pin(self.X_o), [pin(w) for w in self.W]
        hXfp, hXv, hXofp = pin(self.X_fp), pin(self.X_v), pin(self.X_o_fp)
        hio = tb.attention_io(self.desc, hX, hXo, hW, houts, X_fp=hXfp, X_v=hXv, X_o_fp=hXofp)
        keep = (hX, hXo, hW, hXfp, hXv, hXofp, houts)
        h2d = sum(x.numel() * x.element_size() for x in (hX, hXo, hXfp, hXv, hXofp) if x is not None)
        h2d += sum(w.numel() * 4 for w in hW)
        d2h = sum(v.numel() * v.element_size() for o in houts for v in o.values())
        need = tb.tb_attention_layer_workspace(self.desc, hio)
        self.desc.on_host = 0
        return hio, keep, h2d, d2h, need


def measure_layer(cfg, n_tok, dev, seed, steps, warmup, seq_steps, barrier=lambda: None, sampler=None):
    """Times tb_attention_layer: `steps` calls with the independent parts side by side (the headline),
    then `seq_steps` calls one part after the other with the phase timers on."""
    import torch
    import paper_2602_04929_b200 as tb
    prob = LayerProblem(cfg, n_tok, dev, seed)
    for _ in range(warmup):
        prob.step(True)
    torch.cuda.synchronize()
    assert tb.tb_device_error_flag() == 0
    assert int(prob.info.abs().max().item()) == 0, "a Hessian was not positive definite"
    barrier()
    torch.cuda.synchronize()
    if sampler:
        sampler.start()
    n0 = tb.tb_launch_count()
    e0 = ev()
    for _ in range(steps):
        prob.step(True)
    e1 = ev()
    torch.cuda.synchronize()
    launches = tb.tb_launch_count() - n0
    barrier()
    clocks = sampler.stop() if sampler else None
    ms_conc = e0.elapsed_time(e1) / max(steps, 1)
    # one part after the other, with the phase timers
    prob.step(False)
    torch.cuda.synchronize()
    tb.tb_profile_enable(True)
    a = ev()
    for _ in range(seq_steps):
        prob.step(False)
    b = ev()
    torch.cuda.synchronize()
    ms_seq = a.elapsed_time(b) / max(seq_steps, 1)
    phases = {k: v / max(seq_steps, 1) for k, v in tb.tb_profile_read().items()}
    tb.tb_profile_enable(False)
    assert tb.tb_device_error_flag() == 0
    loss = {p.name: float(prob.outs[i]["loss"].sum().item()) for i, p in enumerate(cfg.projections)}
    return prob, dict(ms_concurrent=ms_conc, ms_sequential=ms_seq, phases_ms=phases, launches=launches, clocks=clocks,
                      loss=loss)


# --------------------------------------------------------------------------------------------
# a single projection (the configurations that are one projection: tiny, l2_7b_q)
# --------------------------------------------------------------------------------------------

def measure_projection_config(cfg, n_tok, dev, seed, steps, warmup, barrier=lambda: None, sampler=None):
    """One step = Hessian accumulation and finalisation, H_out, both factors and tb_quantize_layer for
    the one projection of `cfg`, from device-resident activations."""
    import torch
    import paper_2602_04929_b200 as tb
    proj = cfg.projections[0]
    d, d_out, H, dh = proj.d_in, proj.d_out, proj.n_heads, proj.d_head
    desc = tb.layer_desc(d_out, d, H, dh, cfg.bits, cfg.quant_group, cfg.out_block, flags=config_flags(cfg))
    W = torch.from_numpy(tb_inputs.weight(seed, d_out, d)).to(dev)
    if cfg.name == "tiny":
        X = torch.from_numpy(tb_inputs.activations_gaussian(seed, n_tok, d)).to(dev).to(torch.bfloat16)
        G = None
        Hout_fixed = torch.from_numpy(tb_inputs.spd_matrix(seed, dh)[None]).to(dev)
    else:
        X = tb_inputs.heavy_tail_device(tb_inputs.HeavyTailRecipe(d, seed=seed), n_tok, dev, seed)
        G = torch.from_numpy(tb_inputs.weight(seed, d_out, d, tid=tb_inputs.T_WPARTNER)).to(dev)
        Hout_fixed = None
    Hin = torch.empty((d, d), dtype=torch.float32, device=dev)
    Hsum = torch.empty_like(Hin)
    out = tb.empty_result(desc, dev)
    ws = torch.empty(tb.tb_quantize_layer_workspace(desc, False, True), dtype=torch.uint8, device=dev)
    side = torch.cuda.Stream(device=dev)

    def step(record=None):
        marks = [("start", ev())] if record is not None else None
        Hin.zero_()
        tb.tb_accumulate_hessian(Hin, X)
        tb.tb_finalize_hessian(Hin, None, n_tok, cfg.damp, Hsum_out=Hsum)
        if marks is not None:
            marks.append(("hessian", ev()))
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):   # H_out and its factor beside the factor of H_in
            Hout = tb.tb_build_hout(G, Hsum, H, dh, cfg.damp) if G is not None else Hout_fixed
            Uout, _ = tb.tb_factor(Hout)
        Uin, info_in = tb.tb_factor(Hin)
        torch.cuda.current_stream().wait_stream(side)
        if marks is not None:
            marks.append(("factor", ev()))
        tb.tb_quantize_layer(desc, W, Hin, Uin, Hout, Uout, ws=ws, out=out)
        if marks is not None:
            marks.append(("quantize", ev()))
            record.append(marks)
        return info_in

    for _ in range(warmup):
        info = step()
    torch.cuda.synchronize()
    assert int(info.max().item()) == 0, "H_in was not positive definite"
    barrier()
    torch.cuda.synchronize()
    if sampler:
        sampler.start()
    tb.tb_profile_enable(True)
    rec = []
    n0 = tb.tb_launch_count()
    e0 = ev()
    for _ in range(steps):
        step(rec)
    e1 = ev()
    torch.cuda.synchronize()
    launches = tb.tb_launch_count() - n0
    barrier()
    clocks = sampler.stop() if sampler else None
    ms = e0.elapsed_time(e1) / max(steps, 1)
    phases = {k: v / max(steps, 1) for k, v in tb.tb_profile_read().items()}
    tb.tb_profile_enable(False)
    for marks in rec:
        for (_, a), (nm, b) in zip(marks[:-1], marks[1:]):
            phases["step/" + nm] = phases.get("step/" + nm, 0.0) + a.elapsed_time(b) / max(steps, 1)
    phases["hessian"] = phases.pop("step/hessian")
    phases["factor"] = phases.pop("step/factor")   # with the H_out build and its factor beside it
    assert tb.tb_device_error_flag() == 0
    keep = dict(desc=desc, W=W, X=X, G=G, out=out)
    return keep, dict(ms_concurrent=ms, ms_sequential=None, phases_ms=phases, launches=launches, clocks=clocks,
                      loss={proj.name: float(out.loss.sum().item())})


# --------------------------------------------------------------------------------------------
# the oracle on the host cores
# --------------------------------------------------------------------------------------------

def oracle_sample(cfg, n_tok_oracle=4096):
    """The float64 oracle, as it stands, on a bounded sample of `cfg`: the group loop (and scale
    refinement, where the configuration has it) of ONE head of the first projection, from a Hessian of
    n_tok_oracle tokens.  Returns (seconds, rows, description, cores)."""
    import oracle
    import oracle.problems as pu
    proj = cfg.projections[0]
    d, dh = proj.d_in, proj.d_head
    if cfg.name == "tiny":
        prob = pu.make_problem(0, d, 1, dh, 2048, hout="spd", gaussian_x=True)
    else:
        prob = pu.make_problem(0, d, 1, dh, n_tok_oracle, with_r=cfg.with_r)
    od = pu.oracle_desc(prob, cfg.bits, cfg.quant_group, cfg.out_block, config_flags(cfg))
    t0 = time.perf_counter()
    oracle.quantize_layer(od, prob["W"], prob["Hin"][0], prob["Uin"][0], prob["Hout"], prob["Uout"],
                          None if prob["R"] is None else prob["R"][0], None if prob["P"] is None else prob["P"][0],
                          None if prob["C"] is None else prob["C"][0])
    dt = time.perf_counter() - t0
    what = (f"group loop{' + scale refinement' if cfg.cd else ''}{' with R' if cfg.with_r else ''} and loss of 1 head "
            f"({dh} out-channels, {d} columns) of the {proj.name} projection; Hessians and factors not included")
    return dt, dh, what, oracle.num_threads()


def oracle_layer_estimate(cfg, dt_head, rows_head):
    """Seconds per layer extrapolated from one head: heads are independent and cost about the same
    per out-channel at equal width (the output projection has no compensation, so this over-estimates it
    slightly)."""
    width0 = cfg.projections[0].d_in
    return sum(dt_head * (p.d_out / rows_head) * (p.d_in / width0) ** 2 for p in cfg.projections)


def run_reference(args, cfg, rank):
    """--impl reference: the oracle on the same workload, one head of the first projection per step."""
    if rank != 0:
        return
    n_tok = args.tokens or cfg.n_tok
    dts = []
    rows, what, cores = 0, "", 0
    for i in range(args.warmup + args.steps):
        dt, rows, what, cores = oracle_sample(cfg)
        if i >= args.warmup:
            dts.append(dt)
        if sum(dts) > 120.0:   # keep the whole run within a few minutes
            break
    dt = float(np.mean(dts))
    value = rows / dt
    sample = what + f"; {len(dts)} timed step(s) of {args.steps} requested"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": len(dts), "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_summary(cfg, n_tok),
            "seconds_per_attention_layer_extrapolated": oracle_layer_estimate(cfg, dt, rows),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# --------------------------------------------------------------------------------------------
# report
# --------------------------------------------------------------------------------------------

def rooflines(cfg, n_tok, m, peaks):
    """Algorithmic work / measured time per kind of kernel, from the phase timers (for a block: the
    pass that runs one part after the other, so that no two kernels share the GPU while timed)."""
    ph = m["phases_ms"]
    bf16_peak = float(peaks.get("bf16_tflops_sustained", peaks.get("bf16_tflops", 1590.0)))
    bf16_kind = ("measured cuBLAS bf16, sustained (MEASURED_PEAKS.json)" if peaks else "fallback 1.59 PFLOP/s")
    out = {}

    def alu(name, kernel, flops, ms):
        if ms:
            ach = flops / (ms * 1e-3) / 1e12
            out[name] = {"kernel": kernel, "bound": "alu", "achieved": ach, "peak": FP64_ALU_PEAK_TFLOPS,
                         "unit": "TFLOP/s", "frac": ach / FP64_ALU_PEAK_TFLOPS, "peak_kind": FP64_KIND,
                         "frac_of_measured_fp32_ffma": ach / FP32_FFMA_MEASURED_TFLOPS, "ms": ms,
                         "traffic": NCU_TRAFFIC.get((cfg.name, kernel))}

    alu("sweep", "k_sweep_rows", sweep_flops(cfg), ph.get("sweep"))
    seg_fl = sum(16.0 * p.d_out * p.d_in * ((cfg.quant_group or p.d_in) + 1) for p in cfg.projections)
    alu("grid", "k_grid_tri", seg_fl, ph.get("grid"))
    alu("factor", "k_chol_panel + FP64 GEMM engine", factor_flops(cfg), ph.get("factor"))
    loop_ms = ph.get("grid", 0.0) + ph.get("sweep", 0.0) + ph.get("compensation", 0.0)
    alu("loop", "grid + sweep + compensation", loop_flops(cfg), loop_ms)
    if ph.get("hessian"):
        ach = hessian_flops(cfg, n_tok) / (ph["hessian"] * 1e-3) / 1e12
        out["hessian"] = {"kernel": "k_syrk_tc / k_syrk_tc_pair from 6144 columns on (+ mirror, finalize)", "bound": "tensor", "achieved": ach, "peak": bf16_peak,
                          "unit": "TFLOP/s", "frac": ach / bf16_peak, "peak_kind": bf16_kind, "ms": ph["hessian"],
                          "traffic": NCU_TRAFFIC.get((cfg.name, "k_syrk_tc")) if n_tok == NCU_TRAFFIC_TOKENS else None}
    return out, loop_ms


def config_entry(cfg, n_tok, m, peaks, oracle_info, steps):
    roofs, loop_ms = rooflines(cfg, n_tok, m, peaks)
    ph = m["phases_ms"]
    ms = m["ms_concurrent"]
    entry = {
        "workload": cfg.name, "config": config_summary(cfg, n_tok), "out_channels": out_channels(cfg),
        "seconds_per_layer": ms * 1e-3,
        "seconds_per_layer_sequential": None if m["ms_sequential"] is None else m["ms_sequential"] * 1e-3,
        "out_channels_per_s": out_channels(cfg) / (ms * 1e-3),
        "prerequisites_ms": {k: ph.get(k, 0.0) for k in ("hessian", "cross", "hout", "factor", "prep")},
        "quantize_ms": {k: ph.get(k, 0.0) for k in ("setup", "grid", "sweep", "compensation", "cd", "output", "loss")},
        "loop_ms": loop_ms, "loop_out_channels_per_s": out_channels(cfg) / (loop_ms * 1e-3) if loop_ms else None,
        "loop_frac_of_fp64_peak": roofs.get("loop", {}).get("frac"),
        "loop_frac_of_measured_fp32_ffma": roofs.get("loop", {}).get("frac_of_measured_fp32_ffma"),
        "rooflines": roofs, "loss": m["loss"], "gpu_launches_per_step": m["launches"] / max(steps, 1),
    }
    if oracle_info is not None:
        dt, rows, what, cores = oracle_info
        entry["oracle"] = {"seconds": dt, "out_channels": rows, "out_channels_per_s": rows / dt, "cores": cores,
                           "sample": what, "seconds_per_layer_extrapolated": oracle_layer_estimate(cfg, dt, rows)}
    return entry


def rank_seed(rank: int) -> int:
    """Every rank quantizes a layer of its own."""
    return int(rank)


def aggregate_value(cfg, world: int, max_ms_per_step: float) -> float:
    """Whole-job out-channels per second: every rank's layer over the slowest rank's step time."""
    return out_channels(cfg) * world / (max_ms_per_step * 1e-3)


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=8)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(tb_inputs.CONFIGS))
    ap.add_argument("--tokens", type=int, default=0, help="override the token count (default: the config's)")
    ap.add_argument("--heads", type=int, default=0,
                    help="single-projection workloads: keep only this many heads (small captures under a profiler)")
    ap.add_argument("--no-configs", action="store_true", help="skip the other four configurations")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args(argv)
    if args.warmup < 3:
        args.warmup = 3

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    cfg = tb_inputs.CONFIGS[args.workload]
    if args.heads and not is_block(cfg) and cfg.projections[0].partner:
        import dataclasses
        p0 = cfg.projections[0]
        cfg = dataclasses.replace(cfg, name=f"{cfg.name}[{args.heads} heads]",
                                  projections=(dataclasses.replace(p0, n_heads=args.heads,
                                                                   d_out=args.heads * p0.d_head),))
    if args.impl == "reference":
        run_reference(args, cfg, rank)
        return

    import torch
    import paper_2602_04929_b200 as tb
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the quantizer has no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    tb.load()

    def barrier():
        if dist is not None:
            dist.barrier()

    def max_over_ranks(v):
        if dist is None:
            return v
        t = torch.tensor([v], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    n_tok = args.tokens or cfg.n_tok
    sampler = ClockSampler(local_rank)
    if is_block(cfg):
        prob, m = measure_layer(cfg, n_tok, dev, rank_seed(rank), args.steps, args.warmup, min(args.steps, 3), barrier,
                                sampler)
    else:
        prob, m = measure_projection_config(cfg, n_tok, dev, rank_seed(rank), args.steps, args.warmup, barrier, sampler)
    ms_per_step = max_over_ranks(m["ms_concurrent"])

    # ---- end to end: the same layer through the same entry point from pinned host buffers ----
    e2e = None
    e2e_note = None
    if not args.no_e2e and is_block(cfg):
        avail = 0
        try:
            for ln in open("/proc/meminfo"):
                if ln.startswith("MemAvailable"):
                    avail = int(ln.split()[1]) * 1024
        except OSError:
            pass
        need_host = prob.activation_bytes + sum(w.numel() * 8 for w in prob.W) * 2
        if avail and need_host * world > 0.6 * avail:
            e2e_note = (f"skipped: {need_host * world / 2**30:.0f} GiB of pinned host memory needed by {world} rank(s), "
                        f"{avail / 2**30:.0f} GiB available on the host")
        else:
            hio, keep, h2d, d2h, need = prob.host_copies()
            hws = torch.empty(need, dtype=torch.uint8, device=dev)
            prob.desc.on_host, prob.desc.concurrent = 1, 1
            tb.tb_attention_layer(prob.desc, hio, hws)      # warm-up
            n_e2e = 2
            barrier()
            torch.cuda.synchronize()
            a = ev()
            for _ in range(n_e2e):
                tb.tb_attention_layer(prob.desc, hio, hws)
            b = ev()
            torch.cuda.synchronize()
            prob.desc.on_host = 0
            e2e_ms = max_over_ranks(a.elapsed_time(b) / n_e2e)
            e2e = {"value": aggregate_value(cfg, world, e2e_ms), "unit": UNIT, "ms_per_step": e2e_ms,
                   "steps": n_e2e, "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
                   "call": "tb_attention_layer with on_host = 1 (pinned host buffers)"}
            same = all(torch.equal(keep[6][i]["codes"], prob.outs[i]["codes"].cpu()) for i in range(4))
            e2e["codes_equal_device_path"] = bool(same)
            del hio, keep, hws
    elif not args.no_e2e and cfg.name != "tiny":
        # a single projection: tb_quantize_from_host
        proj = cfg.projections[0]
        desc, W, X, G, out = prob["desc"], prob["W"], prob["X"], prob["G"], prob["out"]
        Wp, Xp, Gp = W.cpu().pin_memory(), X.view(torch.int16).cpu().pin_memory(), G.cpu().pin_memory()
        ng = desc.n_groups
        outs = {"codes": torch.empty((proj.d_out, proj.d_in), dtype=torch.uint8).pin_memory(),
                "scales": torch.empty((proj.d_out, ng), dtype=torch.float32).pin_memory(),
                "zeros": torch.empty((proj.d_out, ng), dtype=torch.int32).pin_memory(),
                "w_hat": torch.empty((proj.d_out, proj.d_in), dtype=torch.float32).pin_memory(),
                "loss": torch.empty(proj.n_heads, dtype=torch.float64).pin_memory()}
        hws = torch.empty(tb.tb_quantize_from_host_workspace(desc, n_tok, proj.n_heads), dtype=torch.uint8, device=dev)
        tb.tb_quantize_from_host(desc, Wp, Xp, Gp, cfg.damp, cfg.damp, outs, hws)
        n_e2e = 3
        barrier()
        torch.cuda.synchronize()
        a = ev()
        for _ in range(n_e2e):
            tb.tb_quantize_from_host(desc, Wp, Xp, Gp, cfg.damp, cfg.damp, outs, hws)
        b = ev()
        torch.cuda.synchronize()
        e2e_ms = max_over_ranks(a.elapsed_time(b) / n_e2e)
        h2d = Wp.numel() * 4 + Xp.numel() * 2 + Gp.numel() * 4
        d2h = sum(v.numel() * v.element_size() for v in outs.values())
        e2e = {"value": aggregate_value(cfg, world, e2e_ms), "unit": UNIT, "ms_per_step": e2e_ms, "steps": n_e2e,
               "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h), "call": "tb_quantize_from_host",
               "codes_equal_device_path": bool(torch.equal(outs["codes"], out.codes.cpu()))}

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peaks = {}
    try:
        peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
    except OSError:
        pass
    del prob
    torch.cuda.empty_cache()

    # ---- the oracle on the host cores, and the other configurations (N = 1 only) ----
    oracle_main = None
    if world == 1 and not args.no_cpu_baseline:
        oracle_main = oracle_sample(cfg)
    head = config_entry(cfg, n_tok, m, peaks, oracle_main, args.steps)
    others = []
    if world == 1 and not args.no_configs:
        for name, c in tb_inputs.CONFIGS.items():
            if name == cfg.name:
                continue
            nt = c.n_tok
            k = 3 if is_block(c) else (5 if name == "tiny" else 10)
            if is_block(c):
                p2, m2 = measure_layer(c, nt, dev, 0, k, 3, 2)
            else:
                p2, m2 = measure_projection_config(c, nt, dev, 0, k, 3)
            del p2
            torch.cuda.empty_cache()
            others.append(config_entry(c, nt, m2, peaks, None if args.no_cpu_baseline else oracle_sample(c), k))

    roofs = head["rooflines"]
    # the dominant kernel of the hot loop (the group loop of Algorithm 1): the column sweep
    roofline = dict(roofs.get("sweep", {}))
    line = {
        "metric": METRIC, "value": aggregate_value(cfg, world, ms_per_step), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": dict(config_summary(cfg, n_tok),
                       l2="inputs larger than L2 (every activation tensor %.1f GiB)" % (n_tok * cfg.d_model * 2 / 2 ** 30)),
        "seconds_per_attention_layer": head["seconds_per_layer"],
        "seconds_per_attention_layer_sequential": head["seconds_per_layer_sequential"],
        "prerequisites_ms": head["prerequisites_ms"], "quantize_ms": head["quantize_ms"],
        "loop_ms": head["loop_ms"], "loop_out_channels_per_s": head["loop_out_channels_per_s"],
        "loop_roofline": roofs.get("loop"),
        "clocks": m["clocks"], "gpu_launches": int(m["launches"]),
        "roofline": roofline, "rooflines": roofs, "loss": head["loss"],
        "configs": others,
    }
    if e2e is not None:
        line["e2e"] = e2e
    elif e2e_note:
        line["e2e_note"] = e2e_note
    if oracle_main is not None:
        dt, rows, what, cores = oracle_main
        line["cpu_baseline"] = {"value": rows / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
                                "sample": what + f", {dt:.1f} s",
                                "seconds_per_layer_extrapolated": oracle_layer_estimate(cfg, dt, rows)}
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
