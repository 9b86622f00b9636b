"""Shared pieces of the GPU parity tests: problem construction from the seeded
input recipes (all Hessians and factors come from the float64 oracle, never
from the CUDA path) and the guided comparison of a GPU result with the oracle.

Guided comparison.  Codes are decisions inside an error-feedback chain, so a
single legitimately different rounding at an exact tie changes every later code
of its row.  The oracle therefore receives the GPU's codes / zero-points /
grid candidates as hints and adopts a hint only where its own pre-rounding
value lies within 1e-6 of the boundary (or, for a candidate, where the two
scores agree to 1e-9 relative).  Every adoption is counted and reported; all
other decisions are the oracle's own and must match bit for bit.
"""
from __future__ import annotations

import numpy as np

import oracle
from oracle.problems import cached_problem, f32, make_problem, oracle_desc  # noqa: F401

BAND = 1e-6        # code units; the band inside which a rounding decision may differ
CAND_TOL = 1e-9    # relative score gap below which two grid candidates count as tied
TOL_W = 1e-5       # relative Frobenius error on W_hat, on the scales and on the compensated weights
TOL_LOSS = 1e-4    # relative error on the Hessian-weighted loss


def run_gpu(prob, bits, quant_group, out_block, flags, n_cand=16, cd_iters=1, want_loss=True):
    import torch
    import paper_2602_04929_b200 as tb

    dev = torch.device("cuda:0")

    def t(a):
        return None if a is None else torch.from_numpy(np.ascontiguousarray(a)).to(dev)

    desc = tb.layer_desc(prob["d_out"], prob["d_in"], prob["n_heads"], prob["d_head"], bits, quant_group,
                         out_block, n_hin=prob["n_hin"], n_cand=n_cand, cd_iters=cd_iters, flags=flags)
    res = tb.tb_quantize_layer(desc, t(prob["W"]), t(prob["Hin"]), t(prob["Uin"]), t(prob["Hout"]),
                               t(prob["Uout"]), t(prob["R"]), t(prob["P"]), t(prob["C"]), want_loss=want_loss, want_w_comp=True)
    torch.cuda.synchronize()
    assert tb.tb_device_error_flag() == 0, "a bounded device-side wait ran out"
    return dict(codes=res.codes.cpu().numpy(), scales=res.scales.cpu().numpy(), zeros=res.zeros.cpu().numpy(),
                cand=res.cand.cpu().numpy(), w_hat=res.w_hat.cpu().numpy(), w_comp=res.w_comp.cpu().numpy(),
                loss=None if res.loss is None else res.loss.cpu().numpy(), stats=res.stats_dict())


def head_rows(prob, heads):
    dh = prob["d_head"]
    return np.concatenate([np.arange(h * dh, (h + 1) * dh) for h in heads])


def run_oracle(prob, gpu, bits, quant_group, out_block, flags, n_cand=16, cd_iters=1, heads=None,
               guided=True):
    """Oracle on all heads, or on the listed heads only (heads are independent)."""
    heads = list(range(prob["n_heads"])) if heads is None else list(heads)
    rows = head_rows(prob, heads)
    od = oracle_desc(prob, bits, quant_group, out_block, flags, n_cand, cd_iters, n_heads=len(heads))

    def per_head(a):
        return None if a is None else a[heads]

    per_unit = (lambda a: a if a is None else a[0]) if prob["n_hin"] == 1 else per_head
    hints = {}
    if guided:
        hints = dict(hint_codes=gpu["codes"][rows], hint_zeros=gpu["zeros"][rows], hint_cand=gpu["cand"][rows],
                     band=BAND, cand_tol=CAND_TOL)
    res = oracle.quantize_layer(od, prob["W"][rows], per_unit(prob["Hin"]), per_unit(prob["Uin"]),
                                per_head(prob["Hout"]), per_head(prob["Uout"]), per_unit(prob["R"]),
                                per_unit(prob["P"]), per_unit(prob["C"]), **hints)
    return res, rows


def rel_fro(a, b):
    a = np.asarray(a, np.float64)
    b = np.asarray(b, np.float64)
    den = np.linalg.norm(b)
    return float(np.linalg.norm(a - b) / den) if den > 0 else float(np.linalg.norm(a - b))


def compare(prob, gpu, bits, quant_group, out_block, flags, n_cand=16, cd_iters=1, heads=None,
            raw_too=False, label=""):
    """Asserts the parity bar and returns the report (also printed)."""
    res, rows = run_oracle(prob, gpu, bits, quant_group, out_block, flags, n_cand, cd_iters, heads)
    hsel = list(range(prob["n_heads"])) if heads is None else list(heads)
    rep = dict(label=label, rows=len(rows), elements=int(gpu["codes"][rows].size), **res.counters)
    rep["code_mismatch"] = int(np.count_nonzero(gpu["codes"][rows] != res.codes))
    rep["zero_mismatch"] = int(np.count_nonzero(gpu["zeros"][rows] != res.zeros))
    rep["cand_mismatch"] = int(np.count_nonzero(gpu["cand"][rows] != res.cand))
    rep["scales_rel"] = rel_fro(gpu["scales"][rows], res.scales)
    rep["w_hat_rel"] = rel_fro(gpu["w_hat"][rows], res.w_hat)
    # compensated weights: every row as it stood when its group was taken (the oracle's snapshot W0)
    rep["w_comp_rel"] = rel_fro(gpu["w_comp"][rows], res.w_comp)
    if gpu["loss"] is not None:
        lg, lo = gpu["loss"][hsel], res.loss
        rep["loss_rel"] = float(np.max(np.abs(lg - lo) / np.maximum(np.abs(lo), 1e-300)))
    if raw_too:
        raw, _ = run_oracle(prob, gpu, bits, quant_group, out_block, flags, n_cand, cd_iters, heads, guided=False)
        rep["raw_code_mismatch"] = int(np.count_nonzero(gpu["codes"][rows] != raw.codes))
    rep["gpu_stats"] = gpu["stats"]
    print("PARITY", rep)
    assert rep["code_mismatch"] == 0, rep
    assert rep["zero_mismatch"] == 0, rep
    assert rep["cand_mismatch"] == 0, rep
    assert rep["scales_rel"] <= TOL_W, rep
    assert rep["w_hat_rel"] <= TOL_W, rep
    assert rep["w_comp_rel"] <= TOL_W, rep
    if "loss_rel" in rep:
        assert rep["loss_rel"] <= TOL_LOSS, rep
    return rep
