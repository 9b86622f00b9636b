"""Problem construction for the parity tests and for the timed CPU baseline
(TEST INFRASTRUCTURE, not a product path): float32 inputs of one projection
from the seeded recipes of tb_inputs, with every derived tensor (Hessians,
factors, propagated-error operands, H_out) computed by this oracle in float64
and rounded to float once.  Nothing here comes from the CUDA path.
"""
from __future__ import annotations

import numpy as np

import tb_inputs

from . import ref as oracle


def f32(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.float32)


_INPUT_SIDE = {}


def _input_side(seed, d_in, n_tok, u, with_r, damp, alpha, gaussian_x, vmix_seq):
    """H_in, its undamped form, U_in (and R, P, C) of input-Hessian unit u, kept per process: the
    float64 Hessian and its factor dominate the cost of a wide problem and depend on these
    arguments only (not on the heads or on the out-channel side)."""
    key = (seed, d_in, n_tok, u, with_r, damp, alpha, gaussian_x, vmix_seq)
    if key in _INPUT_SIDE:
        return _INPUT_SIDE[key]
    if vmix_seq:
        # value projection: head u sees the attention-weighted inputs A_u X of the same tokens
        base = tb_inputs.HeavyTailRecipe(d_in, seed=seed).chunk(0, n_tok)
        X, Xfp = tb_inputs.causal_decay_mix(base, tb_inputs.decay_rate(u), vmix_seq), None
    elif gaussian_x:
        X = tb_inputs.activations_gaussian(seed + 101 * u, n_tok, d_in)
        Xfp = None
    else:
        rec = tb_inputs.HeavyTailRecipe(d_in, seed=seed, tid_shift=u)
        if with_r:
            X, Xfp = tb_inputs.DeviationRecipe(rec).chunk(0, n_tok)
        else:
            X, Xfp = rec.chunk(0, n_tok), None
    H, Hs = oracle.hessian(X, damp=damp, return_sum=True)
    H32 = f32(H)
    U32 = f32(oracle.factor_upper(H32))
    out = dict(Hin=H32, Hsum=f32(Hs), Uin=U32, R=None, P=None, C=None)
    if with_r:
        R32 = f32(oracle.cross_correlation(X, Xfp, alpha))
        Pm, Cm = oracle.correction_operands(R32, U32)
        out.update(R=R32, P=f32(Pm), C=f32(Cm))
    _INPUT_SIDE[key] = out
    return out


def make_problem(seed, d_in, n_heads, d_head, n_tok, *, with_r=False, hout="proj", n_hin=1,
                 g_heads=None, damp=0.01, alpha=0.25, gaussian_x=False, vmix_seq=None):
    """float32 inputs of one projection, every derived tensor computed by the oracle."""
    d_out = n_heads * d_head
    W = tb_inputs.weight(seed, d_out, d_in)
    units = [_input_side(seed, d_in, n_tok, u, with_r, damp, alpha, gaussian_x, vmix_seq) for u in range(n_hin)]
    prob = dict(W=W, Hin=np.stack([u["Hin"] for u in units]), Uin=np.stack([u["Uin"] for u in units]),
                Hsum=units[0]["Hsum"], d_out=d_out, d_in=d_in, n_heads=n_heads, d_head=d_head, n_hin=n_hin,
                R=None, P=None, C=None, Hout=None, Uout=None)
    if with_r:
        prob.update(R=np.stack([u["R"] for u in units]), P=np.stack([u["P"] for u in units]),
                    C=np.stack([u["C"] for u in units]))
    if hout == "proj":
        gh = g_heads or n_heads
        G = tb_inputs.weight(seed, gh * d_head, d_in, tid=tb_inputs.T_WPARTNER)
        Ho = f32(oracle.hout_from_projection(G, units[0]["Hsum"], n_heads, d_head, damp=damp))
        prob.update(G=G, Hout=Ho, Uout=f32(oracle.factor_upper(Ho)))
    elif hout == "spd":
        Ho = np.stack([tb_inputs.spd_matrix(seed + h, d_head, cond=1e3) for h in range(n_heads)])
        prob.update(Hout=Ho, Uout=f32(oracle.factor_upper(Ho)))
    return prob


_PROBLEMS = {}


def cached_problem(*args, **kw):
    """make_problem, kept for the tests of one process that share a large problem (read-only use)."""
    key = (args, tuple(sorted(kw.items())))
    if key not in _PROBLEMS:
        _PROBLEMS[key] = make_problem(*args, **kw)
    return _PROBLEMS[key]


def oracle_desc(prob, bits, quant_group, out_block, flags, n_cand=16, cd_iters=1, n_heads=None):
    H = n_heads or prob["n_heads"]
    return oracle.OracleDesc(d_out=H * prob["d_head"], d_in=prob["d_in"], n_heads=H, d_head=prob["d_head"],
                             bits=bits, quant_group=quant_group, out_block=out_block,
                             n_hin=1 if prob["n_hin"] == 1 else H, n_cand=n_cand, cd_iters=cd_iters, flags=flags)


