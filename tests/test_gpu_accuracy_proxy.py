"""Accuracy proxies that need no model: the Hessian-weighted layer loss (the objective in the proofs
of Propositions 3.1 / 3.2) as a function of the out-block N (the paper's Table 2 varies N) and of the
number of coordinate-descent passes (App. F.4, Table 9), on the synthetic 4096-wide and 8192-wide
q_proj shapes.  Every point is the GPU's loss over all heads, with the oracle's value for one sampled
head beside the GPU's for that head (1e-4 relative, codes bit-exact: the full parity bar).  Printed as
PROXY lines; `profiles/accuracy_proxy.md` is made from them."""
import json

import numpy as np
import pytest

from parity_util import cached_problem, compare, run_gpu

pytestmark = pytest.mark.gpu
ADAPT, CD = 1, 2


def _point(shape, prob, bits, gq, g, flags, head, cd_iters=1):
    gpu = run_gpu(prob, bits, gq, g, flags, cd_iters=cd_iters)
    rep = compare(prob, gpu, bits, gq, g, flags, cd_iters=cd_iters, heads=[head], label=f"{shape} g={g} flags={flags}")
    rec = dict(shape=shape, out_block=g, flags=flags, cd_iters=cd_iters if flags & CD else 0,
               loss_all_heads=float(gpu["loss"].sum()), loss_sampled_head_gpu=float(gpu["loss"][head]),
               loss_sampled_head_rel_to_oracle=rep["loss_rel"])
    print("PROXY", json.dumps(rec))
    return rec


def test_loss_versus_out_block_4096_wide():
    """Adaptive grid + one CD pass, N in {1, 8, 32, 64, 128}.  N = 1 is BoA's sequential rule, N = 128 =
    d_head leaves nothing to compensate: the loss can only grow with N, and on these synthetic layers it
    does (the paper reports the effect on perplexity as small up to N = 64; that needs the models)."""
    prob = cached_problem(0, 4096, 32, 128, 16384)
    pts = [_point("4096x4096", prob, 2, 128, g, ADAPT | CD, head=21) for g in (1, 8, 32, 64, 128)]
    loss = [p["loss_all_heads"] for p in pts]
    assert all(b >= a for a, b in zip(loss, loss[1:]))        # less compensation, more loss
    assert loss[2] <= 1.5 * loss[0]                            # N = 32 stays within 50 % of the sequential rule here


def test_loss_versus_cd_passes_4096_wide():
    """cd_iters in {0, 1, 2} at N = 32: non-increasing, and the first pass gives most of the drop."""
    prob = cached_problem(0, 4096, 32, 128, 16384)
    l0 = _point("4096x4096", prob, 2, 128, 32, ADAPT, head=3)["loss_all_heads"]
    l1 = _point("4096x4096", prob, 2, 128, 32, ADAPT | CD, head=3, cd_iters=1)["loss_all_heads"]
    l2 = _point("4096x4096", prob, 2, 128, 32, ADAPT | CD, head=3, cd_iters=2)["loss_all_heads"]
    assert l2 <= l1 <= l0
    assert (l0 - l1) >= (l1 - l2)


def test_loss_versus_out_block_8192_wide_static_grid():
    """The 70B-shaped q_proj in the paper's 'BoA + joint quantization' setting (fixed grid, no CD)."""
    prob = cached_problem(3, 8192, 64, 128, 8192)
    pts = [_point("8192x8192", prob, 2, 128, g, 0, head=50) for g in (1, 32, 128)]
    loss = [p["loss_all_heads"] for p in pts]
    assert loss[0] <= loss[1] <= loss[2]
