"""GPU parity of tb_quantize_layer against the float64 oracle on the same
seeded float32 inputs (stage-isolated: both sides get the same H, U, P, C).
Bar: codes, zero-points and grid candidates bit-exact after the guided
comparison (adoptions counted and printed), W_hat and scales within 1e-5
relative Frobenius error, per-head loss within 1e-4 relative."""
import numpy as np
import pytest

import tb_inputs
from parity_util import cached_problem, compare, make_problem, run_gpu

pytestmark = pytest.mark.gpu

ADAPT, CD = 1, 2


def _case(prob, bits, gq, g, flags, **kw):
    gpu = run_gpu(prob, bits, gq, g, flags, n_cand=kw.get("n_cand", 16), cd_iters=kw.get("cd_iters", 1))
    return compare(prob, gpu, bits, gq, g, flags, n_cand=kw.get("n_cand", 16), cd_iters=kw.get("cd_iters", 1),
                   heads=kw.get("heads"), raw_too=kw.get("raw_too", False), label=kw.get("label", ""))


def test_tiny_config_full():
    """Config 'tiny': 256x256, one head of 256 rows, explicit SPD H_out (cond 1e3),
    Gaussian activations with 4 outlier channels, INT4 per-channel, g = 8, adaptive grid + CD."""
    prob = make_problem(0, 256, 1, 256, 2048, hout="spd", gaussian_x=True)
    rep = _case(prob, 4, 0, 8, ADAPT | CD, raw_too=True, label="tiny")
    assert rep["gpu_stats"]["column_steps"] == 32 * 256


@pytest.mark.parametrize("g", [1, 4, 32, 64])
def test_group_sizes_including_boa_and_gptq_limits(g):
    """g = 1 is BoA's sequential rule; g = d_head has no compensation at all."""
    prob = make_problem(1, 256, 3, 64, 1024)
    _case(prob, 2, 128, g, ADAPT | CD, label=f"g={g}")


@pytest.mark.parametrize("bits,gq", [(2, 128), (3, 128), (4, 64), (3, 0), (8, 32)])
def test_bit_widths_and_column_groups(bits, gq):
    prob = make_problem(2, 384, 2, 64, 1024)
    _case(prob, bits, gq, 16, ADAPT | CD, label=f"b{bits}gq{gq}")


def test_static_grid_without_cd_is_boa_f1_mode():
    prob = make_problem(3, 256, 4, 32, 1024)
    _case(prob, 2, 128, 8, 0, label="static")


def test_identity_hout_is_gptq_mode():
    """H_out = NULL: every row at once, no compensation (GPTQ row of Table 1)."""
    prob = make_problem(4, 256, 2, 100, 1024, hout=None)
    _case(prob, 3, 128, 25, ADAPT | CD, label="gptq")


@pytest.mark.parametrize("hout", ["proj", None])
def test_propagated_error_terms(hout):
    """R != NULL: P term inside the sweep, C term in the compensation, R in CD and loss."""
    prob = make_problem(5, 256, 2, 64, 2048, with_r=True, hout=hout)
    _case(prob, 2, 128, 16, ADAPT | CD, label=f"R/{hout}")


def test_per_head_input_hessians():
    """The W_V row of Table 1: one H_in (and U_in, R, P, C) per head."""
    prob = make_problem(6, 256, 3, 32, 1024, with_r=True, n_hin=3)
    _case(prob, 3, 128, 8, ADAPT | CD, label="per-head H_in")


def test_per_head_input_hessians_without_scale_refinement():
    """One H_in per head, heads of 128 rows, no coordinate descent: the loss then forms (Q - W) H_in
    itself, the heads sharing one tensor-core launch, each against the pieces of its own H_in."""
    prob = make_problem(12, 256, 3, 128, 1024, n_hin=3, hout="spd")
    _case(prob, 3, 128, 32, ADAPT, label="per-head H_in, no CD")


def test_ragged_rows_and_candidate_counts():
    """Row counts that fill neither a panel CTA (8 rows) nor a GEMM tile; 5 and 32 candidates."""
    prob = make_problem(7, 384, 5, 21, 1024)
    _case(prob, 3, 128, 3, ADAPT | CD, n_cand=5, label="ragged/5cand")
    _case(prob, 3, 128, 7, ADAPT, n_cand=32, label="ragged/32cand")


def test_two_cd_passes():
    prob = make_problem(8, 256, 2, 32, 1024)
    _case(prob, 2, 128, 8, ADAPT | CD, cd_iters=2, label="cd2")


def test_degenerate_rows():
    """All-zero rows get s = 1, z = 0, code 0 and a zero CD denominator (skipped)."""
    prob = make_problem(9, 256, 2, 32, 1024)
    prob["W"][5] = 0.0
    prob["W"][40, :128] = 0.0
    _case(prob, 2, 128, 8, ADAPT | CD, label="degenerate")


def test_run_to_run_determinism():
    prob = make_problem(10, 256, 2, 32, 1024, with_r=True)
    a = run_gpu(prob, 2, 128, 8, ADAPT | CD)
    b = run_gpu(prob, 2, 128, 8, ADAPT | CD)
    for k in ("codes", "scales", "zeros", "cand", "w_hat", "loss"):
        assert np.array_equal(a[k], b[k]), k


def test_llama7b_q_proj_shape_sampled_heads():
    """Config 2 at full width (4096 x 4096, 32 heads x 128, INT2, group 128, g = 32,
    adaptive grid + CD) in the launch configuration the benchmark times.  The GPU runs all
    32 heads; the oracle recomputes two of them (heads are independent).  H_in comes from
    16384 heavy-tailed tokens so that the float64 Hessian and its factor stay affordable."""
    prob = make_problem(0, 4096, 32, 128, 16384)
    gpu = run_gpu(prob, 2, 128, 32, ADAPT | CD)
    rep = compare(prob, gpu, 2, 128, 32, ADAPT | CD, heads=[0, 21], label="7b-q sampled heads")
    assert rep["gpu_stats"]["column_steps"] == 4 * 4096


def test_llama7b_q_proj_with_propagated_error_sampled_head():
    """Config 3's q_proj: 4096 x 4096, 32 heads, INT2, group 128, g = 32, adaptive grid + CD, with the
    propagated-error operands R, P, C (alpha = 0.25) from a synthetic input deviation."""
    prob = cached_problem(0, 4096, 32, 128, 8192, with_r=True)
    gpu = run_gpu(prob, 2, 128, 32, ADAPT | CD)
    compare(prob, gpu, 2, 128, 32, ADAPT | CD, heads=[9], label="7b-q with R, sampled head")


def test_llama3_gqa_k_proj_shape_sampled_head():
    """Config 4's k_proj: 1024 x 4096, 8 key/value heads whose H_out sums 4 query heads each, INT3, g = 64."""
    prob = make_problem(1, 4096, 8, 128, 8192, g_heads=32)
    gpu = run_gpu(prob, 3, 128, 64, ADAPT | CD)
    compare(prob, gpu, 3, 128, 64, ADAPT | CD, heads=[5], label="8b-k GQA, sampled head")


def test_o_proj_identity_hout_sampled_rows():
    """o_proj of the block configs: H_out = NULL (all 4096 rows at once); the oracle recomputes 128 of them."""
    prob = make_problem(2, 4096, 32, 128, 8192, hout=None)
    gpu = run_gpu(prob, 2, 128, 32, ADAPT | CD)
    compare(prob, gpu, 2, 128, 32, ADAPT | CD, heads=[3], label="o_proj GPTQ mode, sampled rows")


def test_v_proj_per_head_hessians_full_width():
    """v_proj row of Table 1 at full width: every head has its own H_in = X-bar_h^T X-bar_h with
    X-bar_h = A_h X (synthetic causal decay per head), its own factor, and H_out from the output
    projection side (here an explicit SPD block).  Two heads of 128 rows, 4096 wide, INT2, g = 32."""
    prob = make_problem(4, 4096, 2, 128, 4096, n_hin=2, hout="spd", vmix_seq=2048)
    gpu = run_gpu(prob, 2, 128, 32, ADAPT | CD)
    compare(prob, gpu, 2, 128, 32, ADAPT | CD, heads=[1], label="v_proj per-head H_in, sampled head")


@pytest.mark.parametrize("g", [32, 1, 8, 64, 128])
def test_llama70b_q_proj_shape_sampled_head(g):
    """Config 5's q_proj: 8192 x 8192, 64 heads x 128, INT2, group 128, fixed grid, no CD (the paper's
    'BoA + joint quantization' setting), over the whole sweep of out-blocks: g = 1 is BoA's sequential
    rule, g = 128 = d_head has no compensation left (GPTQ)."""
    prob = cached_problem(3, 8192, 64, 128, 8192)
    gpu = run_gpu(prob, 2, 128, g, 0)
    compare(prob, gpu, 2, 128, g, 0, heads=[37], label=f"70b-q g={g}, sampled head")


def test_llama70b_q_proj_adaptive_grid_and_scale_refinement_sampled_head():
    """Config 5's secondary setting: 8192 wide, adaptive grid + coordinate descent at g = 32.  With 64
    column groups per row the scale refinement takes the row-walking kernel (more groups than the
    column-parallel pass holds)."""
    prob = cached_problem(3, 8192, 64, 128, 8192)
    gpu = run_gpu(prob, 2, 128, 32, ADAPT | CD)
    compare(prob, gpu, 2, 128, 32, ADAPT | CD, heads=[11], label="70b-q adaptive + CD, sampled head")


@pytest.mark.parametrize("flags", [0, ADAPT | CD])
def test_llama70b_kv_proj_shape_sampled_head(flags):
    """Config 5's k_proj / v_proj shape: 1024 x 8192, 8 key/value heads whose H_out sums 8 query heads
    each, INT2, g = 32: 256 rows per step, the cluster form of the sweep over 64 column blocks."""
    prob = cached_problem(3, 8192, 8, 128, 8192, g_heads=64)
    gpu = run_gpu(prob, 2, 128, 32, flags)
    compare(prob, gpu, 2, 128, 32, flags, heads=[5], label=f"70b-k GQA flags={flags}, sampled head")


def test_llama70b_v_proj_per_head_hessians_sampled_head():
    """8192 wide with one H_in per head (the W_V row of Table 1): two heads, each with its own
    attention-weighted inputs, Hessian and factor; fixed grid, no CD, g = 32."""
    prob = cached_problem(5, 8192, 2, 128, 4096, n_hin=2, hout="spd", vmix_seq=2048)
    gpu = run_gpu(prob, 2, 128, 32, 0)
    compare(prob, gpu, 2, 128, 32, 0, heads=[1], label="70b-v per-head H_in, sampled head")


@pytest.mark.parametrize("d_in,gq,with_r", [(4352, 128, False), (1152, 32, True), (4352, 128, True)])
def test_scale_refinement_with_more_than_32_column_groups(d_in, gq, with_r):
    """More column groups per row than the column-parallel pass of Algorithm 3 holds (34 and 36): the
    row-walking kernel runs, fed by the tensor-core blockwise product (groups of 128 columns) or by
    the plain one (groups of 32)."""
    prob = make_problem(13, d_in, 2, 32, 2048, with_r=with_r)
    _case(prob, 3, gq, 8, ADAPT | CD, label=f"CD row walk d_in={d_in} gq={gq} R={with_r}")
    _case(prob, 2, gq, 16, ADAPT | CD, cd_iters=2, label=f"CD row walk, two passes, d_in={d_in}")


DYN = 4


@pytest.mark.parametrize("gq,with_r,n_hin", [(128, False, 1), (64, True, 1), (32, False, 1), (128, True, 2)])
def test_dynamic_column_group_grid(gq, with_r, n_hin):
    """Variant of the column-group reading: a group's (scale, zero) is searched when the sweep arrives at
    the group, from the values the error feedback of the earlier columns has left there.  Same parity
    bar as the default mode; with and without the propagated-error term, shared and per-head H_in,
    with the scale refinement after it."""
    prob = make_problem(15, 384, 2, 64, 1024, with_r=with_r, n_hin=n_hin)
    _case(prob, 3, gq, 16, DYN | CD, label=f"dynamic grid gq={gq} R={with_r} n_hin={n_hin}")
    _case(prob, 2, gq, 64, DYN, label=f"dynamic grid gq={gq}, g = d_head, no CD")


def test_dynamic_grid_special_cases():
    """One group per row: the variant is the adaptive grid, bit for bit.  H_out = NULL mode runs it too.
    Groups wider than 128 columns are refused."""
    import paper_2602_04929_b200 as tb
    prob = make_problem(16, 256, 2, 32, 1024)
    a = run_gpu(prob, 3, 0, 8, DYN | CD)
    b = run_gpu(prob, 3, 0, 8, ADAPT | CD)
    for k in ("codes", "scales", "zeros", "cand", "w_hat", "loss"):
        assert np.array_equal(a[k], b[k]), k
    prob_id = make_problem(16, 256, 2, 32, 1024, hout=None)
    _case(prob_id, 3, 64, 32, DYN | CD, label="dynamic grid, GPTQ mode")
    with pytest.raises(tb.TurboBoAError):
        run_gpu(make_problem(16, 512, 1, 32, 1024), 3, 256, 8, DYN)


def test_dynamic_grid_full_width_sampled_head():
    """4096 wide, 32 heads, INT2, groups of 128, g = 32, dynamic grid + CD; one sampled head."""
    prob = cached_problem(0, 4096, 32, 128, 8192, with_r=True)
    gpu = run_gpu(prob, 2, 128, 32, DYN | CD)
    compare(prob, gpu, 2, 128, 32, DYN | CD, heads=[17], label="7b-q dynamic grid with R, sampled head")


def test_near_constant_segment_under_the_fixed_grid():
    """A row segment whose original range is tiny gets a tiny scale from the fixed grid; after the
    compensation of earlier groups its pre-rounding values lie far outside the code range (and outside
    what a 32-bit integer holds).  Codes must clamp exactly as the oracle's do."""
    prob = make_problem(14, 256, 2, 32, 1024)
    prob["W"][8:, :128] *= np.float32(1e-12)     # scale ~ 4e-14: the compensated values are ~ 1e10 code units
    prob["W"][40, 128:] *= np.float32(1e-9)      # ~ 1e7 code units: far outside the codes, inside 32 bits
    rep = _case(prob, 2, 128, 8, 0, label="near-constant segment, fixed grid")
    assert rep["gpu_stats"]["clamped_codes"] > 0


@pytest.mark.parametrize("with_partner,n_tok", [(True, 5000), (False, 2048)])
def test_host_entry_point_matches_the_device_path(with_partner, n_tok):
    """tb_quantize_from_host chains the same calls (X crosses in pieces, H_out and its factor on
    the helper stream): its outputs must equal, bit for bit, those of the separate calls on
    device-resident inputs."""
    import torch
    import paper_2602_04929_b200 as tb
    d, H, dh = 256, 4, 64
    W_h = tb_inputs.weight(11, H * dh, d)
    G_h = tb_inputs.weight(11, H * dh, d, tid=tb_inputs.T_WPARTNER) if with_partner else None
    X_h = tb_inputs.HeavyTailRecipe(d, seed=11).chunk(0, n_tok)
    Xb = torch.from_numpy(X_h).to(torch.bfloat16)
    desc = tb.layer_desc(H * dh, d, H, dh, 3, 64, 16 if with_partner else dh, flags=3)
    dev = torch.device("cuda:0")
    # separate calls
    X = Xb.to(dev)
    W = torch.from_numpy(W_h).to(dev)
    Hin = torch.zeros((d, d), dtype=torch.float32, device=dev)
    Hsum = torch.empty_like(Hin)
    tb.tb_accumulate_hessian(Hin, X)
    tb.tb_finalize_hessian(Hin, None, n_tok, 0.01, Hsum_out=Hsum)
    Uin, info = tb.tb_factor(Hin)
    Hout = Uout = None
    if with_partner:
        Hout = tb.tb_build_hout(torch.from_numpy(G_h).to(dev), Hsum, H, dh, 0.01)
        Uout, info_out = tb.tb_factor(Hout)
    res = tb.tb_quantize_layer(desc, W, Hin, Uin, Hout, Uout, want_loss=True)
    torch.cuda.synchronize()
    # one call from pinned host buffers
    ng = desc.n_groups
    outs = {"codes": torch.empty((H * dh, d), dtype=torch.uint8).pin_memory(),
            "scales": torch.empty((H * dh, ng), dtype=torch.float32).pin_memory(),
            "zeros": torch.empty((H * dh, ng), dtype=torch.int32).pin_memory(),
            "w_hat": torch.empty((H * dh, d), dtype=torch.float32).pin_memory(),
            "loss": torch.empty(H, dtype=torch.float64).pin_memory()}
    ws = torch.empty(tb.tb_quantize_from_host_workspace(desc, n_tok, H if with_partner else 0), dtype=torch.uint8,
                     device=dev)
    Gp = torch.from_numpy(G_h).pin_memory() if with_partner else None
    for _ in range(2):  # the second call reuses the helper stream and the workspace
        tb.tb_quantize_from_host(desc, torch.from_numpy(W_h).pin_memory(), Xb.view(torch.int16).pin_memory(), Gp, 0.01,
                                 0.01, outs, ws)
        assert tb.tb_device_error_flag() == 0
        assert torch.equal(outs["codes"], res.codes.cpu())
        assert torch.equal(outs["zeros"], res.zeros.cpu())
        assert torch.equal(outs["scales"], res.scales.cpu())
        assert torch.equal(outs["w_hat"], res.w_hat.cpu())
        assert torch.equal(outs["loss"], res.loss.cpu())


def test_whole_path_from_host_against_the_oracle_chain():
    """Chained comparison: tb_quantize_from_host (Hessian, H_out, both factors, loop, scale refinement,
    all on the GPU from the raw activations) against the oracle run from the same X with its own float64
    Hessian, factors and H_out.  The two chains do not see the same H_in (the GPU's is accumulated in
    float: about 1e-6 relative), so a rounding decision whose pre-rounding value lies within that
    distance of a boundary may fall the other way and every later code of its row then differs: codes
    are compared as a mismatching fraction of ROWS, reported, and the result is judged on the loss.
      (i)  the GPU's reported loss against the float64 loss of the GPU's own W_hat under the ORACLE's
           Hessians: 1e-4 relative (the two differ by the Hessians' 1e-6 and float rounding of W_hat);
      (ii) the GPU's loss against the oracle chain's loss per head: a diverged row is another outcome of
           the same greedy procedure, whose row loss differs by a few percent; with at most a few rows
           diverged per head the head loss moves by far less than 2 %, which is the bound asserted."""
    import torch
    import oracle
    import paper_2602_04929_b200 as tb
    d, H, dh, n_tok = 256, 4, 64, 6144
    bits, gq, g, flags = 3, 64, 16, ADAPT | CD
    W_h = tb_inputs.weight(21, H * dh, d)
    G_h = tb_inputs.weight(21, H * dh, d, tid=tb_inputs.T_WPARTNER)
    X_h = tb_inputs.HeavyTailRecipe(d, seed=21).chunk(0, n_tok)
    desc = tb.layer_desc(H * dh, d, H, dh, bits, gq, g, flags=flags)
    ng = desc.n_groups
    outs = {"codes": torch.empty((H * dh, d), dtype=torch.uint8).pin_memory(),
            "scales": torch.empty((H * dh, ng), dtype=torch.float32).pin_memory(),
            "zeros": torch.empty((H * dh, ng), dtype=torch.int32).pin_memory(),
            "w_hat": torch.empty((H * dh, d), dtype=torch.float32).pin_memory(),
            "loss": torch.empty(H, dtype=torch.float64).pin_memory()}
    ws = torch.empty(tb.tb_quantize_from_host_workspace(desc, n_tok, H), dtype=torch.uint8, device="cuda:0")
    tb.tb_quantize_from_host(desc, torch.from_numpy(W_h).pin_memory(),
                             torch.from_numpy(X_h).to(torch.bfloat16).view(torch.int16).pin_memory(),
                             torch.from_numpy(G_h).pin_memory(), 0.01, 0.01, outs, ws)
    assert tb.tb_device_error_flag() == 0
    # the oracle's own chain, float64 throughout
    Hin, Hsum = oracle.hessian(X_h, damp=0.01, return_sum=True)
    Uin = oracle.factor_upper(Hin)
    Hout = oracle.hout_from_projection(G_h, Hsum, H, dh, damp=0.01)
    Uout = oracle.factor_upper(Hout)
    od = oracle.OracleDesc(H * dh, d, H, dh, bits=bits, quant_group=gq, out_block=g, flags=flags)
    ref = oracle.quantize_layer(od, W_h, Hin, Uin, Hout, Uout)
    codes, w_hat, loss = outs["codes"].numpy(), outs["w_hat"].numpy(), outs["loss"].numpy()
    rows_diff = int(np.count_nonzero((codes != ref.codes).any(axis=1)))
    own = np.array([oracle.loss_head(W_h[h * dh:(h + 1) * dh], w_hat[h * dh:(h + 1) * dh], Hin, Hout[h])
                    for h in range(H)])
    rel_own = float(np.max(np.abs(loss - own) / own))
    rel_chain = float(np.max(np.abs(loss - ref.loss) / ref.loss))
    print("CHAIN", dict(rows=H * dh, rows_with_a_different_code=rows_diff, loss_vs_own_w_hat=rel_own,
                        loss_vs_oracle_chain=rel_chain))
    assert rel_own <= 1e-4
    assert rel_chain <= (1e-4 if rows_diff == 0 else 2e-2)   # identical codes: only the Hessians' rounding is left
    assert rows_diff <= H * dh // 4
