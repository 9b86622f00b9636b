"""Block level (Algorithm 1's loop over the projections of an attention layer): tb_quantize_block
against separate tb_quantize_layer calls, and tb_attention_layer against the same chain made of
single calls (bit for bit, device- and host-resident) and against the oracle's own float64 chain
(Table 1's pairing of projections and out-channel Hessians, judged on the loss)."""
import numpy as np
import pytest

import oracle
import tb_inputs
from parity_util import make_problem

pytestmark = pytest.mark.gpu

ADAPT, CD = 1, 2
NAMES = ("q", "k", "v", "o")


def _dev(a, dtype=None):
    import torch
    t = torch.from_numpy(np.ascontiguousarray(a)).to("cuda:0")
    return t if dtype is None else t.to(dtype)


@pytest.mark.parametrize("concurrent", [False, True])
def test_quantize_block_equals_separate_calls(concurrent):
    import torch
    import paper_2602_04929_b200 as tb
    probs = [make_problem(31, 256, 4, 64, 2048, with_r=True), make_problem(32, 256, 2, 64, 2048, g_heads=4),
             make_problem(33, 384, 1, 256, 2048, hout=None)]
    settings = [(2, 128, 16, ADAPT | CD), (3, 64, 32, ADAPT | CD), (4, 128, 256, ADAPT)]
    jobs, outs, refs, keep = [], [], [], []
    for prob, (bits, gq, g, flags) in zip(probs, settings):
        desc = tb.layer_desc(prob["d_out"], prob["d_in"], prob["n_heads"], prob["d_head"], bits, gq, g, flags=flags)
        t = {k: (None if prob[k] is None else _dev(prob[k])) for k in ("W", "Hin", "Uin", "Hout", "Uout", "R", "P", "C")}
        refs.append(tb.tb_quantize_layer(desc, t["W"], t["Hin"], t["Uin"], t["Hout"], t["Uout"], t["R"], t["P"], t["C"],
                                         want_w_comp=True))
        out = tb.empty_result(desc, "cuda:0", want_w_comp=True)
        ws = torch.empty(tb.tb_quantize_layer_workspace(desc, t["R"] is not None, True), dtype=torch.uint8, device="cuda:0")
        jobs.append(tb.projection_job(desc, t["W"], t["Hin"], t["Uin"], t["Hout"], t["Uout"], t["R"], t["P"], t["C"], out, ws))
        outs.append(out)
        keep.append((t, ws))
    tb.tb_quantize_block(jobs, concurrent=concurrent)
    torch.cuda.synchronize()
    assert tb.tb_device_error_flag() == 0
    for out, ref in zip(outs, refs):
        for k in ("codes", "scales", "zeros", "cand", "w_hat", "w_comp", "loss"):
            assert torch.equal(getattr(out, k), getattr(ref, k)), k
    if concurrent:   # a shared workspace is refused before anything is launched
        jobs[1].ws = jobs[0].ws
        with pytest.raises(tb.TurboBoAError):
            tb.tb_quantize_block(jobs, concurrent=True)


def _layer_inputs(seed, d, hq, hkv, dh, n_tok, with_r, per_head_v):
    dq = hq * dh
    W = [tb_inputs.weight(seed, dq, d), tb_inputs.weight(seed, hkv * dh, d, tid=tb_inputs.T_WPARTNER),
         tb_inputs.weight(seed + 1, hkv * dh, d), tb_inputs.weight(seed, d, dq, tid=tb_inputs.T_WOUT)]
    rec = tb_inputs.HeavyTailRecipe(d, seed=seed)
    rec_o = tb_inputs.HeavyTailRecipe(dq, seed=seed, tid_shift=1)
    if with_r:
        X, Xfp = tb_inputs.DeviationRecipe(rec).chunk(0, n_tok)
        Xo, Xofp = tb_inputs.DeviationRecipe(rec_o).chunk(0, n_tok)
    else:
        X, Xfp, Xo, Xofp = rec.chunk(0, n_tok), None, rec_o.chunk(0, n_tok), None
    Xv = None
    if per_head_v:
        Xv = np.stack([tb_inputs.causal_decay_mix(X, tb_inputs.decay_rate(h), 2048) for h in range(hkv)])
    return W, X, Xfp, Xv, Xo, Xofp


def _manual_chain(tb, desc, W, X, Xfp, Xv, Xo, Xofp, piece=None):
    """The layer out of single C-ABI calls on device-resident tensors.  piece: accumulate the
    statistics over token pieces of this size, as the host-buffer mode does (the Hessian's sums do not
    depend on it; the deviation correlation sums its two bf16 pieces per call, so its float sums do)."""
    import torch
    d, hq, hkv, dh, n_tok = desc.d_model, desc.n_q_heads, desc.n_kv_heads, desc.d_head, desc.n_tok

    def input_side(Xd, Xfpd, width):
        H = torch.zeros((width, width), dtype=torch.float32, device="cuda:0")
        R = torch.zeros_like(H) if Xfpd is not None else None
        step = piece or n_tok
        for t0 in range(0, n_tok, step):
            tb.tb_accumulate_hessian(H, Xd[t0:t0 + step])
            if R is not None:
                tb.tb_accumulate_cross(R, Xd[t0:t0 + step], Xfpd[t0:t0 + step], desc.alpha)
        Hsum = torch.empty_like(H)
        tb.tb_finalize_hessian(H, R, n_tok, desc.damp, Hsum_out=Hsum)
        U, info = tb.tb_factor(H)
        assert int(info.max().item()) == 0
        P = C = None
        if R is not None:
            P, C = tb.tb_prepare_correction(R, U)
        return H, Hsum, U, R, P, C

    H, Hsum, U, R, P, C = input_side(X, Xfp, d)
    Ho, _, Uo, Ro, Po, Co = input_side(Xo, Xofp, hq * dh)
    if Xv is not None:
        Hv = torch.stack([input_side(Xv[h], None, d)[0] for h in range(hkv)])
        Uv, info = tb.tb_factor(Hv)
        assert int(info.max().item()) == 0
        v_side = (Hv, Uv, None, None, None)
    else:
        v_side = (H, U, R, P, C)
    hout = [tb.tb_build_hout(W[1], Hsum, hq, dh, desc.damp), tb.tb_build_hout(W[0], Hsum, hkv, dh, desc.damp),
            tb.tb_build_hout(W[3].t().contiguous(), None, hkv, dh, desc.damp)]
    uout = [tb.tb_factor(h)[0] for h in hout]
    sides = [(H, U, R, P, C), (H, U, R, P, C), v_side, (Ho, Uo, Ro, Po, Co)]
    res = []
    for i, (d_out, d_in, heads) in enumerate(tb.attention_layer_shapes(desc)):
        ld = tb.layer_desc(d_out, d_in, heads, d_out // heads, desc.bits, desc.quant_group,
                           desc.out_block if i < 3 else d_out, n_hin=hkv if (i == 2 and Xv is not None) else 1,
                           n_cand=desc.n_cand, cd_iters=desc.cd_iters, flags=desc.flags)
        Hi, Ui, Ri, Pi, Ci = sides[i]
        res.append(tb.tb_quantize_layer(ld, W[i], Hi, Ui, hout[i] if i < 3 else None, uout[i] if i < 3 else None,
                                        Ri, Pi, Ci))
    torch.cuda.synchronize()
    return res, dict(H=H, Hsum=Hsum, Ho=Ho, hout=hout)


@pytest.mark.parametrize("with_r,per_head_v,hkv", [(True, True, 2), (False, False, 4), (True, False, 1)])
def test_attention_layer_equals_the_chain_of_single_calls(with_r, per_head_v, hkv):
    """Device-resident and host-resident, side by side and one after the other: every output of
    tb_attention_layer equals the chain of single calls bit for bit.  20000 tokens: with host buffers
    the activations cross in two pieces (16384 + 3616)."""
    import torch
    import paper_2602_04929_b200 as tb
    d, hq, dh, n_tok = 256, 4, 64, 20000
    Wn, Xn, Xfpn, Xvn, Xon, Xofpn = _layer_inputs(41, d, hq, hkv, dh, n_tok, with_r, per_head_v)
    bf = torch.bfloat16
    W = [_dev(w) for w in Wn]
    X, Xo = _dev(Xn, bf), _dev(Xon, bf)
    Xfp = None if Xfpn is None else _dev(Xfpn, bf)
    Xofp = None if Xofpn is None else _dev(Xofpn, bf)
    Xv = None if Xvn is None else _dev(Xvn, bf)
    desc = tb.attention_desc(d, hq, hkv, dh, 3, 64, 16, n_tok, flags=ADAPT | CD, concurrent=False)
    ref_dev, _ = _manual_chain(tb, desc, W, X, Xfp, Xv, Xo, Xofp)
    ref_host, _ = _manual_chain(tb, desc, W, X, Xfp, Xv, Xo, Xofp, piece=16384) if with_r else (ref_dev, None)
    n_info = tb.tb_attention_layer_info_count(desc, per_head_v)
    assert n_info == 2 + (hkv if per_head_v else 0) + hq + 2 * hkv

    def check(outs, ref, label):
        for i, (o, r) in enumerate(zip(outs, ref)):
            for k in ("codes", "scales", "zeros", "w_hat", "loss"):
                assert torch.equal(o[k].cpu(), getattr(r, k).cpu()), (label, NAMES[i], k)

    for concurrent in (False, True):
        desc.concurrent = int(concurrent)
        desc.on_host = 0
        outs = tb.attention_outputs(desc, device="cuda:0")
        info = torch.full((n_info,), -1, dtype=torch.int32, device="cuda:0")
        io = tb.attention_io(desc, X, Xo, W, outs, X_fp=Xfp, X_v=Xv, X_o_fp=Xofp, info=info)
        ws = torch.empty(tb.tb_attention_layer_workspace(desc, io), dtype=torch.uint8, device="cuda:0")
        for _ in range(2):   # the second call reuses the helper streams and the workspace
            tb.tb_attention_layer(desc, io, ws)
            torch.cuda.synchronize()
            assert tb.tb_device_error_flag() == 0
            assert info.cpu().tolist() == [0] * n_info
            check(outs, ref_dev, f"device concurrent={concurrent}")
        # the same from host buffers
        desc.on_host = 1
        houts = tb.attention_outputs(desc, device=None, pin=True)
        pin = lambda t: None if t is None else t.cpu().pin_memory()
        hio = tb.attention_io(desc, pin(X), pin(Xo), [pin(w) for w in W], houts, X_fp=pin(Xfp), X_v=pin(Xv),
                              X_o_fp=pin(Xofp))
        hws = torch.empty(tb.tb_attention_layer_workspace(desc, hio), dtype=torch.uint8, device="cuda:0")
        tb.tb_attention_layer(desc, hio, hws)
        check(houts, ref_host, f"host concurrent={concurrent}")


def test_attention_layer_against_the_oracle_chain():
    """Table 1's pairing, checked independently of the library's own single calls: the oracle builds
    every Hessian in float64 from the same activations (H_in of X for W_Q and W_K, of A_h X per head
    for W_V, of X_o for the output projection; H_out of W_Q from W_K through X, of W_K from W_Q summed
    over the query heads of a key/value head, of W_V from the head's columns of W_O) and evaluates the
    loss of the GPU's own W_hat under them; the GPU's reported loss must agree to 1e-4 (the Hessians
    differ by float accumulation, about 1e-6).  A wrong partner, a transposed W_O or a wrong head
    grouping changes H_out altogether and fails this by orders of magnitude.  The oracle also runs its
    own chain; rows whose codes differ are counted and the losses compared as in the single-projection
    chained test."""
    import torch
    import paper_2602_04929_b200 as tb
    d, hq, hkv, dh, n_tok = 256, 4, 2, 64, 6144
    Wn, Xn, _, Xvn, Xon, _ = _layer_inputs(43, d, hq, hkv, dh, n_tok, False, True)
    bf = torch.bfloat16
    desc = tb.attention_desc(d, hq, hkv, dh, 3, 64, 16, n_tok, flags=ADAPT | CD, concurrent=True)
    outs = tb.attention_outputs(desc, device="cuda:0")
    W = [_dev(w) for w in Wn]
    io = tb.attention_io(desc, _dev(Xn, bf), _dev(Xon, bf), W, outs, X_v=_dev(Xvn, bf))
    ws = torch.empty(tb.tb_attention_layer_workspace(desc, io), dtype=torch.uint8, device="cuda:0")
    tb.tb_attention_layer(desc, io, ws)
    torch.cuda.synchronize()
    assert tb.tb_device_error_flag() == 0
    # the oracle's Hessians
    Hin, Hsum = oracle.hessian(Xn, damp=0.01, return_sum=True)
    Hin_v = np.stack([oracle.hessian(Xvn[h], damp=0.01) for h in range(hkv)])
    Hin_o = oracle.hessian(Xon, damp=0.01)
    Hout = [oracle.hout_from_projection(Wn[1], Hsum, hq, dh, damp=0.01),
            oracle.hout_from_projection(Wn[0], Hsum, hkv, dh, damp=0.01),
            oracle.hout_from_projection(np.ascontiguousarray(Wn[3].T), None, hkv, dh, damp=0.01)]
    shapes = tb.attention_layer_shapes(desc)
    report = {}
    for i, (d_out, d_in, heads) in enumerate(shapes):
        w_hat, loss = outs[i]["w_hat"].cpu().numpy(), outs[i]["loss"].cpu().numpy()
        rows_per = d_out // heads
        own = []
        for h in range(heads):
            sl = slice(h * rows_per, (h + 1) * rows_per)
            Hi = Hin_v[h] if i == 2 else (Hin_o if i == 3 else Hin)
            own.append(oracle.loss_head(Wn[i][sl], w_hat[sl], Hi, Hout[i][h] if i < 3 else None))
        rel = float(np.max(np.abs(loss - np.array(own)) / np.array(own)))
        # the oracle's own chain for this projection
        Hi = Hin_v if i == 2 else (Hin_o if i == 3 else Hin)
        Ui = oracle.factor_upper(Hi)
        od = oracle.OracleDesc(d_out, d_in, heads, rows_per, bits=3, quant_group=64, out_block=16 if i < 3 else rows_per,
                               n_hin=hkv if i == 2 else 1, flags=ADAPT | CD)
        ref = oracle.quantize_layer(od, Wn[i], Hi, Ui, Hout[i] if i < 3 else None,
                                    oracle.factor_upper(Hout[i]) if i < 3 else None)
        rows_diff = int(np.count_nonzero((outs[i]["codes"].cpu().numpy() != ref.codes).any(axis=1)))
        rel_chain = float(np.max(np.abs(loss - ref.loss) / ref.loss))
        report[NAMES[i]] = dict(loss_vs_own_w_hat=rel, rows=d_out, rows_with_a_different_code=rows_diff,
                                loss_vs_oracle_chain=rel_chain)
        assert rel <= 1e-4, report
        assert rel_chain <= (1e-4 if rows_diff == 0 else 2e-2), report
        assert rows_diff <= d_out // 4, report
    print("LAYER-CHAIN", report)
