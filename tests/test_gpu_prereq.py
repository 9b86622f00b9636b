"""GPU parity of the prerequisites of the quantizer against the float64 oracle:
Hessian accumulation and finalisation, H_out construction, the inverse Cholesky
factor and the propagated-error operands.  All calls go through the C ABI."""
import numpy as np
import pytest

import oracle
import tb_inputs
from parity_util import cached_problem, f32, rel_fro

pytestmark = pytest.mark.gpu


def _t(a, dtype=None):
    import torch
    t = torch.from_numpy(np.ascontiguousarray(a)).to("cuda:0")
    return t if dtype is None else t.to(dtype)


@pytest.mark.parametrize("n_tok,d,bf16", [(5000, 264, True), (4096, 256, False), (9000, 384, True),
                                          (70000, 512, True), (64, 128, True), (3, 8, True),
                                          (6000, 6152, True), (4200, 8192, True)])
def test_hessian_accumulation(n_tok, d, bf16):
    """H = X^T X / n + damping (Table 1) over several launches with a ragged last
    chunk and a width that is not a multiple of the tile; from 6144 columns on the
    kernel that shares a tile between two CTAs runs.  Tolerance: products of
    bf16 inputs are exact in float; each 4096-token launch adds ~sqrt(4096) * 2^-24
    relative rounding and the running sum one more rounding per launch, far below 1e-5."""
    import torch
    import paper_2602_04929_b200 as tb
    rec = tb_inputs.HeavyTailRecipe(d, seed=3)
    X = rec.chunk(0, n_tok, bf16=bf16)
    H = torch.zeros((d, d), dtype=torch.float32, device="cuda:0")
    Xd = _t(X, torch.bfloat16 if bf16 else None)
    half = (n_tok // 2 // 8) * 8
    tb.tb_accumulate_hessian(H, Xd[:half].contiguous())      # running sum over two calls
    tb.tb_accumulate_hessian(H, Xd[half:].contiguous())
    Hsum = torch.empty_like(H)
    tb.tb_finalize_hessian(H, None, n_tok, 0.01, Hsum_out=Hsum)
    torch.cuda.synchronize()
    assert tb.tb_device_error_flag() == 0      # no bounded wait of the tensor-core kernel ran out
    Ho, Hso = oracle.hessian(X, damp=0.01, return_sum=True)
    Hg = H.cpu().numpy()
    assert rel_fro(Hg, Ho) <= 1e-5
    assert rel_fro(Hsum.cpu().numpy(), Hso) <= 1e-5
    assert np.array_equal(Hg, Hg.T)
    scale = np.sqrt(np.outer(np.diag(Ho), np.diag(Ho)))
    assert np.max(np.abs(Hg - Ho) / scale) <= 1e-5


@pytest.mark.parametrize("bf16,d,chunks", [(True, 264, (6000,)), (False, 264, (6000,)), (True, 512, (5000, 64, 3001)),
                                            (True, 128, (7,))])
def test_cross_correlation(bf16, d, chunks):
    """R = alpha (X - Xfp) X^T / n (Algorithm 1, deviation step), not symmetric; several launches with
    ragged token counts and a width that is not a multiple of the tile.  bf16: the deviation is
    split into two bf16 pieces (exact here), every product is exact in float and the float
    accumulation is cut into runs of 2048 steps, so the error stays far below 1e-5."""
    import torch
    import paper_2602_04929_b200 as tb
    n_tok, alpha = sum(chunks), 0.25
    rec = tb_inputs.DeviationRecipe(tb_inputs.HeavyTailRecipe(d, seed=5))
    X, Xfp = rec.chunk(0, n_tok, bf16=bf16)
    if bf16:
        Xfp = tb_inputs.bf16_bits_to_f32(tb_inputs.to_bf16_bits(Xfp))
    dt = torch.bfloat16 if bf16 else None
    R = torch.zeros((d, d), dtype=torch.float32, device="cuda:0")
    H = torch.zeros((d, d), dtype=torch.float32, device="cuda:0")
    t0 = 0
    for n in chunks:
        tb.tb_accumulate_cross(R, _t(X[t0:t0 + n], dt), _t(Xfp[t0:t0 + n], dt), alpha)
        tb.tb_accumulate_hessian(H, _t(X[t0:t0 + n], dt))
        t0 += n
    tb.tb_finalize_hessian(H, R, n_tok, 0.0)
    torch.cuda.synchronize()
    assert tb.tb_device_error_flag() == 0
    Ro = oracle.cross_correlation(X, Xfp, alpha)
    err = rel_fro(R.cpu().numpy(), Ro)
    print("CROSS rel error", err)
    assert err <= 1e-5


@pytest.mark.parametrize("n_heads,g_heads,with_sum", [(4, 4, True), (2, 8, True), (8, 2, True), (4, 4, False)])
def test_build_hout(n_heads, g_heads, with_sum):
    """Table 1: H_out,h = G_h Hsum G_h^T (query / key side, also grouped-query
    attention in both directions) or G_h G_h^T (value side)."""
    import torch
    import paper_2602_04929_b200 as tb
    d, dh = 256, 64
    X = tb_inputs.HeavyTailRecipe(d, seed=7).chunk(0, 2048)
    _, Hs = oracle.hessian(X, return_sum=True)
    Hs32 = f32(Hs)
    G = tb_inputs.weight(7, g_heads * dh, d, tid=tb_inputs.T_WPARTNER)
    Hout = tb.tb_build_hout(_t(G), _t(Hs32) if with_sum else None, n_heads, dh, 0.01)
    torch.cuda.synchronize()
    ref = oracle.hout_from_projection(G, Hs32 if with_sum else None, n_heads, dh, damp=0.01)
    # G Hsum runs on the tensor cores from exact bf16 splits: the six retained piece products drop
    # terms below 2^-24 and each 128-step chunk is accumulated in float before the double sum
    err = rel_fro(Hout.cpu().numpy(), ref)
    print("HOUT rel error", err)
    assert err <= 2e-6


@pytest.mark.parametrize("n_batch,d,cond", [(3, 200, 1e3), (1, 256, 1e5), (2, 64, 1e2), (1, 520, 1e4), (5, 128, 1e3),
                                            (2, 1024, 1e3), (1, 1100, 1e4), (1, 2100, 1e4), (1, 4096, 1e4)])
def test_factor_matches_definition(n_batch, d, cond):
    """U = chol(H^-1)^T (Eq. 2).  The GPU takes the reversed-Cholesky route in
    double and rounds once to float; the oracle inverts and factors.  From 1024 columns on
    the panels, the trailing updates and the inverse of the finished blocks run on streams
    of their own: two matrices at once, a size whose last blocks are partly and wholly
    padding (1100 in 2048), one that reaches the level whose first product is launched
    in pieces (2100 in 4096), and the benchmark's own size."""
    import torch
    import paper_2602_04929_b200 as tb
    H = np.stack([tb_inputs.spd_matrix(11 + b, d, cond=cond) for b in range(n_batch)])
    U, info, Hinv = tb.tb_factor(_t(H), want_inverse=True)
    torch.cuda.synchronize()
    assert info.cpu().tolist() == [0] * n_batch
    Ug, Uo = U.cpu().numpy().astype(np.float64), oracle.factor_upper(H)
    assert np.all(np.tril(Ug, -1) == 0.0)
    assert np.all(np.diagonal(Ug, axis1=1, axis2=2) > 0)
    for b in range(n_batch):
        assert rel_fro(Ug[b], Uo[b]) <= 1e-6
        I = Ug[b] @ H[b].astype(np.float64) @ Ug[b].T
        assert np.max(np.abs(I - np.eye(d))) <= 1e-6 * cond ** 0.5 + 1e-5
        assert rel_fro(Hinv.cpu().numpy()[b], np.linalg.inv(H[b].astype(np.float64))) <= 1e-5


def test_factor_at_the_width_of_the_headline_benchmark():
    """U = chol(H^-1)^T (Eq. 2) at 8192 columns, the width of the headline benchmark's ten input Hessians:
    H is the damped Hessian of 16 384 seeded heavy-tailed tokens (built by the library), the oracle inverts
    and factors it in float64.  The same matrix twice in one batched call (the form the benchmark uses for
    the value projection's per-head Hessians) must give the single call's factor bit for bit."""
    import torch
    import paper_2602_04929_b200 as tb
    d, n_tok = 8192, 16384
    X = tb_inputs.heavy_tail_device(tb_inputs.HeavyTailRecipe(d, seed=7), n_tok, "cuda:0", seed=2)
    H = torch.zeros((d, d), dtype=torch.float32, device="cuda:0")
    tb.tb_accumulate_hessian(H, X)
    tb.tb_finalize_hessian(H, None, n_tok, 0.01)
    del X
    U1, info1 = tb.tb_factor(H)
    U2, info2 = tb.tb_factor(torch.stack([H, H]))
    torch.cuda.synchronize()
    assert tb.tb_device_error_flag() == 0
    assert int(info1.max()) == 0 and int(info2.max()) == 0
    assert torch.equal(U2[0], U1.reshape(d, d)) and torch.equal(U2[1], U1.reshape(d, d))
    Ug = U1.reshape(d, d).cpu().numpy().astype(np.float64)
    Uo = oracle.factor_upper(H.cpu().numpy()[None])[0]
    assert np.all(np.tril(Ug, -1) == 0.0) and np.all(np.diag(Ug) > 0)
    err = rel_fro(Ug, Uo)
    print("FACTOR 8192 rel error", err)
    assert err <= 1e-6
    del H, U1, U2
    torch.cuda.empty_cache()


def test_factor_reports_a_non_positive_pivot():
    """A matrix that is not positive definite yields a device-side info word, no fault."""
    import torch
    import paper_2602_04929_b200 as tb
    H = np.stack([tb_inputs.spd_matrix(1, 96), -np.eye(96, dtype=np.float32), tb_inputs.spd_matrix(2, 96)])
    H[2, 95, 95] = -1.0   # last row is eliminated first
    U, info = tb.tb_factor(_t(H))
    torch.cuda.synchronize()
    info = info.cpu().tolist()
    assert info[0] == 0 and info[1] == 1 and info[2] == 1


def test_factor_is_independent_of_other_work_on_the_gpu():
    """The factor must not depend on how many of a launch's blocks run at the same time.
    A second stream keeps every SM busy with unrelated work while the factor is queued
    several times without a host synchronisation in between; every result must equal,
    bit for bit, the one computed on an idle GPU."""
    import torch
    import paper_2602_04929_b200 as tb
    d = 2048
    g = torch.Generator(device="cuda:0").manual_seed(5)
    X = torch.randn(2 * d, d, device="cuda:0", generator=g)
    H = (X.T @ X / (2 * d) + 0.01 * torch.eye(d, device="cuda:0")).contiguous()
    U0, info0 = tb.tb_factor(H)
    torch.cuda.synchronize()
    assert int(info0.max()) == 0
    side = torch.cuda.Stream(device="cuda:0")
    filler = torch.empty(32 << 20, device="cuda:0")
    results = []
    for _ in range(4):
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            for _ in range(12):
                filler.normal_()
        results.append(tb.tb_factor(H))
        torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    for U, info in results:
        assert int(info.max()) == 0
        assert torch.equal(U, U0)


@pytest.mark.parametrize("n_batch,d", [(1, 256), (2, 200)])
def test_prepare_correction(n_batch, d):
    """P = ((R U^T) masked strictly upper) U (Algorithm 2, its masked operand); C = R U^T U (Proposition 3.2)."""
    import torch
    import paper_2602_04929_b200 as tb
    Rs, Us = [], []
    for b in range(n_batch):
        rec = tb_inputs.DeviationRecipe(tb_inputs.HeavyTailRecipe(d, seed=20 + b))
        X, Xfp = rec.chunk(0, 2048)
        H32 = f32(oracle.hessian(X, damp=0.01))
        Us.append(f32(oracle.factor_upper(H32)))
        Rs.append(f32(oracle.cross_correlation(X, Xfp, 0.25)))
    R, U = np.stack(Rs), np.stack(Us)
    P, C = tb.tb_prepare_correction(_t(R), _t(U))
    torch.cuda.synchronize()
    Po, Co = oracle.correction_operands(R, U)
    Pg = P.cpu().numpy()
    assert np.all(np.tril(Pg) == 0.0)
    assert rel_fro(Pg, Po) <= 1e-5
    assert rel_fro(C.cpu().numpy(), Co) <= 1e-5


def test_prerequisites_at_full_width():
    """Every prerequisite at the benchmark's width (4096 columns, 32 heads of 128 rows), in the launch
    shapes that size produces, against the oracle's float64 results for the same 8192 seeded tokens:
    Hessian and its undamped sum, deviation correlation R, the factor of H_in (helper streams, all
    doubling levels), the correction operands P and C on the tensor-core path, H_out from the partner
    projection and its 32 small factors.  Each call gets the oracle's (float32-rounded) inputs, so the
    stages are compared one by one."""
    import torch
    import paper_2602_04929_b200 as tb
    d, H, dh, n_tok, alpha, damp = 4096, 32, 128, 8192, 0.25, 0.01
    prob = cached_problem(0, d, H, dh, n_tok, with_r=True)
    X, Xfp = tb_inputs.DeviationRecipe(tb_inputs.HeavyTailRecipe(d, seed=0)).chunk(0, n_tok)
    Xd, Xfd = _t(X, torch.bfloat16), _t(Xfp, torch.bfloat16)
    Hg = torch.zeros((d, d), dtype=torch.float32, device="cuda:0")
    Rg = torch.zeros((d, d), dtype=torch.float32, device="cuda:0")
    Hsum = torch.empty_like(Hg)
    for t0, t1 in ((0, 6144), (6144, n_tok)):     # two launches, the second shorter
        tb.tb_accumulate_hessian(Hg, Xd[t0:t1].contiguous())
        tb.tb_accumulate_cross(Rg, Xd[t0:t1].contiguous(), Xfd[t0:t1].contiguous(), alpha)
    tb.tb_finalize_hessian(Hg, Rg, n_tok, damp, Hsum_out=Hsum)
    torch.cuda.synchronize()
    assert tb.tb_device_error_flag() == 0
    assert rel_fro(Hg.cpu().numpy(), prob["Hin"][0]) <= 1e-5
    assert rel_fro(Hsum.cpu().numpy(), prob["Hsum"]) <= 1e-5
    assert rel_fro(Rg.cpu().numpy(), prob["R"][0]) <= 1e-5
    U, info = tb.tb_factor(_t(prob["Hin"]))
    P, C = tb.tb_prepare_correction(_t(prob["R"]), _t(prob["Uin"]))
    Hout = tb.tb_build_hout(_t(prob["G"]), _t(prob["Hsum"]), H, dh, damp)
    Uout, info_out = tb.tb_factor(_t(prob["Hout"]))
    torch.cuda.synchronize()
    assert tb.tb_device_error_flag() == 0
    assert int(info.max()) == 0 and int(info_out.max()) == 0
    errs = {"U_in": rel_fro(U.cpu().numpy()[0], prob["Uin"][0]), "P": rel_fro(P.cpu().numpy(), prob["P"]),
            "C": rel_fro(C.cpu().numpy(), prob["C"]), "H_out": rel_fro(Hout.cpu().numpy(), prob["Hout"]),
            "U_out": max(rel_fro(Uout.cpu().numpy()[h], prob["Uout"][h]) for h in range(H))}
    print("FULL-WIDTH PREREQUISITES rel errors", errs)
    assert errs["U_in"] <= 1e-6 and errs["U_out"] <= 1e-6
    assert errs["P"] <= 1e-5 and errs["C"] <= 1e-5
    assert errs["H_out"] <= 2e-6


def test_hessian_at_the_benchmark_size_on_sampled_entries():
    """The Hessian of the headline benchmark (262 144 bf16 tokens, 8192 columns: one call, the launch the
    benchmark times, CTA pairs on 256 x 256 tiles) against the oracle on sampled entries: the oracle gets
    the sampled columns of the same seeded activations and returns their block of X^T X / n in float64.
    The columns are chosen around tile edges (127 | 128, 255 | 256), in the first and the last tile and
    across distant tiles, so that every kind of tile (diagonal, below the diagonal, last round) and the
    mirrored half are hit.  Tolerance as in the small cases: 1e-5 of sqrt(H_ii H_jj) per entry."""
    import torch
    import paper_2602_04929_b200 as tb
    d, n_tok = 8192, 262144
    rec = tb_inputs.HeavyTailRecipe(d, seed=5)
    X = tb_inputs.heavy_tail_device(rec, n_tok, "cuda:0", seed=1)
    H = torch.zeros((d, d), dtype=torch.float32, device="cuda:0")
    Hsum = torch.empty_like(H)
    tb.tb_accumulate_hessian(H, X)
    tb.tb_finalize_hessian(H, None, n_tok, 0.0, Hsum_out=Hsum)
    torch.cuda.synchronize()
    assert tb.tb_device_error_flag() == 0
    cols = sorted({0, 1, 63, 64, 127, 128, 129, 255, 256, 257, 511, 512, 1000, 2047, 2048, 3071, 4095, 4096, 4097,
                   5000, 6143, 6144, 7000, 7935, 7936, 8063, 8064, 8190, 8191})
    idx = torch.tensor(cols, device="cuda:0")
    Xs = X[:, idx].float().cpu().numpy()                 # bf16 values are exact in float
    Ho = oracle.hessian(Xs, damp=0.0)                    # [len(cols)]^2 block of X^T X / n in float64
    Hg = Hsum[idx][:, idx].cpu().numpy().astype(np.float64)
    scale = np.sqrt(np.outer(np.diag(Ho), np.diag(Ho)))
    err = np.max(np.abs(Hg - Ho) / scale)
    print("FULL-SIZE HESSIAN sampled entries:", len(cols) ** 2, "max scaled error", err)
    assert err <= 1e-5
    assert np.array_equal(Hg, Hg.T)                      # the mirrored half is a copy
    del X, H, Hsum
    torch.cuda.empty_cache()


def test_bounded_wait_gives_up_and_leaves_the_context_usable():
    """A wait on a hardware barrier at which nothing ever arrives, with a budget of about 1 ms: the
    kernel must return by itself, the device error word must be raised (and cleared by reading it),
    and the next real call must be clean."""
    import torch
    import paper_2602_04929_b200 as tb
    assert tb.tb_device_error_flag() == 0
    gave_up = torch.zeros(1, dtype=torch.int32, device="cuda:0")
    tb.tb_selftest_bounded_wait(2_000_000, gave_up)
    torch.cuda.synchronize()
    assert int(gave_up.item()) == 1
    assert tb.tb_device_error_flag() == 1
    assert tb.tb_device_error_flag() == 0          # reading it cleared it
    # the context is intact: a tensor-core Hessian right after it, against the oracle
    X = tb_inputs.HeavyTailRecipe(128, seed=9).chunk(0, 4096)
    H = torch.zeros((128, 128), dtype=torch.float32, device="cuda:0")
    tb.tb_accumulate_hessian(H, _t(X, torch.bfloat16))
    tb.tb_finalize_hessian(H, None, 4096, 0.01)
    torch.cuda.synchronize()
    assert tb.tb_device_error_flag() == 0
    assert rel_fro(H.cpu().numpy(), oracle.hessian(X, damp=0.01)) <= 1e-5
