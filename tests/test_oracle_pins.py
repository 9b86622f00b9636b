"""Pins of the float64 oracle against what the paper and the mathematics fix.

Each test checks the oracle against something other than itself: a primary
definition evaluated another way, a closed form, an invariant of the paper's
proofs, a reduction the paper states, or brute force on tiny inputs.
"""
import itertools

import numpy as np
import pytest

import oracle
from oracle import OracleDesc, F_ADAPTIVE_GRID, F_CD_REFINE
from helpers import small_problem, explicit_loss


def rne(x):
    return np.rint(x)


# --------------------------------------------------------------------------- O0
def test_hessian_is_sum_of_outer_products():
    g = np.random.default_rng(1)
    X = g.standard_normal((37, 6))
    H = oracle.hessian(X, damp=0.0)
    ref = np.zeros((6, 6))
    for t in range(37):
        ref += np.outer(X[t], X[t])
    ref /= 37
    assert np.allclose(H, ref, rtol=1e-13, atol=1e-13)
    Hd = oracle.hessian(X, damp=0.01)
    assert np.allclose(Hd - H, 0.01 * np.trace(ref) / 6 * np.eye(6), atol=1e-14)
    assert np.all(np.linalg.eigvalsh(Hd) > 0)


def test_cross_correlation_layout():
    # R[a, b] = alpha/n sum_t dx_t[a] x_t[b]  (paper: R = alpha dX X^T, X is d x L)
    g = np.random.default_rng(2)
    X, Xfp = g.standard_normal((20, 5)), g.standard_normal((20, 5))
    R = oracle.cross_correlation(X, Xfp, 0.25)
    ref = np.zeros((5, 5))
    for t in range(20):
        for a in range(5):
            for b in range(5):
                ref[a, b] += (X[t, a] - Xfp[t, a]) * X[t, b]
    assert np.allclose(R, 0.25 * ref / 20, atol=1e-14)


def test_hout_from_projection_matches_table1():
    g = np.random.default_rng(3)
    d, dh, L = 12, 4, 50
    X = g.standard_normal((L, d))             # token-major
    Wk = g.standard_normal((2 * dh, d))       # 2 kv heads
    Hs = X.T @ X / L
    # 4 query heads, 2 per kv head: H_out,h = K_k^T K_k with K_k = X Wk_k^T (L x dh)
    Ho = oracle.hout_from_projection(Wk, Hs, n_heads=4, d_head=dh)
    for h in range(4):
        K = X @ Wk[(h // 2) * dh:(h // 2 + 1) * dh].T
        assert np.allclose(Ho[h], K.T @ K / L, atol=1e-12)
    # 1 kv head fed by 2 query-head blocks: the sum of the per-head Grams
    Ho2 = oracle.hout_from_projection(Wk, Hs, n_heads=1, d_head=dh)
    K0, K1 = X @ Wk[:dh].T, X @ Wk[dh:].T
    assert np.allclose(Ho2[0], (K0.T @ K0 + K1.T @ K1) / L, atol=1e-12)
    # value projection: W_out,h^T W_out,h with G = W_out^T and no middle factor
    Wo = g.standard_normal((d, 2 * dh))
    Hv = oracle.hout_from_projection(Wo.T.copy(), None, n_heads=2, d_head=dh)
    assert np.allclose(Hv[1], Wo[:, dh:].T @ Wo[:, dh:], atol=1e-12)


# --------------------------------------------------------------------------- O1
def test_factor_upper_definition_and_second_route():
    g = np.random.default_rng(4)
    A = g.standard_normal((9, 30))
    H = A @ A.T / 30 + 0.05 * np.eye(9)
    U = oracle.factor_upper(H)
    assert np.allclose(U, np.triu(U)) and np.all(np.diag(U) > 0)
    assert np.linalg.norm(U.T @ U @ H - np.eye(9)) < 1e-10
    # second route: H = M M^T with M upper (Cholesky of the index-reversed matrix), U = M^{-1}
    J = np.eye(9)[::-1]
    L = np.linalg.cholesky(J @ H @ J)
    M = J @ L @ J
    assert np.allclose(M, np.triu(M))
    assert np.allclose(U, np.linalg.inv(M), rtol=1e-9, atol=1e-11)
    # trailing-block identity that keeps the update rules valid at every step
    for i in (1, 4, 7):
        assert np.allclose(U[i:, i:].T @ U[i:, i:], np.linalg.inv(H[i:, i:]), rtol=1e-8, atol=1e-10)


# --------------------------------------------------------------------------- O2
def test_correction_operands_elementwise():
    g = np.random.default_rng(5)
    d = 7
    A = g.standard_normal((d, 25))
    H = A @ A.T / 25 + 0.1 * np.eye(d)
    U = oracle.factor_upper(H)
    R = g.standard_normal((d, d))
    P, C = oracle.correction_operands(R, U)
    RUt = np.zeros((d, d))
    for a in range(d):
        for m in range(d):
            RUt[a, m] = sum(R[a, k] * U[m, k] for k in range(d))
    Pref = np.zeros((d, d))
    for a in range(d):
        for b in range(d):
            Pref[a, b] = sum(RUt[a, m] * U[m, b] for m in range(d) if m > a)
    assert np.allclose(P, Pref, atol=1e-12)
    assert np.allclose(P, np.triu(P, 1))
    assert np.allclose(C, R @ np.linalg.inv(H), rtol=1e-9, atol=1e-11)
    P0, C0 = oracle.correction_operands(np.zeros((d, d)), U)
    assert not P0.any() and not C0.any()


# --------------------------------------------------------------------------- O3
def py_grid(w, H, bits, n_cand):
    maxq = 2 ** bits - 1
    mn, mx = min(w.min(), 0.0), max(w.max(), 0.0)
    out = []
    for k in range(n_cand):
        p = 1 - k / 32
        lo, hi = p * mn, p * mx
        if hi == lo:
            s, z = 1.0, 0.0
        else:
            s = (hi - lo) / maxq
            z = min(max(rne(-lo / s), 0), maxq)
        c = np.clip(rne(w / s + z), 0, maxq)
        e = w - s * (c - z)
        out.append((float(e @ H @ e), s, int(z)))
    return out


@pytest.mark.parametrize("gq,bits", [(0, 4), (8, 2), (8, 3)])
def test_grid_search_exhaustive(gq, bits):
    pr = small_problem(10, dh=6, d=16)
    W, Hin = pr["W"], pr["Hin"]
    s, z, cand, scores = oracle.grid_rows(W, Hin, gq, bits, n_cand=16, with_scores=True)
    seg = gq or 16
    for r in range(W.shape[0]):
        for gi in range(16 // seg):
            sl = slice(gi * seg, (gi + 1) * seg)
            ref = py_grid(W[r, sl], Hin[sl, sl], bits, 16)
            J = np.array([t[0] for t in ref])
            assert np.allclose(scores[r, gi], J, rtol=1e-10, atol=1e-18)
            k = int(np.argmin(J))  # first minimum = lowest k
            assert cand[r, gi] == k
            assert scores[r, gi, k] <= scores[r, gi, 0]
            assert np.isclose(s[r, gi], ref[k][1], rtol=1e-14) and z[r, gi] == ref[k][2]


def test_grid_candidate_zero_is_minmax_and_on_grid_input_is_free():
    g = np.random.default_rng(11)
    bits, d = 3, 16
    s0 = 0.013
    # rows exactly on an asymmetric min-max grid whose extremes are both hit
    codes = g.integers(0, 8, size=(5, d))
    codes[:, 0], codes[:, 1] = 0, 7
    W = s0 * (codes - 3.0)
    H = np.eye(d) + 0.1
    s, z, cand, scores = oracle.grid_rows(W, H, 0, bits, with_scores=True)
    assert np.all(cand == 0) and np.all(z == 3)
    assert np.allclose(s, s0, rtol=1e-12) and np.all(np.abs(scores[:, :, 0]) < 1e-28)
    # all-zero segment: s = 1, z = 0
    s, z, cand = oracle.grid_rows(np.zeros((1, d)), H, 0, bits)
    assert s[0, 0] == 1.0 and z[0, 0] == 0 and cand[0, 0] == 0


# --------------------------------------------------------------------------- O4
def fixed_grid(W, bits):
    """plain per-row min-max grid (used only to hand a grid to the sweep)."""
    maxq = 2 ** bits - 1
    mn, mx = np.minimum(W.min(1), 0), np.maximum(W.max(1), 0)
    s = (mx - mn) / maxq
    z = np.clip(rne(-mn / s), 0, maxq).astype(np.int32)
    return s[:, None], z[:, None]


def test_sweep_gptq_identity_and_row_loss():
    pr = small_problem(20, dh=5, d=24)
    W, Hin = pr["W"], pr["Hin"]
    U = oracle.factor_upper(Hin)
    s, z = fixed_grid(W, 3)
    codes, Q, err, _ = oracle.sweep_rows(W, U, s, z, 0, 3)
    # W0 - Q = Err U  and  e H e^T = ||Err||^2  (U H U^T = I)
    assert np.allclose(W - Q, err @ U, atol=1e-13)
    e = W - Q
    assert np.allclose(np.einsum("ra,ab,rb->r", e, Hin, e), np.sum(err ** 2, 1), rtol=1e-9)
    assert np.allclose(Q, s * (codes - z), atol=1e-15)
    assert codes.max() <= 7


def test_sweep_equals_textbook_obs_without_cholesky():
    """Eq. 2 through the Cholesky factor must equal the classical OBS route:
    dw = -(w_j - q_j)/[H^-1]_jj H^-1[j,:], then eliminate j from H^-1."""
    pr = small_problem(21, dh=4, d=12)
    W, Hin = pr["W"], pr["Hin"]
    bits = 2
    s, z = fixed_grid(W, bits)
    codes, Q, _, _ = oracle.sweep_rows(W, oracle.factor_upper(Hin), s, z, 0, bits)
    for r in range(W.shape[0]):
        w = W[r].copy()
        Hinv = np.linalg.inv(Hin)
        for j in range(12):
            q = np.clip(rne(w[j] / s[r, 0] + z[r, 0]), 0, 3)
            qv = s[r, 0] * (q - z[r, 0])
            assert q == codes[r, j]
            w = w - (w[j] - qv) / Hinv[j, j] * Hinv[j]
            w[j] = qv
            Hinv = Hinv - np.outer(Hinv[:, j], Hinv[j]) / Hinv[j, j]
        assert np.allclose(w, Q[r], atol=1e-12)


def test_sweep_fixed_point():
    g = np.random.default_rng(22)
    d, bits = 16, 4
    codes0 = g.integers(0, 16, size=(3, d)).astype(np.uint8)
    s = np.full((3, 1), 0.01)
    z = np.full((3, 1), 7, np.int32)
    W = s * (codes0 - z)
    pr = small_problem(22, dh=3, d=d)
    codes, Q, err, _ = oracle.sweep_rows(W, oracle.factor_upper(pr["Hin"]), s, z, 0, bits)
    assert np.array_equal(codes, codes0) and np.allclose(Q, W, atol=1e-17) and np.abs(err).max() < 1e-14


def test_sweep_with_P_cumulative_stationarity():
    """Algorithm 2 with the P term solves, at column j, min ||dw X + w_j dX_j||^2
    with the first j+1 entries fixed.  Accumulated over columns: for k > j,
    [dw_cum H + (a * 1_{<=j}) R]_k = 0, a = values on arrival."""
    pr = small_problem(23, dh=1, d=10, with_r=True)
    Hin, R = pr["Hin"], pr["R"]
    U = oracle.factor_upper(Hin)
    P, _ = oracle.correction_operands(R, U)
    w0 = pr["W"][0]
    s, z = fixed_grid(w0[None], 2)
    codes, Q, err, _ = oracle.sweep_rows(w0[None], U, s, z, 0, 2, P=P)
    # replay with the oracle's own decisions to obtain the intermediate rows
    w = w0.copy()
    arrival = np.zeros(10)
    for j in range(10):
        arrival[j] = w[j]
        e = (w[j] - Q[0, j]) / U[j, j]
        assert np.isclose(e, err[0, j], rtol=1e-12, atol=1e-15)
        w[j + 1:] -= e * U[j, j + 1:] + w[j] * P[j, j + 1:]
        w[j] = Q[0, j]
        dw = w - w0
        a = np.where(np.arange(10) <= j, arrival, 0.0)
        grad = dw @ Hin + a @ R
        scale = np.linalg.norm(Hin) * np.linalg.norm(w0)
        if j < 9:
            assert np.abs(grad[j + 1:]).max() <= 1e-10 * scale
    assert np.array_equal(np.clip(rne(arrival / s[0, 0] + z[0, 0]), 0, 3), codes[0])


def test_sweep_group_boundaries_use_their_own_grid():
    pr = small_problem(24, dh=2, d=16)
    W, Hin = pr["W"], pr["Hin"]
    s = np.array([[0.01, 0.02], [0.015, 0.005]])
    z = np.array([[1, 2], [0, 3]], np.int32)
    codes, Q, _, _ = oracle.sweep_rows(W, oracle.factor_upper(Hin), s, z, 8, 2)
    for r in range(2):
        for j in range(16):
            assert np.isclose(Q[r, j], s[r, j // 8] * (codes[r, j] - z[r, j // 8]), atol=1e-16)


# --------------------------------------------------------------------------- O5
def test_comp_matrix_equals_hessian_inverse_form():
    pr = small_problem(30, dh=9, d=4)
    Ho = pr["Hout"][0]
    Uo = oracle.factor_upper(Ho)
    Hinv = np.linalg.inv(Ho)
    for i0, nb in [(0, 3), (2, 4), (5, 1), (0, 1)]:
        T = oracle.comp_matrix(Uo, i0, nb)
        # the trailing problem has rows < i0 frozen: use the inverse of the trailing block
        Hi = np.linalg.inv(Ho[i0:, i0:])
        ref = Hi[nb:, :nb] @ np.linalg.inv(Hi[:nb, :nb])
        assert np.allclose(T, ref, rtol=1e-9, atol=1e-11)
        if i0 == 0:
            ref0 = Hinv[nb:, :nb] @ np.linalg.inv(Hinv[:nb, :nb])
            assert np.allclose(T, ref0, rtol=1e-9, atol=1e-11)


@pytest.mark.parametrize("with_r", [False, True])
@pytest.mark.parametrize("g", [1, 2, 4])
def test_stationarity_after_every_step(g, with_r):
    """After each step the gradient of the attention loss w.r.t. the rows not
    yet quantized vanishes: [H_out (dW_cum H_in + S R)]_{rem,:} = 0, S holding
    the snapshots W0 of the rows already processed."""
    dh, d = 8, 12
    pr = small_problem(31 + g, dh=dh, d=d, with_r=with_r)
    W, Hin, Ho = pr["W"], pr["Hin"], pr["Hout"][0]
    Uin, Uo = oracle.factor_upper(Hin), oracle.factor_upper(Ho)
    R = pr.get("R")
    P, C = oracle.correction_operands(R, Uin) if with_r else (None, None)
    desc = OracleDesc(dh, d, 1, dh, bits=2, quant_group=4, out_block=g, flags=F_ADAPTIVE_GRID)
    out = oracle.group_loop_trace(desc, W, Hin, Uin, Uo, P, C)
    S = np.zeros_like(W)
    for step in range(dh // g):
        rows = slice(step * g, (step + 1) * g)
        S[rows] = out["w_comp"][rows]
        Wt = out["trace"][step]
        assert np.allclose(Wt[: (step + 1) * g], out["Q"][: (step + 1) * g], atol=0)
        dW = Wt - W
        inner = dW @ Hin + (S @ R if with_r else 0.0)
        grad = (Ho @ inner)[(step + 1) * g:]
        scale = np.linalg.norm(Ho) * np.linalg.norm(Hin) * max(np.linalg.norm(dW), 1e-30)
        if grad.size:
            assert np.abs(grad).max() <= 1e-10 * scale


def test_g1_is_boa_sequential_rule():
    """N = 1: the update of the remaining rows is Eq. 2 applied on the out side."""
    dh, d = 6, 8
    pr = small_problem(40, dh=dh, d=d)
    W, Hin, Ho = pr["W"], pr["Hin"], pr["Hout"][0]
    Uin, Uo = oracle.factor_upper(Hin), oracle.factor_upper(Ho)
    desc = OracleDesc(dh, d, 1, dh, bits=3, quant_group=0, out_block=1, flags=F_ADAPTIVE_GRID)
    out = oracle.group_loop_trace(desc, W, Hin, Uin, Uo)
    Wt = W.copy()
    for i in range(dh):
        assert np.allclose(Wt[i], out["w_comp"][i], atol=1e-14)
        q = out["Q"][i]
        err = Wt[i] - q
        Wt[i + 1:] -= np.outer(Uo[i, i + 1:] / Uo[i, i], err)
        Wt[i] = q
        assert np.allclose(Wt, out["trace"][i], atol=1e-13)


def test_block_update_is_composition_of_rank1_eliminations():
    dh, d, nb = 7, 5, 3
    pr = small_problem(41, dh=dh, d=d)
    Uo = oracle.factor_upper(pr["Hout"][0])
    g = np.random.default_rng(41)
    W0 = g.standard_normal((dh, d))
    QB = W0[:nb] + 0.1 * g.standard_normal((nb, d))
    T = oracle.comp_matrix(Uo, 0, nb)
    block = W0[nb:] - T @ (W0[:nb] - QB)
    Wt = W0.copy()
    for i in range(nb):  # row i is forced to its preassigned value; later rows (B too) move
        err = Wt[i] - QB[i]
        Wt[i + 1:] -= np.outer(Uo[i, i + 1:] / Uo[i, i], err)
        Wt[i] = QB[i]
    assert np.allclose(Wt[nb:], block, atol=1e-12)


@pytest.mark.parametrize("with_r", [False, True])
def test_compensation_solves_constrained_qp_kkt(with_r):
    """4x4: minimise tr(Ho dW Hin dW^T) + 2 tr(Ho[:,B] W_B R dW^T) s.t. dW_B fixed,
    by dense KKT elimination on the explicit 16x16 Kronecker Hessian."""
    pr = small_problem(42, dh=4, d=4, with_r=with_r)
    W, Hin, Ho = pr["W"], pr["Hin"], pr["Hout"][0]
    R = pr["R"] if with_r else np.zeros((4, 4))
    Uin, Uo = oracle.factor_upper(Hin), oracle.factor_upper(Ho)
    nb = 2
    g = np.random.default_rng(42)
    QB = W[:nb] + 0.01 * g.standard_normal((nb, 4))
    # vec by rows: dW.flatten(); quadratic form v^T (Ho kron Hin) v + 2 c^T v
    K = np.kron(Ho, Hin)
    c = (Ho[:, :nb] @ W[:nb] @ R).flatten()
    fixed = np.arange(nb * 4)
    free = np.arange(nb * 4, 16)
    vfix = (QB - W[:nb]).flatten()
    vfree = np.linalg.solve(K[np.ix_(free, free)], -(K[np.ix_(free, fixed)] @ vfix + c[free]))
    T = oracle.comp_matrix(Uo, 0, nb)
    E = W[:nb] - QB
    if with_r:
        E = E - W[:nb] @ (R @ np.linalg.inv(Hin))
    assert np.allclose((-T @ E).flatten(), vfree, rtol=1e-8, atol=1e-12)


# --------------------------------------------------------------------------- O4(iii), (iv): reductions
def run_layer(pr, bits, gq, g, flags, hout=True, with_r=False, cd_iters=1, n_heads=1, dh=None):
    W, Hin = pr["W"], pr["Hin"]
    dh = dh or W.shape[0] // n_heads
    Uin = oracle.factor_upper(Hin)
    Ho = pr["Hout"] if hout else None
    Uo = oracle.factor_upper(Ho) if hout else None
    R = pr["R"] if with_r else None
    P, C = oracle.correction_operands(R, Uin) if with_r else (None, None)
    desc = OracleDesc(W.shape[0], W.shape[1], n_heads, dh, bits=bits, quant_group=gq, out_block=g,
                      cd_iters=cd_iters, flags=flags)
    return oracle.quantize_layer(desc, W, Hin, Uin, Ho, Uo, R, P, C)


@pytest.mark.parametrize("with_r", [False, True])
def test_identity_hout_reduces_to_rowwise_gptq(with_r):
    pr = small_problem(50, dh=8, d=16, with_r=with_r)
    pr_id = dict(pr, Hout=np.eye(8)[None])
    ref = run_layer(pr, 3, 8, 8, F_ADAPTIVE_GRID, hout=False, with_r=with_r)
    for g in (1, 2, 4, 8):
        out = run_layer(pr_id, 3, 8, g, F_ADAPTIVE_GRID, with_r=with_r)
        assert np.array_equal(out.codes, ref.codes)
        assert np.allclose(out.w_hat, ref.w_hat, atol=1e-15)
        assert np.allclose(out.w_comp, pr["W"], atol=1e-15)  # nothing is ever compensated
    # and the NULL mode is the plain row-wise sweep on a grid from the original rows
    s, z, _ = oracle.grid_rows(pr["W"], pr["Hin"], 8, 3)
    Uin = oracle.factor_upper(pr["Hin"])
    P = oracle.correction_operands(pr["R"], Uin)[0] if with_r else None
    codes, Q, _, _ = oracle.sweep_rows(pr["W"], Uin, s, z, 8, 3, P=P)
    assert np.array_equal(codes, ref.codes) and np.allclose(Q, ref.w_hat, atol=1e-15)


def test_g_equal_dh_is_gptq():
    pr = small_problem(51, dh=8, d=16)
    a = run_layer(pr, 2, 0, 8, F_ADAPTIVE_GRID)            # dense H_out but one group
    b = run_layer(pr, 2, 0, 8, F_ADAPTIVE_GRID, hout=False)
    assert np.array_equal(a.codes, b.codes) and np.allclose(a.w_hat, b.w_hat, atol=1e-15)


def test_static_grid_mode_is_boa_grid():
    """Without the adaptive flag the grid comes once from the original rows."""
    pr = small_problem(52, dh=8, d=16)
    out = run_layer(pr, 3, 0, 2, 0)
    s, z, _ = oracle.grid_rows(pr["W"], pr["Hin"], 0, 3)
    assert np.allclose(out.scales, s, atol=0) and np.array_equal(out.zeros, z)
    ada = run_layer(pr, 3, 0, 2, F_ADAPTIVE_GRID)
    assert not np.allclose(ada.scales[2:], s[2:])          # later rows see compensated weights
    assert np.allclose(ada.scales[:2], s[:2], atol=0)      # the first group does not


# --------------------------------------------------------------------------- loss
@pytest.mark.parametrize("with_r", [False, True])
def test_loss_matches_primary_definition(with_r):
    pr = small_problem(60, dh=5, d=7, with_r=with_r)
    g = np.random.default_rng(60)
    W = pr["W"]
    Q = W + 0.01 * g.standard_normal(W.shape)
    G, X, n = pr["G"][0], pr["X"], pr["n_tok"]
    lam = 0.01 * np.mean(np.diag(X @ X.T / n))
    ref = explicit_loss(G, Q - W, X, W, pr.get("dX"), pr.get("alpha", 1.0), n, damp_term=lam)
    val = oracle.loss_head(W, Q, pr["Hin"], pr["Hout"][0], pr.get("R"))
    assert np.isclose(val, ref, rtol=1e-10)


# --------------------------------------------------------------------------- 4x4 INT2 brute force
def brute_force_min(W, s, z, Hin, Ho, bits, upper=np.inf):
    """Exact minimum of tr(dW Hin dW^T Ho) over all code matrices: depth-first
    enumeration of every code matrix, skipping only branches whose partial sum
    of squares (Cholesky form, all terms non-negative) already exceeds the best
    complete assignment found so far (or `upper`, a known achievable loss)."""
    dh, d = W.shape
    K = np.kron(Ho, Hin)
    Lt = np.linalg.cholesky(K).T          # v^T K v = ||Lt v||^2, Lt upper: row i involves v[i:]
    n = dh * d
    levels = 2 ** bits
    svec = np.repeat(s[:, 0], d)
    zvec = np.repeat(z[:, 0], d)
    wv = W.flatten()
    cand = [[float(svec[i] * (c - zvec[i]) - wv[i]) for c in range(levels)] for i in range(n)]
    rows = [[float(x) for x in Lt[i]] for i in range(n)]
    best = [float(upper) * (1 + 1e-12) if np.isfinite(upper) else np.inf]
    v = [0.0] * n

    def rec(i, acc):
        if i < 0:
            if acc < best[0]:
                best[0] = acc
            return
        ri = rows[i]
        tail = 0.0
        for k in range(i + 1, n):
            tail += ri[k] * v[k]
        lii = ri[i]
        terms = sorted(((lii * c + tail) ** 2, c) for c in cand[i])
        for t, c in terms:
            if acc + t >= best[0]:
                break
            v[i] = c
            rec(i - 1, acc + t)

    rec(n - 1, 0.0)
    return best[0]


def test_bruteforce_search_is_exhaustive_on_2x2():
    g = np.random.default_rng(70)
    for seed in range(5):
        pr = small_problem(70 + seed, dh=2, d=2, n_tok=8)
        W, Hin, Ho = pr["W"], pr["Hin"], pr["Hout"][0]
        s, z = fixed_grid(W, 2)
        bf = brute_force_min(W, s, z, Hin, Ho, 2)
        best = np.inf
        for codes in itertools.product(range(4), repeat=4):
            Q = s * (np.array(codes, float).reshape(2, 2) - z)
            best = min(best, np.trace((Q - W) @ Hin @ (Q - W).T @ Ho))
        assert np.isclose(bf, best, rtol=1e-10)


def _tiny_case(seed):
    pr = small_problem(100 + seed, dh=4, d=4, n_tok=16, cond_out=20.0)
    W, Hin, Ho = pr["W"], pr["Hin"], pr["Hout"][0]
    Uin, Uo = oracle.factor_upper(Hin), oracle.factor_upper(Ho)
    desc = OracleDesc(4, 4, 1, 4, bits=2, quant_group=0, out_block=2, n_cand=1, flags=0)
    out = oracle.quantize_layer(desc, W, Hin, Uin, Ho[None], Uo[None])
    s, z = out.scales, out.zeros
    assert np.allclose(s, fixed_grid(W, 2)[0]) and np.array_equal(z, fixed_grid(W, 2)[1])
    rtn = s * (np.clip(rne(W / s + z), 0, 3) - z)
    l_rtn = np.trace((rtn - W) @ Hin @ (rtn - W).T @ Ho)
    assert np.isclose(out.loss[0], np.trace((out.w_hat - W) @ Hin @ (out.w_hat - W).T @ Ho), rtol=1e-10)
    return W, Hin, Ho, s, z, out, l_rtn


def test_4x4_int2_against_brute_force():
    """The method's loss can never be below the true minimum over all 4^16 code
    matrices (same fixed grids), and that minimum is never above plain rounding."""
    for seed in range(8):
        W, Hin, Ho, s, z, out, l_rtn = _tiny_case(seed)
        bf = brute_force_min(W, s, z, Hin, Ho, 2, upper=min(l_rtn, out.loss[0]))
        assert out.loss[0] >= bf * (1 - 1e-9)
        assert bf <= l_rtn * (1 + 1e-9)


def test_4x4_int2_method_usually_beats_plain_rounding():
    """Greedy, so not a theorem: required on three quarters of 200 seeds."""
    better = sum(_tiny_case(seed)[5].loss[0] <= _tiny_case(seed)[6] * (1 + 1e-12) for seed in range(200))
    assert better >= 150


# --------------------------------------------------------------------------- O6
def literal_cd_step(Wint_bar, W, Q, Hin, Ho, R, j, cols):
    """Proposition 3.3 evaluated literally for out-channel j (restricted to a column group)."""
    Wb = np.zeros_like(Wint_bar)
    Wb[j, cols] = Wint_bar[j, cols]
    Rm = R if R is not None else np.zeros_like(Hin)
    num = (Wb @ (Hin @ (W - Q).T - Rm.T @ W.T) @ Ho)[j, j]
    den = (Wb @ Hin @ Wb.T)[j, j] * Ho[j, j]
    return num / den


@pytest.mark.parametrize("with_r", [False, True])
@pytest.mark.parametrize("gq", [0, 4])
def test_cd_matches_literal_formula_and_is_exact_line_minimiser(gq, with_r):
    dh, d = 5, 8
    pr = small_problem(80, dh=dh, d=d, with_r=with_r)
    W, Hin, Ho, R = pr["W"], pr["Hin"], pr["Hout"][0], pr.get("R")
    g = np.random.default_rng(80)
    seg = gq or d
    ng = d // seg
    codes = g.integers(0, 4, size=(dh, d)).astype(np.uint8)
    zeros = g.integers(0, 4, size=(dh, ng)).astype(np.int32)
    s0 = 0.02 * (1 + 0.2 * g.random((dh, ng)))
    desc = OracleDesc(dh, d, 1, dh, bits=2, quant_group=gq, cd_iters=1)
    s1 = oracle.cd_refine(desc, W, codes, zeros, s0, Hin, Ho, R)
    Wb = codes.astype(float) - np.repeat(zeros, seg, axis=1)
    s = s0.copy()

    def loss_of(sc):
        Q = np.repeat(sc, seg, axis=1) * Wb
        return oracle.loss_head(W, Q, Hin, Ho, R)

    prev = loss_of(s)
    for j in range(dh):
        for gi in range(ng):
            cols = slice(gi * seg, (gi + 1) * seg)
            Q = np.repeat(s, seg, axis=1) * Wb
            if not Wb[j, cols].any():
                continue
            delta = literal_cd_step(Wb, W, Q, Hin, Ho, R, j, cols)
            # exact minimiser of the (quadratic) loss along this coordinate: parabola through 3 points
            def f(t):
                s2 = s.copy(); s2[j, gi] += t
                return loss_of(s2)
            h = 1e-3
            f0, fp, fm = f(0.0), f(h), f(-h)
            t_star = -h * (fp - fm) / (2 * (fp - 2 * f0 + fm))
            assert np.isclose(delta, t_star, rtol=1e-6, atol=1e-12)
            s[j, gi] += delta
            cur = loss_of(s)
            assert cur <= prev + 1e-15
            prev = cur
    assert np.allclose(s1, s, rtol=1e-10, atol=1e-15)


def test_cd_converges_to_direct_solution():
    """One pass is a Gauss-Seidel sweep on A s = b with
    A = (Wbar Hin Wbar^T) o Hout, b = diag[Wbar (Hin - R)^T W^T Hout]."""
    dh, d = 6, 10
    pr = small_problem(81, dh=dh, d=d, with_r=True)
    W, Hin, Ho, R = pr["W"], pr["Hin"], pr["Hout"][0], pr["R"]
    g = np.random.default_rng(81)
    codes = g.integers(0, 8, size=(dh, d)).astype(np.uint8)
    zeros = np.full((dh, 1), 3, np.int32)
    Wb = codes.astype(float) - 3
    A = (Wb @ Hin @ Wb.T) * Ho
    b = np.diag(Wb @ (Hin - R).T @ W.T @ Ho)
    s_direct = np.linalg.solve(A, b)
    s0 = np.full((dh, 1), 0.01)
    # one Gauss-Seidel sweep by hand
    s_gs = s0[:, 0].copy()
    for j in range(dh):
        s_gs[j] = (b[j] - A[j] @ s_gs + A[j, j] * s_gs[j]) / A[j, j]
    desc = OracleDesc(dh, d, 1, dh, bits=3, quant_group=0, cd_iters=1)
    s1 = oracle.cd_refine(desc, W, codes, zeros, s0, Hin, Ho, R)
    assert np.allclose(s1[:, 0], s_gs, rtol=1e-9)
    desc.cd_iters = 3000
    s_inf = oracle.cd_refine(desc, W, codes, zeros, s0, Hin, Ho, R)
    assert np.allclose(s_inf[:, 0], s_direct, rtol=1e-6)


def test_cd_first_iteration_dominates():
    pr = small_problem(82, dh=8, d=16)
    l0 = run_layer(pr, 2, 8, 2, F_ADAPTIVE_GRID).loss[0]
    l1 = run_layer(pr, 2, 8, 2, F_ADAPTIVE_GRID | F_CD_REFINE, cd_iters=1).loss[0]
    l2 = run_layer(pr, 2, 8, 2, F_ADAPTIVE_GRID | F_CD_REFINE, cd_iters=2).loss[0]
    assert l2 <= l1 <= l0
    assert (l0 - l1) >= (l1 - l2)


# --------------------------------------------------------------------------- whole-layer metamorphic
def test_rescaling_hessians_changes_nothing():
    pr = small_problem(90, dh=8, d=16, with_r=True)
    a = run_layer(pr, 3, 8, 4, F_ADAPTIVE_GRID | F_CD_REFINE, with_r=True)
    pr2 = dict(pr, Hin=pr["Hin"] * 4.0, R=pr["R"] * 4.0, Hout=pr["Hout"] * 0.125)
    b = run_layer(pr2, 3, 8, 4, F_ADAPTIVE_GRID | F_CD_REFINE, with_r=True)
    assert np.array_equal(a.codes, b.codes) and np.array_equal(a.zeros, b.zeros)
    assert np.allclose(a.scales, b.scales, rtol=1e-10)
    assert np.isclose(b.loss[0], a.loss[0] * 0.5, rtol=1e-9)


def test_heads_are_independent_and_permutable():
    pr = small_problem(91, dh=4, d=8, n_heads=3)
    full = run_layer(pr, 2, 4, 2, F_ADAPTIVE_GRID | F_CD_REFINE, n_heads=3)
    for h in range(3):
        sub = dict(pr, W=pr["W"][h * 4:(h + 1) * 4], Hout=pr["Hout"][h:h + 1])
        one = run_layer(sub, 2, 4, 2, F_ADAPTIVE_GRID | F_CD_REFINE)
        assert np.array_equal(one.codes, full.codes[h * 4:(h + 1) * 4])
        assert np.allclose(one.scales, full.scales[h * 4:(h + 1) * 4], atol=0)
        assert np.isclose(one.loss[0], full.loss[h], rtol=1e-12)


def test_zero_R_equals_no_R_and_determinism():
    pr = small_problem(92, dh=8, d=16, with_r=True)
    pr0 = dict(pr, R=np.zeros_like(pr["R"]))
    a = run_layer(pr0, 2, 8, 4, F_ADAPTIVE_GRID | F_CD_REFINE, with_r=True)
    b = run_layer(pr, 2, 8, 4, F_ADAPTIVE_GRID | F_CD_REFINE, with_r=False)
    c = run_layer(pr, 2, 8, 4, F_ADAPTIVE_GRID | F_CD_REFINE, with_r=False)
    assert np.array_equal(a.codes, b.codes) and np.allclose(a.scales, b.scales, atol=0)
    assert np.array_equal(b.codes, c.codes) and np.array_equal(b.w_hat, c.w_hat)


def test_propagated_error_term_lowers_the_full_objective():
    """With dX != 0 the R-aware procedure should reach a lower attention loss
    (including the cross term) than ignoring R, on most seeds."""
    wins = 0
    for seed in range(10):
        pr = small_problem(200 + seed, dh=8, d=16, with_r=True, alpha=1.0)
        with_r = run_layer(pr, 3, 0, 4, F_ADAPTIVE_GRID, with_r=True)
        without = run_layer(pr, 3, 0, 4, F_ADAPTIVE_GRID, with_r=False)
        l_without = oracle.loss_head(pr["W"], without.w_hat, pr["Hin"], pr["Hout"][0], pr["R"])
        wins += with_r.loss[0] <= l_without
    assert wins >= 8


# --------------------------------------------------------------------------- guided comparison
def test_hints_are_adopted_only_inside_the_band():
    pr = small_problem(95, dh=4, d=16)
    base = run_layer(pr, 2, 0, 2, F_ADAPTIVE_GRID)
    W, Hin = pr["W"], pr["Hin"]
    Uin, Ho = oracle.factor_upper(Hin), pr["Hout"]
    Uo = oracle.factor_upper(Ho)
    desc = OracleDesc(4, 16, 1, 4, bits=2, quant_group=0, out_block=2, flags=F_ADAPTIVE_GRID)
    wrong = (base.codes + 1) % 4
    out = oracle.quantize_layer(desc, W, Hin, Uin, Ho, Uo, hint_codes=wrong, hint_zeros=base.zeros,
                                hint_cand=base.cand)
    assert np.array_equal(out.codes, base.codes) and out.counters["adopted_codes"] == 0
    # a weight placed exactly on a rounding boundary: both neighbours are acceptable
    s, z = 0.5, 1
    Wt = np.array([[s * (1.5 - z), 1.0, -0.5, 0.25]])
    U = np.eye(4)
    c0, _, _, cnt0 = oracle.sweep_rows(Wt, U, np.array([[s]]), np.array([[z]]), 0, 2)
    assert c0[0, 0] == 2 and cnt0["near_tie_codes"] >= 1          # 1.5 -> 2 (half to even)
    hint = c0.copy(); hint[0, 0] = 1
    c1, _, _, cnt1 = oracle.sweep_rows(Wt, U, np.array([[s]]), np.array([[z]]), 0, 2, hint_codes=hint)
    assert c1[0, 0] == 1 and cnt1["adopted_codes"] == 1


# --------------------------------------------------------------------------- one H_in per head (the W_V row of Table 1)
@pytest.mark.parametrize("with_r", [False, True])
def test_per_head_input_hessians_equal_head_by_head_runs(with_r):
    """n_hin = n_heads: head h must see H_in[h], U_in[h] (and R, P, C [h]) and nothing else.
    Three heads with three different input Hessians, run once as one layer and once head by head
    with a shared-H_in description each."""
    dh, d, H = 4, 8, 3
    prs = [small_problem(300 + h, dh=dh, d=d, with_r=with_r) for h in range(H)]
    W = np.concatenate([p["W"] for p in prs])
    Hin = np.stack([p["Hin"] for p in prs])
    Uin = np.stack([oracle.factor_upper(p["Hin"]) for p in prs])
    Ho = np.stack([p["Hout"][0] for p in prs])
    Uo = oracle.factor_upper(Ho)
    R = P = C = None
    if with_r:
        R = np.stack([p["R"] for p in prs])
        P, C = oracle.correction_operands(R, Uin)
    flags = F_ADAPTIVE_GRID | F_CD_REFINE
    desc = OracleDesc(H * dh, d, H, dh, bits=2, quant_group=4, out_block=2, n_hin=H, flags=flags)
    full = oracle.quantize_layer(desc, W, Hin, Uin, Ho, Uo, R, P, C)
    assert not np.allclose(Hin[0], Hin[1])
    for h in range(H):
        one_desc = OracleDesc(dh, d, 1, dh, bits=2, quant_group=4, out_block=2, n_hin=1, flags=flags)
        sl = slice(h * dh, (h + 1) * dh)
        one = oracle.quantize_layer(one_desc, W[sl], Hin[h], Uin[h], Ho[h:h + 1], Uo[h:h + 1],
                                    None if R is None else R[h], None if P is None else P[h],
                                    None if C is None else C[h])
        assert np.array_equal(one.codes, full.codes[sl]) and np.array_equal(one.zeros, full.zeros[sl])
        assert np.array_equal(one.cand, full.cand[sl])
        assert np.allclose(one.scales, full.scales[sl], atol=0)
        assert np.allclose(one.w_comp, full.w_comp[sl], atol=0)
        assert np.isclose(one.loss[0], full.loss[h], rtol=1e-12)
        # and the per-head loss is the loss under that head's own Hessians
        ref = oracle.loss_head(W[sl], full.w_hat[sl], Hin[h], Ho[h], None if R is None else R[h])
        assert np.isclose(full.loss[h], ref, rtol=1e-12)


# --------------------------------------------------------------------------- H_out = NULL branches of CD and loss
@pytest.mark.parametrize("with_r", [False, True])
@pytest.mark.parametrize("gq", [0, 4])
def test_cd_and_loss_without_hout_equal_identity_hout(gq, with_r):
    """The GPTQ / GPTAQ row of Table 1 (H_out = I): the NULL branches of the scale refinement and of
    the loss against Proposition 3.3 evaluated literally with H_out = I, against the explicit loss
    ||dW X||^2 (+ cross term) with G = I, and against the dense-identity branch."""
    dh, d = 5, 8
    pr = small_problem(83, dh=dh, d=d, with_r=with_r)
    W, Hin, R = pr["W"], pr["Hin"], pr.get("R")
    eye = np.eye(dh)
    g = np.random.default_rng(83)
    seg = gq or d
    ng = d // seg
    codes = g.integers(0, 4, size=(dh, d)).astype(np.uint8)
    zeros = g.integers(0, 4, size=(dh, ng)).astype(np.int32)
    s0 = 0.02 * (1 + 0.2 * g.random((dh, ng)))
    desc = OracleDesc(dh, d, 1, dh, bits=2, quant_group=gq, cd_iters=1)
    s_null = oracle.cd_refine(desc, W, codes, zeros, s0, Hin, None, R)
    s_eye = oracle.cd_refine(desc, W, codes, zeros, s0, Hin, eye, R)
    assert np.allclose(s_null, s_eye, rtol=1e-13, atol=0)
    Wb = codes.astype(float) - np.repeat(zeros, seg, axis=1)
    s = s0.copy()
    for j in range(dh):
        for gi in range(ng):
            cols = slice(gi * seg, (gi + 1) * seg)
            if not Wb[j, cols].any():
                continue
            Q = np.repeat(s, seg, axis=1) * Wb
            s[j, gi] += literal_cd_step(Wb, W, Q, Hin, eye, R, j, cols)
    assert np.allclose(s_null, s, rtol=1e-10, atol=1e-15)
    # rows are independent without H_out: refining one row alone gives that row's scales
    one = OracleDesc(1, d, 1, 1, bits=2, quant_group=gq, cd_iters=1)
    for j in range(dh):
        sj = oracle.cd_refine(one, W[j:j + 1], codes[j:j + 1], zeros[j:j + 1], s0[j:j + 1], Hin, None, R)
        assert np.allclose(sj, s_null[j:j + 1], rtol=1e-12, atol=0)
    # loss
    Q = np.repeat(s_null, seg, axis=1) * Wb
    l_null = oracle.loss_head(W, Q, Hin, None, R)
    assert np.isclose(l_null, oracle.loss_head(W, Q, Hin, eye, R), rtol=1e-13)
    X, n = pr["X"], pr["n_tok"]
    lam = 0.01 * np.mean(np.diag(X @ X.T / n))
    ref = explicit_loss(eye, Q - W, X, W, pr.get("dX"), pr.get("alpha", 1.0), n, damp_term=lam)
    assert np.isclose(l_null, ref, rtol=1e-10)


def test_identity_mode_layer_reports_refined_scales_and_loss():
    """Whole-layer run in the H_out = NULL mode with the scale refinement on: the scales equal
    cd_refine on the pre-refinement scales, and the reported loss is the loss of w_hat."""
    pr = small_problem(84, dh=6, d=16, with_r=True)
    out = run_layer(pr, 3, 8, 6, F_ADAPTIVE_GRID | F_CD_REFINE, hout=False, with_r=True)
    desc = OracleDesc(6, 16, 1, 6, bits=3, quant_group=8, cd_iters=1)
    s1 = oracle.cd_refine(desc, pr["W"], out.codes, out.zeros, out.scales_pre_cd, pr["Hin"], None, pr["R"])
    assert np.allclose(out.scales, s1, atol=0)
    assert not np.allclose(out.scales, out.scales_pre_cd)
    assert np.isclose(out.loss[0], oracle.loss_head(pr["W"], out.w_hat, pr["Hin"], None, pr["R"]), rtol=1e-13)
    pre = np.repeat(out.scales_pre_cd, 8, axis=1) * (out.codes.astype(float) - np.repeat(out.zeros, 8, axis=1))
    assert out.loss[0] <= oracle.loss_head(pr["W"], pre, pr["Hin"], None, pr["R"])


# --------------------------------------------------------------------------- packed integer weights
@pytest.mark.parametrize("bits", [2, 3, 4, 5, 8])
def test_packing_is_the_little_endian_bit_stream(bits):
    """The reference packer against a brute-force bit stream held in one Python integer per row, and
    its round trip; for 3 bits, codes straddle word boundaries."""
    g = np.random.default_rng(700 + bits)
    codes = g.integers(0, 1 << bits, size=(5, 64)).astype(np.uint8)
    packed = oracle.pack_codes(codes, bits)
    assert packed.dtype == np.uint32 and packed.shape == (5, 64 * bits // 32)
    for r in range(5):
        big = 0
        for j, c in enumerate(codes[r].tolist()):
            big |= c << (j * bits)
        words = [(big >> (32 * w)) & 0xFFFFFFFF for w in range(64 * bits // 32)]
        assert packed[r].tolist() == words
    assert np.array_equal(oracle.unpack_codes(packed, bits, 64), codes)
    if bits == 3:   # hand example: codes 0..7 fill 24 bits: 0b111_110_101_100_011_010_001_000
        row = np.array([[0, 1, 2, 3, 4, 5, 6, 7] + [0] * 24], np.uint8)
        assert oracle.pack_codes(row, 3)[0].tolist() == [0b111110101100011010001000, 0, 0]


def test_dequantize_is_s_times_code_minus_zero():
    codes = np.array([[0, 3, 1, 2], [2, 2, 0, 1]], np.uint8)
    s = np.array([[0.5, 2.0], [1.0, 0.25]])
    z = np.array([[1, 2], [0, 1]])
    want = np.array([[-0.5, 1.0, -2.0, 0.0], [2.0, 2.0, -0.25, 0.0]])
    assert np.array_equal(oracle.dequantize(codes, s, z, 2), want)
    assert np.array_equal(oracle.dequantize(codes, s[:, :1], z[:, :1], 0), s[:, :1] * (codes - z[:, :1]))


# --------------------------------------------------------------------------- dynamic per-column-group grid (variant)
from oracle import F_DYNAMIC_GRID  # noqa: E402


def test_dynamic_grid_is_the_grid_search_on_the_arrival_values():
    """Variant of the column-group reading: the (s, z) of a group is searched when the sweep arrives
    at it.  Pinned by reconstruction: the arrival values of group G are W0[:, G] - Err[:, <G] U[<G, G]
    (GPTQ identity), and the grid found in the sweep must be the plain grid search (exhaustively
    re-evaluated in Python above) on exactly those values.  The first group sees the snapshot."""
    pr = small_problem(400, dh=6, d=16)
    W, Hin = pr["W"], pr["Hin"]
    U = oracle.factor_upper(Hin)
    gq, bits = 4, 3
    codes, Q, err, _, s, z = oracle.sweep_rows(W, U, None, None, gq, bits, Hin_dyn=Hin)
    s_static, z_static, _ = oracle.grid_rows(W, Hin, gq, bits)
    assert np.allclose(s[:, 0], s_static[:, 0], atol=0) and np.array_equal(z[:, 0], z_static[:, 0])
    assert not np.allclose(s[:, 1:], s_static[:, 1:])
    for g in range(16 // gq):
        c0 = g * gq
        arrival = W[:, c0:c0 + gq] - err[:, :c0] @ U[:c0, c0:c0 + gq]
        for r in range(6):
            cands = py_grid(arrival[r], Hin[c0:c0 + gq, c0:c0 + gq], bits, 16)
            best = min(range(16), key=lambda k: (cands[k][0], k))     # lowest score, lowest k on ties
            # a runner-up within rounding of the best score may legitimately win: accept either grid
            ok = [k for k in range(16) if cands[k][0] <= cands[best][0] * (1 + 1e-12) + 1e-300]
            assert any(np.isclose(s[r, g], cands[k][1], rtol=1e-12) and z[r, g] == cands[k][2] for k in ok)
    # and the codes are the sweep's codes on those grids: a static sweep handed the same grids agrees
    codes2, Q2, _, _ = oracle.sweep_rows(W, U, s, z, gq, bits)
    assert np.array_equal(codes, codes2) and np.allclose(Q, Q2, atol=0)


def test_dynamic_grid_reductions_still_hold():
    """One group per row: the variant is the adaptive grid.  H_out = I or g = d_head: independent of g
    (row-wise GPTQ).  Weights on a grid whose every group spans the full code range: fixed point."""
    pr = small_problem(401, dh=8, d=16)
    a = run_layer(pr, 3, 0, 2, F_ADAPTIVE_GRID)
    b = run_layer(pr, 3, 0, 2, F_DYNAMIC_GRID)
    assert np.array_equal(a.codes, b.codes) and np.allclose(a.scales, b.scales, atol=0)
    ref = run_layer(pr, 3, 4, 8, F_DYNAMIC_GRID, hout=False)
    pr_id = dict(pr, Hout=np.eye(8)[None])
    for g in (1, 2, 8):
        out = run_layer(pr_id, 3, 4, g, F_DYNAMIC_GRID)
        assert np.array_equal(out.codes, ref.codes) and np.allclose(out.w_hat, ref.w_hat, atol=1e-15)
    assert np.array_equal(run_layer(pr, 3, 4, 8, F_DYNAMIC_GRID).codes, ref.codes)      # g = d_head
    # fixed point: every group of every row holds codes 0 and 3 (the min-max grid is the true grid)
    g = np.random.default_rng(401)
    codes = g.integers(0, 4, size=(8, 16)).astype(np.uint8)
    codes[:, 0::4], codes[:, 1::4] = 0, 3
    s_true = 0.5 ** g.integers(3, 6, size=(8, 4))
    z_true = g.integers(1, 3, size=(8, 4))
    Wg = np.repeat(s_true, 4, axis=1) * (codes - np.repeat(z_true, 4, axis=1))
    out = run_layer(dict(pr, W=Wg), 2, 4, 2, F_DYNAMIC_GRID)
    assert np.array_equal(out.codes, codes) and np.array_equal(out.zeros, z_true)
    assert np.allclose(out.scales, s_true, atol=0) and np.allclose(out.w_comp, Wg, atol=0) and out.loss[0] == 0.0


def test_dynamic_grid_usually_lowers_the_loss():
    wins = 0
    for seed in range(20):
        pr = small_problem(420 + seed, dh=8, d=32)
        dyn = run_layer(pr, 2, 8, 4, F_DYNAMIC_GRID).loss[0]
        ada = run_layer(pr, 2, 8, 4, F_ADAPTIVE_GRID).loss[0]
        wins += dyn <= ada
    assert wins >= 12


# --------------------------------------------------------------------------- why the loop is carried in double
def _sweep_in_float32(W0, U, s, z, maxq):
    """Algorithm 2's column loop with every operation rounded to float32 (rows vectorised, columns in
    order), division and round-half-even as in the oracle.  Returns the codes."""
    w = W0.astype(np.float32).copy()
    U = U.astype(np.float32)
    s = s.astype(np.float32)
    z = z.astype(np.float32)
    m, d = w.shape
    codes = np.zeros((m, d), np.uint8)
    for j in range(d):
        wj = w[:, j].copy()
        x = wj / s[:, j] + z[:, j]
        q = np.clip(np.rint(x), np.float32(0), np.float32(maxq))
        codes[:, j] = q.astype(np.uint8)
        e = (wj - s[:, j] * (q - z[:, j])) / U[j, j]
        w[:, j + 1:] -= e[:, None] * U[j, j + 1:][None, :]
    return codes


def test_float32_chain_changes_codes_where_double_does_not():
    """Measured, not estimated: the same sweep carried in float32 against the oracle's float64 codes, on
    the tiny configuration's shape (256 columns, INT4, one group per row) and on one head (128 rows) of
    the 4096-wide INT2 shape with groups of 128.  Float32 drifts by a few 1e-6 code units over a row and the
    first decision that falls the other way changes every later code of its row; float64 arithmetic in a
    different order (the reciprocal of the scale instead of the division) changes none.  This is why
    the CUDA loop runs in double: the parity bar allows differing codes only within 1e-6 of a tie."""
    import oracle.problems as pu
    report = {}
    for name, (d, rows, n_tok, bits, gq) in {"tiny": (256, 64, 2048, 4, 0), "4096-wide": (4096, 128, 4096, 2, 128)}.items():
        prob = pu.make_problem(0, d, 1, rows, n_tok, hout=None, gaussian_x=(name == "tiny"))
        W, Hin, Uin = prob["W"].astype(np.float64), prob["Hin"][0].astype(np.float64), prob["Uin"][0].astype(np.float64)
        s, z, _ = oracle.grid_rows(W, Hin, gq, bits)
        seg = gq or d
        ref, _, _, cnt = oracle.sweep_rows(W, Uin, s, z, gq, bits)
        c32 = _sweep_in_float32(W, Uin, np.repeat(s, seg, axis=1), np.repeat(z, seg, axis=1), 2 ** bits - 1)
        rows_off = int(np.count_nonzero((c32 != ref).any(axis=1)))
        first = [int(np.argmax(c32[r] != ref[r])) for r in range(rows) if (c32[r] != ref[r]).any()]
        # float64 with the GPU's reformulation (multiply by 1/s): every code must survive
        rs = 1.0 / np.repeat(s, seg, axis=1)
        w = W.copy()
        c64 = np.zeros_like(ref)
        zz = np.repeat(z, seg, axis=1).astype(np.float64)
        ss = np.repeat(s, seg, axis=1)
        for j in range(d):
            wj = w[:, j].copy()
            q = np.clip(np.rint(wj * rs[:, j] + zz[:, j]), 0, 2 ** bits - 1)
            c64[:, j] = q.astype(np.uint8)
            e = (wj - ss[:, j] * (q - zz[:, j])) * (1.0 / Uin[j, j])
            w[:, j + 1:] -= e[:, None] * Uin[j, j + 1:][None, :]
        report[name] = dict(rows=rows, columns=d, codes_off_float32=int(np.count_nonzero(c32 != ref)),
                            rows_off_float32=rows_off, first_flip_column=min(first) if first else None,
                            near_ties_float64=cnt["near_tie_codes"], codes_off_float64_reciprocal=int(np.count_nonzero(c64 != ref)))
        assert np.count_nonzero(c64 != ref) <= cnt["near_tie_codes"]
    print("FLOAT32-CHAIN", report)
    assert report["4096-wide"]["rows_off_float32"] >= 1     # float32 does not reproduce the codes at this width
