"""Small-problem builders for the oracle pins (numpy only; no method arithmetic
beyond textbook definitions used as independent checks)."""
import numpy as np


def small_problem(seed, dh=8, d=16, n_tok=64, with_r=False, n_heads=1, cond_out=50.0, alpha=0.25):
    """Explicit G, X, dX so that every Hessian has its primary definition:
    H_in = X X^T / n, H_out = G^T G, R = alpha dX X^T / n (paper layout X: d x L)."""
    g = np.random.default_rng(seed)
    X = g.standard_normal((d, n_tok))
    X[: max(1, d // 8)] *= 5.0
    mix = np.eye(d) + 0.3 * g.standard_normal((d, d)) / np.sqrt(d)
    X = mix @ X
    Hin = X @ X.T / n_tok
    Hin += 0.01 * np.mean(np.diag(Hin)) * np.eye(d)
    Xeff = None
    Gs, Houts = [], []
    for _ in range(n_heads):
        G = g.standard_normal((dh + 3, dh))
        G = G @ np.diag(np.logspace(0, -np.log10(cond_out) / 2, dh))
        Gs.append(G)
        Houts.append(G.T @ G)
    W = 0.02 * g.standard_normal((n_heads * dh, d))
    out = dict(X=X, Hin=Hin, G=Gs, Hout=np.stack(Houts), W=W, n_tok=n_tok)
    if with_r:
        dX = 0.1 * g.standard_normal((d, d)) @ X / np.sqrt(d) + 0.05 * g.standard_normal((d, n_tok))
        out["dX"] = dX
        out["R"] = alpha * dX @ X.T / n_tok
        out["alpha"] = alpha
    return out


def explicit_loss(G, dW, X, W=None, dX=None, alpha=1.0, n_tok=1, damp_term=None):
    """||G dW X||_F^2 / n  (+ cross term 2 <G dW X, G W alpha dX> / n).
    damp_term = lambda * tr(H_out dW dW^T) accounts for the damping added to H_in."""
    A = G @ dW @ X
    val = np.sum(A * A) / n_tok
    if dX is not None:
        Bm = G @ W @ (alpha * dX)
        val += 2.0 * np.sum(A * Bm) / n_tok
    if damp_term is not None:
        val += damp_term * np.trace(G.T @ G @ dW @ dW.T)
    return val
