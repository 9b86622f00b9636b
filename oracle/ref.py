"""ctypes loader for the C oracle plus the numpy float64 steps around it.

TEST INFRASTRUCTURE.  Nothing here is tuned; nothing here touches CUDA.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass, field

import numpy as np

F_ADAPTIVE_GRID = 1
F_CD_REFINE = 2
F_DYNAMIC_GRID = 4   # variant: a column group's grid is searched when the sweep arrives at it

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "turboboa_oracle.c")
_LIB = os.path.join(_HERE, "libtboracle.so")
_lib = None


def build_oracle(force: bool = False) -> str:
    """Compile the C oracle with gcc (OpenMP over rows only)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


class _Desc(ctypes.Structure):
    _fields_ = [
        ("d_out", ctypes.c_int),
        ("d_in", ctypes.c_int),
        ("n_heads", ctypes.c_int),
        ("d_head", ctypes.c_int),
        ("n_hin", ctypes.c_int),
        ("bits", ctypes.c_int),
        ("quant_group", ctypes.c_int),
        ("out_block", ctypes.c_int),
        ("n_cand", ctypes.c_int),
        ("cd_iters", ctypes.c_int),
        ("flags", ctypes.c_uint),
    ]


class _Counters(ctypes.Structure):
    _fields_ = [
        ("near_tie_codes", ctypes.c_longlong),
        ("adopted_codes", ctypes.c_longlong),
        ("adopted_zeros", ctypes.c_longlong),
        ("adopted_cands", ctypes.c_longlong),
    ]


@dataclass
class OracleDesc:
    d_out: int
    d_in: int
    n_heads: int
    d_head: int
    bits: int
    quant_group: int = 0
    out_block: int = 1
    n_hin: int = 1
    n_cand: int = 16
    cd_iters: int = 1
    flags: int = 0

    def c(self) -> _Desc:
        return _Desc(self.d_out, self.d_in, self.n_heads, self.d_head, self.n_hin, self.bits,
                     self.quant_group, self.out_block, self.n_cand, self.cd_iters, self.flags)

    @property
    def n_groups(self) -> int:
        return 1 if self.quant_group == 0 else self.d_in // self.quant_group


@dataclass
class OracleResult:
    codes: np.ndarray
    scales: np.ndarray
    zeros: np.ndarray
    cand: np.ndarray
    w_hat: np.ndarray
    w_comp: np.ndarray
    scales_pre_cd: np.ndarray
    loss: np.ndarray
    counters: dict = field(default_factory=dict)


def _load():
    global _lib
    if _lib is None:
        build_oracle()
        _lib = ctypes.CDLL(_LIB)
        _lib.tbo_loss_head.restype = ctypes.c_double
        _lib.tbo_quantize_layer.restype = ctypes.c_int
        _lib.tbo_num_threads.restype = ctypes.c_int
    return _lib


def _p(a, ct=ctypes.c_double):
    if a is None:
        return None
    return a.ctypes.data_as(ctypes.POINTER(ct))


def _f64(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.float64)


def num_threads() -> int:
    return int(_load().tbo_num_threads())


# ----------------------------------------------------------------------------
# Dense steps with a textbook definition (numpy float64 routines as steps)
# ----------------------------------------------------------------------------

def hessian(X, damp: float = 0.0, return_sum: bool = False):
    """H_in = X^T X / n (+ damp * mean(diag) * I).  X is [n_tok, d]; the paper's
    X is its transpose, so this is X X^T of Table 1, divided by the token count."""
    X = _f64(X)
    n = X.shape[0]
    Hs = X.T @ X / n
    H = Hs + damp * np.mean(np.diag(Hs)) * np.eye(Hs.shape[0])
    return (H, Hs) if return_sum else H


def cross_correlation(X, Xfp, alpha: float):
    """R = alpha (X - Xfp) X^T in the paper's layout (Algorithm 1, deviation step), i.e.
    R[a, b] = alpha / n * sum_t (x_t[a] - xfp_t[a]) x_t[b] for token-major X."""
    X, Xfp = _f64(X), _f64(Xfp)
    return alpha * ((X - Xfp).T @ X) / X.shape[0]


def hout_from_projection(G, Hsum, n_heads: int, d_head: int, damp: float = 0.0):
    """Out-channel Hessians of Table 1 from the partner projection.

    G is [g_heads * d_head, d]: rows of W_K (when W_Q is quantized), of W_Q
    (when W_K is quantized) or of W_out^T (when W_V is quantized; then Hsum is
    None and the middle factor is the identity).  H_out of block b is
    G_b Hsum G_b^T, which is K_h^T K_h (resp. Q_h^T Q_h, W_out,h^T W_out,h)
    with K_h = (G_b X)^T.  With grouped-query attention the number of blocks in
    G and n_heads differ by an integer factor: a query head takes the block of
    its key/value head; a key/value head takes the sum over its query heads."""
    G = _f64(G)
    d = G.shape[1]
    g_heads = G.shape[0] // d_head
    M = np.eye(d) if Hsum is None else _f64(Hsum)
    blocks = []
    for b in range(g_heads):
        Gb = G[b * d_head:(b + 1) * d_head]
        blocks.append(Gb @ M @ Gb.T)
    out = np.zeros((n_heads, d_head, d_head))
    if g_heads >= n_heads:
        rep = g_heads // n_heads
        for h in range(n_heads):
            for r in range(rep):
                out[h] += blocks[h * rep + r]
    else:
        rep = n_heads // g_heads
        for h in range(n_heads):
            out[h] = blocks[h // rep]
    for h in range(n_heads):
        out[h] += damp * np.mean(np.diag(out[h])) * np.eye(d_head)
    return out


def factor_upper(H):
    """U = Chol(H^{-1})^T, upper triangular with H^{-1} = U^T U (Eq. 2).
    Written as the definition: invert, lower Cholesky, transpose."""
    H = _f64(H)
    if H.ndim == 3:
        return np.stack([factor_upper(h) for h in H])
    Hinv = np.linalg.inv(H)
    Hinv = 0.5 * (Hinv + Hinv.T)
    L = np.linalg.cholesky(Hinv)
    return np.ascontiguousarray(L.T)


def correction_operands(R, U):
    """P = ((R U^T) * M_U) U with M_U the strictly-upper mask (Algorithm 2,
    its masked operand) and C = R H_in^{-1} = R U^T U (Proposition 3.2)."""
    R, U = _f64(R), _f64(U)
    if R.ndim == 3:
        pc = [correction_operands(r, u) for r, u in zip(R, U)]
        return np.stack([p for p, _ in pc]), np.stack([c for _, c in pc])
    RUt = R @ U.T
    P = np.triu(RUt, k=1) @ U
    C = RUt @ U
    return np.ascontiguousarray(P), np.ascontiguousarray(C)


# ----------------------------------------------------------------------------
# The C loops
# ----------------------------------------------------------------------------

def quantize_layer(desc: OracleDesc, W, Hin, Uin, Hout=None, Uout=None, R=None, P=None, C=None,
                   hint_codes=None, hint_zeros=None, hint_cand=None, band: float = 1e-6,
                   cand_tol: float = 0.0) -> OracleResult:
    lib = _load()
    W, Hin, Uin = _f64(W), _f64(Hin), _f64(Uin)
    Hout, Uout, R, P, C = _f64(Hout), _f64(Uout), _f64(R), _f64(P), _f64(C)
    ng = desc.n_groups
    codes = np.zeros((desc.d_out, desc.d_in), np.uint8)
    scales = np.ones((desc.d_out, ng), np.float64)
    zeros = np.zeros((desc.d_out, ng), np.int32)
    cand = np.zeros((desc.d_out, ng), np.uint8)
    w_hat = np.zeros((desc.d_out, desc.d_in), np.float64)
    w_comp = np.zeros((desc.d_out, desc.d_in), np.float64)
    s_pre = np.ones((desc.d_out, ng), np.float64)
    loss = np.zeros(desc.n_heads, np.float64)
    cnt = _Counters()
    if hint_codes is not None:
        hint_codes = np.ascontiguousarray(hint_codes, np.uint8)
    if hint_zeros is not None:
        hint_zeros = np.ascontiguousarray(hint_zeros, np.int32)
    if hint_cand is not None:
        hint_cand = np.ascontiguousarray(hint_cand, np.uint8)
    cd = desc.c()
    rc = lib.tbo_quantize_layer(
        ctypes.byref(cd), _p(W), _p(Hin), _p(Uin), _p(Hout), _p(Uout), _p(R), _p(P), _p(C),
        ctypes.c_double(band), ctypes.c_double(cand_tol),
        _p(hint_codes, ctypes.c_ubyte), _p(hint_zeros, ctypes.c_int), _p(hint_cand, ctypes.c_ubyte),
        _p(codes, ctypes.c_ubyte), _p(scales), _p(zeros, ctypes.c_int), _p(cand, ctypes.c_ubyte),
        _p(w_hat), _p(w_comp), _p(s_pre), _p(loss), ctypes.byref(cnt))
    if rc != 0:
        raise ValueError(f"oracle rejected the layer description (code {rc})")
    counters = {k: int(getattr(cnt, k)) for k, _ in _Counters._fields_}
    return OracleResult(codes, scales, zeros, cand, w_hat, w_comp, s_pre, loss, counters)


def grid_rows(W0, Hin, gq: int, bits: int, n_cand: int = 16, with_scores: bool = False):
    lib = _load()
    W0, Hin = _f64(W0), _f64(Hin)
    m, d = W0.shape
    ng = 1 if gq == 0 else d // gq
    s = np.ones((m, ng))
    z = np.zeros((m, ng), np.int32)
    cand = np.zeros((m, ng), np.uint8)
    scores = np.zeros((m, ng, n_cand)) if with_scores else None
    lib.tbo_grid_rows(_p(W0), m, d, gq, _p(Hin), bits, n_cand, _p(s), _p(z, ctypes.c_int),
                      _p(cand, ctypes.c_ubyte), _p(scores))
    return (s, z, cand, scores) if with_scores else (s, z, cand)


def sweep_rows(W0, Uin, s, z, gq: int, bits: int, P=None, band: float = 1e-6, hint_codes=None, Hin_dyn=None,
               n_cand: int = 16):
    """Hin_dyn given: the dynamic-grid variant; s and z may be None and the grids found in the sweep are
    returned as two extra values."""
    lib = _load()
    W0, Uin, P = _f64(W0), _f64(Uin), _f64(P)
    m, d = W0.shape
    ng = 1 if gq == 0 else d // gq
    Hin_dyn = _f64(Hin_dyn)
    s = np.ones((m, ng)) if s is None else np.array(s, dtype=np.float64, copy=True)
    z = np.zeros((m, ng), np.int32) if z is None else np.array(z, dtype=np.int32, copy=True)
    codes = np.zeros((m, d), np.uint8)
    Q = np.zeros((m, d))
    err = np.zeros((m, d))
    cnt = _Counters()
    if hint_codes is not None:
        hint_codes = np.ascontiguousarray(hint_codes, np.uint8)
    lib.tbo_sweep_rows(_p(W0), m, d, gq, _p(Uin), _p(P), _p(s), _p(z, ctypes.c_int), bits,
                       ctypes.c_double(band), _p(hint_codes, ctypes.c_ubyte),
                       _p(codes, ctypes.c_ubyte), _p(Q), _p(err), ctypes.byref(cnt), _p(Hin_dyn), n_cand)
    counters = {k: int(getattr(cnt, k)) for k, _ in _Counters._fields_}
    if Hin_dyn is not None:
        return codes, Q, err, counters, s, z
    return codes, Q, err, counters


def comp_matrix(Uout, i0: int, nb: int):
    lib = _load()
    Uout = _f64(Uout)
    dh = Uout.shape[0]
    T = np.zeros((dh - i0 - nb, nb))
    lib.tbo_comp_matrix(_p(Uout), dh, i0, nb, _p(T))
    return T


def cd_refine(desc: OracleDesc, W, codes, zeros, scales, Hin, Hout=None, R=None):
    """One head (desc.d_head rows).  Returns the refined scales."""
    lib = _load()
    W, Hin, Hout, R = _f64(W), _f64(Hin), _f64(Hout), _f64(R)
    codes = np.ascontiguousarray(codes, np.uint8)
    zeros = np.ascontiguousarray(zeros, np.int32)
    s = np.array(scales, dtype=np.float64, copy=True)
    cd = desc.c()
    lib.tbo_cd_refine(ctypes.byref(cd), _p(W), _p(codes, ctypes.c_ubyte), _p(zeros, ctypes.c_int),
                      _p(s), _p(Hin), _p(Hout), _p(R))
    return s


def loss_head(W, Q, Hin, Hout=None, R=None) -> float:
    lib = _load()
    W, Q, Hin, Hout, R = _f64(W), _f64(Q), _f64(Hin), _f64(Hout), _f64(R)
    dh, d = W.shape
    return float(lib.tbo_loss_head(dh, d, _p(W), _p(Q), _p(Hin), _p(Hout), _p(R)))


def group_loop_trace(desc: OracleDesc, W, Hin, Uin, Uout=None, P=None, C=None):
    """Group loop of ONE head, recording W-tilde after every step.
    Returns dict(codes, scales, zeros, Q, w_comp, trace[n_steps, dh, d])."""
    lib = _load()
    W, Hin, Uin, Uout, P, C = _f64(W), _f64(Hin), _f64(Uin), _f64(Uout), _f64(P), _f64(C)
    dh, d = W.shape
    ng = desc.n_groups
    N = desc.out_block if Uout is not None else dh
    n_steps = (dh + N - 1) // N
    Wt = W.copy()
    codes = np.zeros((dh, d), np.uint8)
    scales = np.ones((dh, ng))
    zeros = np.zeros((dh, ng), np.int32)
    Q = np.zeros((dh, d))
    w_comp = np.zeros((dh, d))
    trace = np.zeros((n_steps, dh, d))
    cd = desc.c()
    lib.tbo_group_loop_trace(ctypes.byref(cd), _p(Wt), _p(Hin), _p(Uin), _p(Uout), _p(P), _p(C),
                             _p(codes, ctypes.c_ubyte), _p(scales), _p(zeros, ctypes.c_int), _p(Q),
                             _p(w_comp), _p(trace))
    return dict(codes=codes, scales=scales, zeros=zeros, Q=Q, w_comp=w_comp, trace=trace)


# ----------------------------------------------------------------------------
# Packed integer weights (Section 2.1: Q = diag(s) W_int, W_int in {0 .. 2^b - 1})
# ----------------------------------------------------------------------------

def pack_codes(codes, bits: int):
    """Row-wise little-endian bit stream: code j of a row in bits [j b, (j + 1) b) from the least
    significant bit of the row's first 32-bit word.  Written bit by bit (one boolean per stream bit)."""
    codes = np.ascontiguousarray(codes, np.uint8)
    d_out, d_in = codes.shape
    if (d_in * bits) % 32:
        raise ValueError("a row must fill whole 32-bit words")
    stream = np.zeros((d_out, d_in, bits), np.uint8)
    for k in range(bits):
        stream[:, :, k] = (codes >> k) & 1          # bit k of code j is stream bit j * bits + k
    stream = stream.reshape(d_out, d_in * bits // 32, 32).astype(np.uint64)
    words = np.zeros(stream.shape[:2], np.uint64)
    for k in range(32):
        words |= stream[:, :, k] << np.uint64(k)
    return words.astype(np.uint32)


def unpack_codes(packed, bits: int, d_in: int):
    packed = np.ascontiguousarray(packed, np.uint32)
    d_out = packed.shape[0]
    stream = np.zeros((d_out, packed.shape[1], 32), np.uint8)
    for k in range(32):
        stream[:, :, k] = (packed >> np.uint32(k)) & np.uint32(1)
    stream = stream.reshape(d_out, d_in, bits)
    codes = np.zeros((d_out, d_in), np.uint8)
    for k in range(bits):
        codes |= stream[:, :, k] << k
    return codes


def dequantize(codes, scales, zeros, quant_group: int):
    """Q = s (W_int - z) per (row, column group), float64 (Algorithm 1, final step)."""
    codes = np.asarray(codes)
    seg = quant_group or codes.shape[1]
    s = np.repeat(np.asarray(scales, np.float64), seg, axis=1)
    z = np.repeat(np.asarray(zeros, np.float64), seg, axis=1)
    return s * (codes.astype(np.float64) - z)
