"""Seeded synthetic inputs shared by the tests, the benchmark and the oracle checks.

This module only draws random tensors with the shapes and statistics of the
five benchmark configurations.  It contains none of the quantizer's
arithmetic and imports neither the CUDA package nor the oracle.  The synthetic
tensors stand in for Llama projection weights and WikiText-2 calibration
activations (128 sequences x 2048 tokens), which are not available offline.

Every tensor comes from a counter-based Philox stream keyed by (seed,
tensor id), so any tensor can be regenerated independently of the others.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

# tensor ids (fixed; part of the recipe)
T_W, T_WPARTNER, T_X, T_XFACTOR, T_XLOAD, T_XTOK, T_OUTLIER, T_HOUT, T_DEV, T_DEVN, T_WOUT = range(11)


def _rng(seed: int, tid: int, sub: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[(seed << 8) + tid, sub]))


def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bfloat16 bit patterns (uint16), round-to-nearest-even."""
    u = np.ascontiguousarray(x, np.float32).view(np.uint32)
    r = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
    return (r >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def weight(seed: int, d_out: int, d_in: int, tid: int = T_W, std: float = 0.02) -> np.ndarray:
    """Projection weight ~ N(0, std^2), float32, row = out-channel."""
    return (_rng(seed, tid).standard_normal((d_out, d_in), dtype=np.float32) * np.float32(std))


def outlier_channels(seed: int, d: int, count: int) -> np.ndarray:
    return np.sort(_rng(seed, T_OUTLIER).permutation(d)[:count])


def activations_gaussian(seed: int, n_tok: int, d: int, n_outlier: int = 4,
                         outlier_scale: float = 20.0) -> np.ndarray:
    """Tiny-config activations: N(0,1) with a few channels scaled up."""
    X = _rng(seed, T_X).standard_normal((n_tok, d), dtype=np.float32)
    X[:, outlier_channels(seed, d, n_outlier)] *= np.float32(outlier_scale)
    return X


@dataclass
class HeavyTailRecipe:
    """x_t = sigma_c * tau_t * (n_t + 2 F f_t): per-channel outlier scale sigma_c
    (outlier_scale on outlier_frac of the channels), log-normal per-token scale
    tau_t, and a rank-`rank` common factor that makes X^T X ill-conditioned."""
    d: int
    seed: int = 0
    rank: int = 64
    outlier_frac: float = 0.01
    outlier_scale: float = 20.0
    tok_sigma: float = 0.5
    tid_shift: int = 0  # distinct streams for a second activation tensor

    def __post_init__(self):
        n_out = max(1, int(round(self.outlier_frac * self.d)))
        self.sigma_c = np.ones(self.d, np.float32)
        self.sigma_c[outlier_channels(self.seed + self.tid_shift, self.d, n_out)] = self.outlier_scale
        self.F = (_rng(self.seed, T_XLOAD, self.tid_shift).standard_normal((self.rank, self.d), dtype=np.float32)
                  / np.float32(np.sqrt(self.rank)))

    def chunk(self, t0: int, n: int, bf16: bool = True) -> np.ndarray:
        """Tokens t0..t0+n-1 as float32 (values representable in bf16 if bf16)."""
        g = _rng(self.seed, T_X, (self.tid_shift << 40) + t0)
        noise = g.standard_normal((n, self.d), dtype=np.float32)
        f = _rng(self.seed, T_XFACTOR, (self.tid_shift << 40) + t0).standard_normal((n, self.rank), dtype=np.float32)
        tau = np.exp(np.float32(self.tok_sigma) *
                     _rng(self.seed, T_XTOK, (self.tid_shift << 40) + t0).standard_normal((n, 1), dtype=np.float32))
        x = (noise + np.float32(2.0) * (f @ self.F)) * tau * self.sigma_c[None, :]
        if bf16:
            x = bf16_bits_to_f32(to_bf16_bits(x))
        return x


@dataclass
class DeviationRecipe:
    """Quantized-path input X = Xfp + dX with dX = 0.1 Xfp D + 0.03 sigma_c n',
    D of rank `rank` with unit spectral scale (a stand-in for the error that
    earlier quantized layers would have propagated)."""
    base: HeavyTailRecipe
    rank: int = 32

    def __post_init__(self):
        d, s = self.base.d, self.base.seed
        g = _rng(s, T_DEV, self.base.tid_shift)
        A = g.standard_normal((d, self.rank), dtype=np.float32) / np.float32(np.sqrt(d))
        B = g.standard_normal((self.rank, d), dtype=np.float32) / np.float32(np.sqrt(d))
        self.A, self.B = A, B

    def chunk(self, t0: int, n: int, bf16: bool = True):
        """Returns (X, Xfp) for tokens t0..t0+n-1."""
        xfp = self.base.chunk(t0, n, bf16=bf16)
        noise = _rng(self.base.seed, T_DEVN, (self.base.tid_shift << 40) + t0).standard_normal(
            (n, self.base.d), dtype=np.float32)
        dx = np.float32(0.1) * ((xfp @ self.A) @ self.B) + np.float32(0.03) * self.base.sigma_c[None, :] * noise
        x = xfp + dx
        if bf16:
            x = bf16_bits_to_f32(to_bf16_bits(x))
        return x, xfp


def decay_rate(head: int) -> float:
    """Decay of the synthetic causal attention of a head: rho_h = 1 - 2^-(1 + h mod 6)."""
    return 1.0 - 2.0 ** -(1 + head % 6)


def causal_decay_mix(X: np.ndarray, rho: float, seq_len: int, bf16: bool = True) -> np.ndarray:
    """Stand-in for the attention-weighted inputs A_h X of a value projection: inside every
    sequence of seq_len tokens, row t of A_h holds rho^(t-s) for s <= t, normalised to sum 1.
    Evaluated as the recurrence num_t = rho num_(t-1) + x_t, den_t = rho den_(t-1) + 1,
    xbar_t = num_t / den_t, in float64; the result is rounded to bf16-representable float32."""
    n, d = X.shape
    out = np.empty((n, d), np.float32)
    for s0 in range(0, n, seq_len):
        num = np.zeros(d, np.float64)
        den = 0.0
        for t in range(s0, min(s0 + seq_len, n)):
            num = rho * num + X[t]
            den = rho * den + 1.0
            out[t] = (num / den).astype(np.float32)
    return bf16_bits_to_f32(to_bf16_bits(out)) if bf16 else out


def causal_decay_matrix(rho: float, seq_len: int) -> np.ndarray:
    """The explicit A_h of causal_decay_mix for one sequence: A[t, s] = rho^(t-s) / sum_{s' <= t} rho^(t-s')
    for s <= t, 0 above the diagonal (float64)."""
    t = np.arange(seq_len)
    A = np.tril(rho ** np.maximum(t[:, None] - t[None, :], 0).astype(np.float64))
    return A / A.sum(axis=1, keepdims=True)


# ----------------------------------------------------------------------------
# The same recipes drawn on a CUDA device with torch's seeded generator, for tensors too large to
# draw with numpy in reasonable time (the benchmark's 128 x 2048 tokens of width 4096 or 8192).
# Same distributions and structure as the numpy recipes above (the outlier channels and the common
# factor are the numpy ones), not the same random numbers.
# ----------------------------------------------------------------------------

def heavy_tail_device(rec: "HeavyTailRecipe", n_tok: int, device, seed: int = 0, chunk: int = 16384):
    """bf16 [n_tok, d] activations of HeavyTailRecipe on `device`."""
    import torch
    g = torch.Generator(device=device)
    g.manual_seed((rec.seed << 20) + (rec.tid_shift << 10) + seed + 12345)
    F = torch.from_numpy(rec.F).to(device)
    sig = torch.from_numpy(rec.sigma_c).to(device)
    out = torch.empty((n_tok, rec.d), dtype=torch.bfloat16, device=device)
    for t0 in range(0, n_tok, chunk):
        n = min(chunk, n_tok - t0)
        noise = torch.randn((n, rec.d), generator=g, device=device)
        f = torch.randn((n, rec.rank), generator=g, device=device)
        tau = torch.exp(rec.tok_sigma * torch.randn((n, 1), generator=g, device=device))
        out[t0:t0 + n] = ((noise + 2.0 * (f @ F)) * tau * sig[None, :]).to(torch.bfloat16)
    return out


def deviation_device(dev_rec: "DeviationRecipe", Xfp, seed: int = 0, chunk: int = 16384):
    """Quantized-path twin of Xfp (bf16 on a device): X = Xfp + 0.1 Xfp A B + 0.03 sigma_c n'."""
    import torch
    device = Xfp.device
    g = torch.Generator(device=device)
    g.manual_seed((dev_rec.base.seed << 20) + (dev_rec.base.tid_shift << 10) + seed + 777)
    A = torch.from_numpy(dev_rec.A).to(device)
    B = torch.from_numpy(dev_rec.B).to(device)
    sig = torch.from_numpy(dev_rec.base.sigma_c).to(device)
    out = torch.empty_like(Xfp)
    for t0 in range(0, Xfp.shape[0], chunk):
        x = Xfp[t0:t0 + chunk].float()
        noise = torch.randn(x.shape, generator=g, device=device)
        out[t0:t0 + chunk] = (x + 0.1 * ((x @ A) @ B) + 0.03 * sig[None, :] * noise).to(torch.bfloat16)
    return out


def causal_decay_mix_device(X, rho: float, seq_len: int):
    """causal_decay_mix on a device: A_h X per sequence through the explicit matrix (float32 product)."""
    import torch
    n, d = X.shape
    A = torch.from_numpy(causal_decay_matrix(rho, seq_len).astype(np.float32)).to(X.device)
    out = torch.empty_like(X)
    for s0 in range(0, n, seq_len):
        m = min(seq_len, n - s0)
        out[s0:s0 + m] = (A[:m, :m] @ X[s0:s0 + m].float()).to(X.dtype)
    return out


def spd_matrix(seed: int, n: int, cond: float = 1e3, tid: int = T_HOUT) -> np.ndarray:
    """V diag(lambda) V^T with V the Q-factor of a Gaussian matrix and lambda
    log-spaced from 1 down to 1/cond.  float32 (the layout the library takes)."""
    g = _rng(seed, tid)
    V, _ = np.linalg.qr(g.standard_normal((n, n)))
    lam = np.logspace(0.0, -np.log10(cond), n)
    H = (V * lam[None, :]) @ V.T
    H = 0.5 * (H + H.T)
    return H.astype(np.float32)


# ----------------------------------------------------------------------------
# The five benchmark configurations
# ----------------------------------------------------------------------------

@dataclass
class Projection:
    name: str
    d_out: int
    d_in: int
    n_heads: int
    d_head: int
    partner: str | None  # which weight builds H_out: "k", "q", "o" or None (identity)


@dataclass
class Config:
    name: str
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    d_head: int
    bits: int
    quant_group: int
    out_block: int
    n_seq: int = 128
    seq_len: int = 2048
    adaptive: bool = True
    cd: bool = True
    with_r: bool = False
    alpha: float = 0.25
    damp: float = 0.01
    projections: tuple = field(default_factory=tuple)

    @property
    def n_tok(self) -> int:
        return self.n_seq * self.seq_len


def _block(d, hq, hkv, dh):
    return (Projection("q", hq * dh, d, hq, dh, "k"), Projection("k", hkv * dh, d, hkv, dh, "q"),
            Projection("v", hkv * dh, d, hkv, dh, "o"), Projection("o", d, hq * dh, 1, d, None))


CONFIGS = {
    # Tiny single projection; explicit SPD H_out; per-channel INT4; g = 8
    "tiny": Config("tiny", 256, 1, 1, 256, bits=4, quant_group=0, out_block=8, n_seq=1, seq_len=2048,
                   projections=(Projection("q", 256, 256, 1, 256, None),)),
    # Llama-2-7B-shaped q_proj; INT2, group 128, g = 32
    "l2_7b_q": Config("l2_7b_q", 4096, 32, 32, 128, bits=2, quant_group=128, out_block=32,
                      projections=(Projection("q", 4096, 4096, 32, 128, "k"),)),
    # Full Llama-2-7B-shaped attention block with the propagated-error term
    "l2_7b_block": Config("l2_7b_block", 4096, 32, 32, 128, bits=2, quant_group=128, out_block=32,
                          with_r=True, projections=_block(4096, 32, 32, 128)),
    # Llama-3-8B GQA-shaped block; INT3, g = 64
    "l3_8b_block": Config("l3_8b_block", 4096, 32, 8, 128, bits=3, quant_group=128, out_block=64,
                          projections=_block(4096, 32, 8, 128)),
    # Llama-2-70B-shaped block; INT2; g swept over {1, 8, 32, 64, 128}
    "l2_70b_block": Config("l2_70b_block", 8192, 64, 8, 128, bits=2, quant_group=128, out_block=32,
                           adaptive=False, cd=False, projections=_block(8192, 64, 8, 128)),
}
