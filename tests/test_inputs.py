"""The seeded input recipes that serve both the oracle and the CUDA path (no method arithmetic)."""
import numpy as np

import tb_inputs


def test_causal_decay_mix_is_the_normalised_decay_matrix():
    """X-bar = A_h X with A_h[t][s] = rho^(t-s) / sum_{s'<=t} rho^(t-s'), restarted at every sequence."""
    X = tb_inputs.HeavyTailRecipe(8, seed=3).chunk(0, 10)
    rho = tb_inputs.decay_rate(1)
    assert rho == 0.75
    got = tb_inputs.causal_decay_mix(X, rho, seq_len=5, bf16=False)
    A = np.zeros((10, 10))
    for t in range(10):
        s0 = (t // 5) * 5
        for s in range(s0, t + 1):
            A[t, s] = rho ** (t - s)
    A /= A.sum(axis=1, keepdims=True)
    assert np.allclose(got, A @ X.astype(np.float64), rtol=0, atol=1e-6 * np.abs(X).max())
    # rows of A sum to one: a constant input is left unchanged
    ones = np.ones((7, 3), np.float32)
    assert np.array_equal(tb_inputs.causal_decay_mix(ones, 0.5, seq_len=4, bf16=False), ones)
    assert [tb_inputs.decay_rate(h) for h in (0, 5, 6)] == [0.5, 1 - 2.0 ** -6, 0.5]


def test_explicit_decay_matrix_equals_the_recurrence():
    X = tb_inputs.HeavyTailRecipe(8, seed=4).chunk(0, 12, bf16=False)
    A = tb_inputs.causal_decay_matrix(0.875, 6)
    assert np.allclose(A.sum(axis=1), 1.0) and np.array_equal(A, np.tril(A))
    want = tb_inputs.causal_decay_mix(X, 0.875, seq_len=6, bf16=False)
    got = np.concatenate([A @ X[:6].astype(np.float64), A @ X[6:].astype(np.float64)])
    assert np.allclose(got, want, rtol=0, atol=1e-6 * np.abs(X).max())


def test_device_recipes_have_the_structure_of_the_numpy_ones():
    """The torch twins of the recipes (run here on the CPU device): bf16, right shapes, the outlier
    channels about outlier_scale times larger, a deviation of the stated relative size, and the mixing
    equal to the numpy recurrence."""
    import torch
    rec = tb_inputs.HeavyTailRecipe(256, seed=2)
    X = tb_inputs.heavy_tail_device(rec, 4096, torch.device("cpu"), chunk=1000)
    assert X.dtype == torch.bfloat16 and tuple(X.shape) == (4096, 256)
    rms = X.float().pow(2).mean(dim=0).sqrt().numpy()
    out = rec.sigma_c > 1
    assert 10 < np.median(rms[out]) / np.median(rms[~out]) < 40
    ref_rms = np.sqrt((rec.chunk(0, 4096) ** 2).mean(axis=0))
    assert 0.8 < np.median(rms[~out]) / np.median(ref_rms[~out]) < 1.25
    Xq = tb_inputs.deviation_device(tb_inputs.DeviationRecipe(rec), X, chunk=1000)
    rel = float((Xq.float() - X.float()).norm() / X.float().norm())
    xs, xf = tb_inputs.DeviationRecipe(rec).chunk(0, 4096)
    rel_ref = float(np.linalg.norm(xs - xf) / np.linalg.norm(xf))
    assert 0.5 * rel_ref < rel < 2.0 * rel_ref
    Xf = X[:600].float()
    mixed = tb_inputs.causal_decay_mix_device(Xf, 0.75, 256)
    want = tb_inputs.causal_decay_mix(Xf.numpy(), 0.75, 256, bf16=False)
    assert np.allclose(mixed.numpy(), want, rtol=0, atol=1e-4 * float(Xf.abs().max()))
