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
