"""Pins of the oracle's projection for the write step (K = X W_K, V = X W_V; Sec. 2.1 and the write step of Sec. 2.2):
brute force over tiny inputs, closed forms (identity and selector weights), linearity, and the library's linear layer."""
import numpy as np
import torch

from oracle import moda_oracle as orc


def test_brute_force_on_tiny_inputs():
    rng = np.random.default_rng(0)
    B, T, D, Hk, d = 2, 3, 5, 2, 4
    X, Wk, Wv = rng.standard_normal((B, T, D)), rng.standard_normal((Hk * d, D)), rng.standard_normal((Hk * d, D))
    K, V = orc.project_kv(X, Wk, Wv, Hk)
    assert K.shape == V.shape == (B, T, Hk, d)
    for b in range(B):
        for t in range(T):
            for h in range(Hk):
                for j in range(d):
                    k = sum(X[b, t, m] * Wk[h * d + j, m] for m in range(D))
                    v = sum(X[b, t, m] * Wv[h * d + j, m] for m in range(D))
                    assert abs(K[b, t, h, j] - k) < 1e-12 and abs(V[b, t, h, j] - v) < 1e-12


def test_identity_and_selector_weights():
    rng = np.random.default_rng(1)
    B, T, Hk, d = 1, 7, 2, 3
    D = Hk * d
    X = rng.standard_normal((B, T, D))
    K, V = orc.project_kv(X, np.eye(D), 2.0 * np.eye(D), Hk)
    assert np.array_equal(K.reshape(B, T, D), X) and np.array_equal(V.reshape(B, T, D), 2.0 * X)
    # a weight row that picks input feature m puts X[..., m] at that output feature; key and value weights are not swapped
    Wk = np.zeros((D, D)); Wk[4, 1] = 1.0
    Wv = np.zeros((D, D)); Wv[0, 5] = 1.0
    K, V = orc.project_kv(X, Wk, Wv, Hk)
    assert np.array_equal(K[0, :, 1, 1], X[0, :, 1]) and np.count_nonzero(K) == np.count_nonzero(X[0, :, 1])
    assert np.array_equal(V[0, :, 0, 0], X[0, :, 5]) and np.count_nonzero(V) == np.count_nonzero(X[0, :, 5])


def test_linearity_and_the_library_linear_layer():
    rng = np.random.default_rng(2)
    B, T, D, Hk, d = 2, 9, 16, 2, 8
    X1, X2 = rng.standard_normal((B, T, D)), rng.standard_normal((B, T, D))
    Wk, Wv = rng.standard_normal((Hk * d, D)), rng.standard_normal((Hk * d, D))
    K1, V1 = orc.project_kv(X1, Wk, Wv, Hk)
    K2, V2 = orc.project_kv(X2, Wk, Wv, Hk)
    K3, V3 = orc.project_kv(2.0 * X1 - 3.0 * X2, Wk, Wv, Hk)
    assert np.allclose(K3, 2.0 * K1 - 3.0 * K2, rtol=0, atol=1e-12) and np.allclose(V3, 2.0 * V1 - 3.0 * V2, rtol=0, atol=1e-12)
    Kl = torch.nn.functional.linear(torch.from_numpy(X1), torch.from_numpy(Wk)).numpy().reshape(B, T, Hk, d)
    Vl = torch.nn.functional.linear(torch.from_numpy(X1), torch.from_numpy(Wv)).numpy().reshape(B, T, Hk, d)
    assert np.allclose(K1, Kl, rtol=0, atol=1e-12) and np.allclose(V1, Vl, rtol=0, atol=1e-12)
