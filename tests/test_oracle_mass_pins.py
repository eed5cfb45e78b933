"""Pins of the oracle's depth-slot attention mass (the depth probabilities of Sec. 2.2's single softmax, summed over the
positions): brute force with an explicit softmax over the union of keys, conservation of probability against a library
softmax over the flattened key set, a closed form (harmonic sums when every score is equal), slot permutation, l = 0."""
import numpy as np
import torch

from oracle import moda_oracle as orc


def _inputs(B, T, Hq, Hk, d, l, seed):
    rng = np.random.default_rng(seed)
    Q = rng.standard_normal((B, T, Hq, d))
    K, V = rng.standard_normal((B, T, Hk, d)), rng.standard_normal((B, T, Hk, d))
    Kd, Vd = rng.standard_normal((l, B, T, Hk, d)), rng.standard_normal((l, B, T, Hk, d))
    return Q, K, V, Kd, Vd


def test_brute_force_with_an_explicit_softmax_over_the_union():
    B, T, Hq, Hk, d, l = 2, 5, 4, 2, 3, 3
    scale = 0.37
    Q, K, V, Kd, Vd = _inputs(B, T, Hq, Hk, d, l, 0)
    _, LSE = orc.forward_gqa(Q, K, V, Kd, Vd, scale)
    mass = orc.depth_slot_mass(Q, Kd, LSE, scale)
    G = Hq // Hk
    for b in range(B):
        for h in range(Hq):
            want = np.zeros(l)
            for t in range(T):
                s = [scale * float(Q[b, t, h] @ K[b, j, h // G]) for j in range(t + 1)]
                u = [scale * float(Q[b, t, h] @ Kd[i, b, t, h // G]) for i in range(l)]
                z = sum(np.exp(x) for x in s + u)
                for i in range(l):
                    want[i] += np.exp(u[i]) / z
            assert np.allclose(mass[b, h], want, rtol=1e-12, atol=1e-14)


def test_probability_is_conserved_against_a_library_softmax():
    # per (b, h): depth mass + sequence mass = T, the sequence mass taken from torch.softmax over the flattened key set
    B, T, H, d, l = 1, 9, 2, 4, 4
    scale = d ** -0.5
    Q, K, V, Kd, Vd = _inputs(B, T, H, H, d, l, 1)
    _, LSE = orc.forward(Q, K, V, Kd, Vd, scale)
    mass = orc.depth_slot_mass(Q, Kd, LSE, scale)
    for h in range(H):
        q = torch.from_numpy(Q[0, :, h])                               # [T, d]
        s = scale * q @ torch.from_numpy(K[0, :, h]).T                 # [T, T]
        s = s.masked_fill(torch.triu(torch.ones(T, T, dtype=torch.bool), 1), float("-inf"))
        u = scale * torch.einsum("td,itd->ti", q, torch.from_numpy(Kd[:, 0, :, h]))   # [T, l]
        p = torch.softmax(torch.cat([s, u], dim=1), dim=1).numpy()
        assert np.allclose(mass[0, h], p[:, T:].sum(axis=0), rtol=1e-12)
        assert abs(mass[0, h].sum() + p[:, :T].sum() - T) < 1e-12


def test_equal_scores_give_harmonic_sums():
    # q = 0: every visible key has the same probability 1 / (t + 1 + l), so every slot collects sum_t 1 / (t + 1 + l)
    B, T, H, d, l = 1, 12, 1, 2, 3
    Q, K, V, Kd, Vd = _inputs(B, T, H, H, d, l, 2)
    Q[:] = 0
    _, LSE = orc.forward(Q, K, V, Kd, Vd, 0.5)
    mass = orc.depth_slot_mass(Q, Kd, LSE, 0.5)
    want = sum(1.0 / (t + 1 + l) for t in range(T))
    assert np.allclose(mass, want, rtol=1e-13)


def test_slot_permutation_and_no_slots():
    B, T, Hq, Hk, d, l = 1, 6, 2, 1, 3, 4
    Q, K, V, Kd, Vd = _inputs(B, T, Hq, Hk, d, l, 3)
    _, LSE = orc.forward_gqa(Q, K, V, Kd, Vd, 0.6)
    mass = orc.depth_slot_mass(Q, Kd, LSE, 0.6)
    perm = [2, 0, 3, 1]
    _, LSE_p = orc.forward_gqa(Q, K, V, Kd[perm], Vd[perm], 0.6)
    assert np.allclose(LSE_p, LSE, rtol=1e-13)
    assert np.allclose(orc.depth_slot_mass(Q, Kd[perm], LSE_p, 0.6), mass[:, :, perm], rtol=1e-12)
    _, LSE0 = orc.forward_gqa(Q, K, V, None, None, 0.6)
    assert orc.depth_slot_mass(Q, np.zeros((0, B, T, Hk, d)), LSE0, 0.6).shape == (B, Hq, 0)
