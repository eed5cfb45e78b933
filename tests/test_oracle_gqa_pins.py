"""Pins of the grouped-query functions of the fp64 oracle (CPU only).

Grouped-query MoDA (paper Sec. 3, group-aware depth KV): Hq query heads share Hk = Hq / G
key/value heads, flattened query row i_q = t G + g has base time floor(i_q / G) = t, sees the
sequence keys up to its base time and the depth keys stored at its base time.

  G1  masked library attention over the flattened key set with the two masks the paper states
      for the group-aware kernel (floor(i_q / G) >= i_k, floor(i_q / G) == floor(j_d / L)), rows
      flattened as i_q = t G + g; forward and (through library autograd) every gradient
  G2  head repetition: the same values as the G = 1 oracle on K, V, Kd, Vd repeated G times
      along the head axis; gradients of the shared tensors are the sums over the group
  G3  G = 1 reduces to the plain functions
  G4  the paper's worked base-time example (tests/golden/paper_group_base_time_example.txt)
  G5  central finite differences on a tiny case
"""
import os

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import moda_oracle as orc


def rand_inputs(rng, B, T, Hq, Hk, d, l):
    Q = rng.standard_normal((B, T, Hq, d))
    K = rng.standard_normal((B, T, Hk, d))
    V = rng.standard_normal((B, T, Hk, d))
    Kd = rng.standard_normal((l, B, T, Hk, d))
    Vd = rng.standard_normal((l, B, T, Hk, d))
    dO = rng.standard_normal((B, T, Hq, d))
    return Q, K, V, Kd, Vd, dO


def flattened_group_attention(Q, K, V, Kd, Vd, scale):
    """Library attention per KV head over T*G flattened query rows (torch, float64)."""
    B, T, Hq, d = Q.shape
    Hk = K.shape[2]
    G = Hq // Hk
    l = Kd.shape[0]
    # rows of KV head hk: i_q = t * G + g  <->  Q[b, t, hk * G + g]
    q = Q.reshape(B, T, Hk, G, d).permute(0, 2, 1, 3, 4).reshape(B, Hk, T * G, d)
    kf = torch.cat([K.permute(0, 2, 1, 3), Kd.permute(1, 3, 2, 0, 4).reshape(B, Hk, T * l, d)], dim=2)
    vf = torch.cat([V.permute(0, 2, 1, 3), Vd.permute(1, 3, 2, 0, 4).reshape(B, Hk, T * l, d)], dim=2)
    base = torch.arange(T * G)[:, None] // G
    causal = base >= torch.arange(T)[None, :]
    depth = base == (torch.arange(T * l)[None, :] // max(l, 1))
    mask = torch.cat([causal, depth], dim=1)
    o = F.scaled_dot_product_attention(q, kf, vf, attn_mask=mask, scale=scale)
    s = (q @ kf.transpose(-1, -2)) * scale
    lse = torch.logsumexp(s.masked_fill(~mask, float("-inf")), dim=-1)            # [B,Hk,T*G]
    O = o.reshape(B, Hk, T, G, d).permute(0, 2, 1, 3, 4).reshape(B, T, Hq, d)
    LSE = lse.reshape(B, Hk, T, G).permute(0, 1, 3, 2).reshape(B, Hq, T)
    return O, LSE


@pytest.mark.parametrize("B,T,Hq,Hk,d,l", [(1, 5, 2, 1, 4, 2), (2, 9, 4, 2, 8, 3), (1, 17, 8, 2, 8, 0), (1, 12, 6, 2, 4, 5)])
def test_g1_flattened_masked_library_attention_and_autograd(B, T, Hq, Hk, d, l):
    rng = np.random.default_rng(100 + T)
    Q, K, V, Kd, Vd, dO = rand_inputs(rng, B, T, Hq, Hk, d, l)
    scale = 0.41
    O, LSE = orc.forward_gqa(Q, K, V, Kd, Vd, scale)
    ts = [torch.from_numpy(x).requires_grad_(True) for x in (Q, K, V, Kd, Vd)]
    o_ref, lse_ref = flattened_group_attention(*ts, scale)
    np.testing.assert_allclose(O, o_ref.detach().numpy(), rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(LSE, lse_ref.detach().numpy(), rtol=1e-12, atol=1e-12)
    (o_ref * torch.from_numpy(dO)).sum().backward()
    got = orc.backward_gqa(Q, K, V, Kd, Vd, dO, scale)
    for name, g, t in zip(("dQ", "dK", "dV", "dKd", "dVd"), got, ts):
        ref = t.grad.numpy() if t.grad is not None else np.zeros_like(g)
        np.testing.assert_allclose(g, ref, rtol=1e-10, atol=1e-11, err_msg=name)


@pytest.mark.parametrize("G", [2, 4])
def test_g2_head_repetition_identity(G):
    rng = np.random.default_rng(7)
    B, T, Hk, d, l = 2, 11, 2, 8, 3
    Hq = Hk * G
    Q, K, V, Kd, Vd, dO = rand_inputs(rng, B, T, Hq, Hk, d, l)
    scale = 1.0 / np.sqrt(d)
    rep = lambda x, ax: np.repeat(x, G, axis=ax)
    O, LSE = orc.forward_gqa(Q, K, V, Kd, Vd, scale)
    O1, LSE1 = orc.forward(Q, rep(K, 2), rep(V, 2), rep(Kd, 3), rep(Vd, 3), scale)
    np.testing.assert_allclose(O, O1, rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(LSE, LSE1, rtol=1e-13, atol=1e-13)
    dQ, dK, dV, dKd, dVd = orc.backward_gqa(Q, K, V, Kd, Vd, dO, scale)
    dQ1, dK1, dV1, dKd1, dVd1 = orc.backward(Q, rep(K, 2), rep(V, 2), rep(Kd, 3), rep(Vd, 3), dO, scale)
    np.testing.assert_allclose(dQ, dQ1, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(dK, dK1.reshape(B, T, Hk, G, d).sum(3), rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(dV, dV1.reshape(B, T, Hk, G, d).sum(3), rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(dKd, dKd1.reshape(l, B, T, Hk, G, d).sum(4), rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(dVd, dVd1.reshape(l, B, T, Hk, G, d).sum(4), rtol=1e-12, atol=1e-13)


def test_g3_one_head_per_group_is_the_plain_operator():
    rng = np.random.default_rng(3)
    Q, K, V, Kd, Vd, dO = rand_inputs(rng, 2, 7, 3, 3, 8, 2)
    for a, b in zip(orc.forward_gqa(Q, K, V, Kd, Vd, 0.3), orc.forward(Q, K, V, Kd, Vd, 0.3)):
        np.testing.assert_allclose(a, b, rtol=1e-14, atol=1e-14)
    for a, b in zip(orc.backward_gqa(Q, K, V, Kd, Vd, dO, 0.3), orc.backward(Q, K, V, Kd, Vd, dO, 0.3)):
        np.testing.assert_allclose(a, b, rtol=1e-12, atol=1e-13)


def test_g4_paper_base_time_example():
    path = os.path.join(os.path.dirname(__file__), "golden", "paper_group_base_time_example.txt")
    rows = [l.split() for l in open(path) if l.strip() and not l.startswith("#")]
    assert rows, "fixture is empty"
    for G, first, last, start, end in (tuple(map(int, r)) for r in rows):
        base = [orc.base_time(i, G) for i in range(first, last + 1)]
        assert min(base) == start and max(base) + 1 == end
        assert sorted(set(base)) == list(range(start, end))


def test_g5_finite_differences():
    rng = np.random.default_rng(11)
    B, T, Hq, Hk, d, l = 1, 4, 4, 2, 3, 2
    Q, K, V, Kd, Vd, dO = rand_inputs(rng, B, T, Hq, Hk, d, l)
    scale = 0.5
    grads = orc.backward_gqa(Q, K, V, Kd, Vd, dO, scale)
    args = [Q, K, V, Kd, Vd]
    loss = lambda a: float((orc.forward_gqa(*a, scale)[0] * dO).sum())
    eps = 1e-6
    for ai, (x, g) in enumerate(zip(args, grads)):
        flat = x.reshape(-1)
        for k in rng.choice(flat.size, size=min(12, flat.size), replace=False):
            old = flat[k]
            flat[k] = old + eps; up = loss(args)
            flat[k] = old - eps; dn = loss(args)
            flat[k] = old
            assert abs((up - dn) / (2 * eps) - g.reshape(-1)[k]) < 1e-6, (ai, k)


def test_group_size_must_divide_the_query_heads():
    rng = np.random.default_rng(0)
    Q, K, V, Kd, Vd, _ = rand_inputs(rng, 1, 3, 3, 2, 4, 1)
    with pytest.raises(ValueError):
        orc.forward_gqa(Q, K, V, Kd, Vd, 1.0)
