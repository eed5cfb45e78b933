"""Pins of the decode-step function of the fp64 oracle (CPU only).

Decode (T_q = 1): the newest token attends to its layer's T_kv cached sequence keys and to its own
l depth key/value pairs (paper Table 1, decoding cache of 2 l H_k d values per token).

  D1  library attention (no mask, one query row) over the concatenated key set, and library logsumexp
  D2  the last row of the separately pinned full-sequence oracle on the same tensors
  D3  closed forms: identical keys give the mean of the values and LSE = s + log(n); one very large
      score selects its value; l = 0 is plain attention of the last token
  D4  a depth key counts exactly like a sequence key: moving a pair from the depth set to the end of
      the sequence set changes nothing
"""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import moda_oracle as orc


def rand(rng, B, Tkv, Hq, Hk, d, l):
    return (rng.standard_normal((B, Hq, d)), rng.standard_normal((B, Tkv, Hk, d)), rng.standard_normal((B, Tkv, Hk, d)),
            rng.standard_normal((l, B, Hk, d)), rng.standard_normal((l, B, Hk, d)))


@pytest.mark.parametrize("B,Tkv,Hq,Hk,d,l", [(1, 7, 2, 1, 4, 3), (2, 33, 4, 2, 8, 5), (1, 1, 2, 2, 4, 2), (2, 20, 6, 2, 8, 0)])
def test_d1_library_attention_over_the_concatenated_keys(B, Tkv, Hq, Hk, d, l):
    rng = np.random.default_rng(Tkv)
    q, K, V, kd, vd = rand(rng, B, Tkv, Hq, Hk, d, l)
    scale = 0.37
    o, lse = orc.decode_gqa(q, K, V, kd, vd, scale)
    G = Hq // Hk
    tq = torch.from_numpy(q)[:, :, None, :]                                             # [B,Hq,1,d]
    keys = torch.cat([torch.from_numpy(K).permute(0, 2, 1, 3), torch.from_numpy(kd).permute(1, 2, 0, 3)], dim=2)
    vals = torch.cat([torch.from_numpy(V).permute(0, 2, 1, 3), torch.from_numpy(vd).permute(1, 2, 0, 3)], dim=2)
    keys, vals = keys.repeat_interleave(G, dim=1), vals.repeat_interleave(G, dim=1)    # [B,Hq,T_kv+l,d]
    ref = F.scaled_dot_product_attention(tq, keys, vals, scale=scale)[:, :, 0, :]
    ref_lse = torch.logsumexp((tq @ keys.transpose(-1, -2))[:, :, 0, :] * scale, dim=-1)
    np.testing.assert_allclose(o, ref.numpy(), rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(lse, ref_lse.numpy(), rtol=1e-12, atol=1e-12)


@pytest.mark.parametrize("B,T,Hq,Hk,d,l", [(1, 9, 2, 1, 4, 3), (2, 17, 4, 2, 8, 2), (1, 6, 3, 3, 4, 0)])
def test_d2_last_row_of_the_full_sequence_oracle(B, T, Hq, Hk, d, l):
    rng = np.random.default_rng(50 + T)
    Q = rng.standard_normal((B, T, Hq, d)); K = rng.standard_normal((B, T, Hk, d)); V = rng.standard_normal((B, T, Hk, d))
    Kd = rng.standard_normal((l, B, T, Hk, d)); Vd = rng.standard_normal((l, B, T, Hk, d))
    O, LSE = orc.forward_gqa(Q, K, V, Kd, Vd, 0.5)
    o, lse = orc.decode_gqa(Q[:, -1], K, V, Kd[:, :, -1] if l else None, Vd[:, :, -1] if l else None, 0.5)
    np.testing.assert_allclose(o, O[:, -1], rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(lse, LSE[:, :, -1], rtol=1e-11, atol=1e-12)
    # and a shorter cache is the row of that position
    t = T // 2
    o, lse = orc.decode_gqa(Q[:, t], K[:, :t + 1], V[:, :t + 1], Kd[:, :, t] if l else None, Vd[:, :, t] if l else None, 0.5)
    np.testing.assert_allclose(o, O[:, t], rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(lse, LSE[:, :, t], rtol=1e-11, atol=1e-12)


def test_d3_closed_forms():
    rng = np.random.default_rng(3)
    B, Tkv, Hq, Hk, d, l = 1, 11, 2, 1, 4, 5
    q, K, V, kd, vd = rand(rng, B, Tkv, Hq, Hk, d, l)
    k0 = rng.standard_normal(d)
    K[:] = k0; kd[:] = k0
    o, lse = orc.decode_gqa(q, K, V, kd, vd, 0.7)
    mean = (V[0, :, 0].sum(0) + vd[:, 0, 0].sum(0)) / (Tkv + l)
    for h in range(Hq):
        np.testing.assert_allclose(o[0, h], mean, rtol=1e-12)
        np.testing.assert_allclose(lse[0, h], 0.7 * (q[0, h] @ k0) + np.log(Tkv + l), rtol=1e-12)
    # one dominant depth key selects its value
    q, K, V, kd, vd = rand(rng, B, Tkv, Hq, Hk, d, l)
    kd[2, 0, 0] = 200.0 * q[0, 0] / (q[0, 0] @ q[0, 0])
    o, _ = orc.decode_gqa(q[:, :1], K, V, kd, vd, 1.0)
    np.testing.assert_allclose(o[0, 0], vd[2, 0, 0], atol=1e-9)
    # l = 0: plain attention of one row
    o, lse = orc.decode_gqa(q, K, V, None, None, 0.3)
    s = np.einsum("hd,td->ht", q[0], K[0, :, 0]) * 0.3
    p = np.exp(s - s.max(1, keepdims=True)); p /= p.sum(1, keepdims=True)
    np.testing.assert_allclose(o[0], p @ V[0, :, 0], rtol=1e-12)
    np.testing.assert_allclose(lse[0], np.log(np.exp(s).sum(1)), rtol=1e-12)


def test_d4_depth_pairs_count_like_sequence_pairs():
    rng = np.random.default_rng(8)
    B, Tkv, Hq, Hk, d, l = 2, 6, 4, 2, 8, 3
    q, K, V, kd, vd = rand(rng, B, Tkv, Hq, Hk, d, l)
    o1, lse1 = orc.decode_gqa(q, K, V, kd, vd, 0.4)
    K2 = np.concatenate([K, kd[-1][:, None]], axis=1); V2 = np.concatenate([V, vd[-1][:, None]], axis=1)
    o2, lse2 = orc.decode_gqa(q, K2, V2, kd[:-1], vd[:-1], 0.4)
    np.testing.assert_allclose(o1, o2, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(lse1, lse2, rtol=1e-12, atol=1e-13)


def test_invalid_shapes_are_rejected():
    with pytest.raises(ValueError):
        orc.decode_gqa(np.zeros((1, 3, 4)), np.zeros((1, 5, 2, 4)), np.zeros((1, 5, 2, 4)), None, None, 1.0)
    with pytest.raises(ValueError):
        orc.decode_gqa(np.zeros((1, 2, 4)), np.zeros((1, 0, 2, 4)), np.zeros((1, 0, 2, 4)), None, None, 1.0)
