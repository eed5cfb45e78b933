"""Pins of the prefill-with-cache function of the fp64 oracle (CPU only).

The T_q newest positions of a sequence attend to T_kv >= T_q cached sequence keys (causal at their
absolute positions) and to the depth pairs of their own positions.

  F1  the last T_q rows of the separately pinned full-sequence oracle over all T_kv positions
  F2  masked library attention (explicit offset-causal mask over the flattened key set) and logsumexp
  F3  T_q = T_kv is the plain forward; T_q = 1 is the decode function
"""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import moda_oracle as orc


def rand(rng, B, Tq, Tkv, Hq, Hk, d, l):
    return (rng.standard_normal((B, Tq, Hq, d)), rng.standard_normal((B, Tkv, Hk, d)), rng.standard_normal((B, Tkv, Hk, d)),
            rng.standard_normal((l, B, Tq, Hk, d)), rng.standard_normal((l, B, Tq, Hk, d)))


@pytest.mark.parametrize("B,Tq,Tkv,Hq,Hk,d,l", [(1, 3, 9, 2, 1, 4, 2), (2, 5, 5, 4, 2, 8, 3), (1, 7, 20, 3, 3, 4, 0), (1, 1, 6, 2, 2, 4, 4)])
def test_f1_last_rows_of_the_full_sequence_oracle(B, Tq, Tkv, Hq, Hk, d, l):
    rng = np.random.default_rng(7 * Tq + Tkv)
    Qf = rng.standard_normal((B, Tkv, Hq, d)); K = rng.standard_normal((B, Tkv, Hk, d)); V = rng.standard_normal((B, Tkv, Hk, d))
    Kdf = rng.standard_normal((l, B, Tkv, Hk, d)); Vdf = rng.standard_normal((l, B, Tkv, Hk, d))
    O, LSE = orc.forward_gqa(Qf, K, V, Kdf, Vdf, 0.45)
    o, lse = orc.forward_prefill_gqa(Qf[:, -Tq:], K, V, Kdf[:, :, -Tq:] if l else None, Vdf[:, :, -Tq:] if l else None, 0.45)
    np.testing.assert_allclose(o, O[:, -Tq:], rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(lse, LSE[:, :, -Tq:], rtol=1e-11, atol=1e-12)


@pytest.mark.parametrize("B,Tq,Tkv,Hq,Hk,d,l", [(1, 4, 11, 2, 1, 4, 3), (2, 6, 9, 4, 2, 8, 2)])
def test_f2_masked_library_attention(B, Tq, Tkv, Hq, Hk, d, l):
    rng = np.random.default_rng(Tkv)
    Q, K, V, Kd, Vd = rand(rng, B, Tq, Tkv, Hq, Hk, d, l)
    scale = 0.3
    o, lse = orc.forward_prefill_gqa(Q, K, V, Kd, Vd, scale)
    G = Hq // Hk
    off = Tkv - Tq
    tq = torch.from_numpy(Q).permute(0, 2, 1, 3)                                        # [B,Hq,Tq,d]
    kf = torch.cat([torch.from_numpy(K).permute(0, 2, 1, 3), torch.from_numpy(Kd).permute(1, 3, 2, 0, 4).reshape(B, Hk, Tq * l, d)], dim=2)
    vf = torch.cat([torch.from_numpy(V).permute(0, 2, 1, 3), torch.from_numpy(Vd).permute(1, 3, 2, 0, 4).reshape(B, Hk, Tq * l, d)], dim=2)
    kf, vf = kf.repeat_interleave(G, dim=1), vf.repeat_interleave(G, dim=1)
    rows = torch.arange(Tq)[:, None]
    mask = torch.cat([torch.arange(Tkv)[None, :] <= rows + off, (torch.arange(Tq * l)[None, :] // max(l, 1)) == rows], dim=1)
    ref = F.scaled_dot_product_attention(tq, kf, vf, attn_mask=mask, scale=scale).permute(0, 2, 1, 3)
    s = (tq @ kf.transpose(-1, -2)) * scale
    ref_lse = torch.logsumexp(s.masked_fill(~mask, float("-inf")), dim=-1)
    np.testing.assert_allclose(o, ref.numpy(), rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(lse, ref_lse.numpy(), rtol=1e-11, atol=1e-12)


def test_f3_the_two_ends_of_the_range():
    rng = np.random.default_rng(1)
    B, T, Hq, Hk, d, l = 1, 8, 4, 2, 4, 3
    Q, K, V, Kd, Vd = rand(rng, B, T, T, Hq, Hk, d, l)
    o, lse = orc.forward_prefill_gqa(Q, K, V, Kd, Vd, 0.5)
    O, LSE = orc.forward_gqa(Q, K, V, Kd, Vd, 0.5)
    np.testing.assert_allclose(o, O, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(lse, LSE, rtol=1e-12, atol=1e-13)
    o1, lse1 = orc.forward_prefill_gqa(Q[:, -1:], K, V, Kd[:, :, -1:], Vd[:, :, -1:], 0.5)
    od, lsed = orc.decode_gqa(Q[:, -1], K, V, Kd[:, :, -1], Vd[:, :, -1], 0.5)
    np.testing.assert_allclose(o1[:, 0], od, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(lse1[:, :, 0], lsed, rtol=1e-12, atol=1e-13)
    with pytest.raises(ValueError):
        orc.forward_prefill_gqa(Q, K[:, :5], V[:, :5], None, None, 1.0)
