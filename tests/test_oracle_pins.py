"""Pins of the fp64 oracle against things other than itself (CPU only).

The MoDA operator is exactly defined (paper Sec. 2.2: one softmax over the causal
sequence keys and the same-position depth keys), so each pin below is a value fixed by
the mathematics or by a library routine on a special case:

  P1  masked library attention over the flattened key set [T sequence | T*l depth] with
      the masks of Alg. 1 (causal j <= i; depth floor(j_d / L) == i), plus a per-row
      explicit-softmax brute force
  P2  l = 0 reduces to library causal attention
  P3  O = w O_seq + (1-w) O_dep, LSE = logaddexp(LSE_seq, LSE_dep): a single softmax over
      the union, not a sum of two softmaxes
  P4  closed forms: zero queries (uniform weights over t+1+l keys), T = 1 (pure depth
      attention over l+1 keys), one dominating key
  P5  invariances: depth-slot permutation, common key shift, position locality
  P6  gradients against central finite differences and against library autograd
  P7  gradient sum identities
"""
import numpy as np
import pytest
import torch
import torch.nn.functional as F
from scipy.special import logsumexp, softmax

from oracle import moda_oracle as orc


def rand_inputs(rng, B, T, H, d, l, amp=1.0):
    Q = rng.standard_normal((B, T, H, d)) * amp
    K = rng.standard_normal((B, T, H, d)) * amp
    V = rng.standard_normal((B, T, H, d))
    Kd = rng.standard_normal((l, B, T, H, d)) * amp
    Vd = rng.standard_normal((l, B, T, H, d))
    dO = rng.standard_normal((B, T, H, d))
    return Q, K, V, Kd, Vd, dO


def flattened_masked_attention(Q, K, V, Kd, Vd, scale):
    """Library attention over [sequence keys | flattened depth keys] (torch, float64).

    Depth column j_d = t*l + i holds slot i of position t; mask as in Alg. 1."""
    B, T, H, d = Q.shape
    l = Kd.shape[0]
    q = Q.permute(0, 2, 1, 3)                                   # [B,H,T,d]
    kf = torch.cat([K.permute(0, 2, 1, 3), Kd.permute(1, 3, 2, 0, 4).reshape(B, H, T * l, d)], dim=2)
    vf = torch.cat([V.permute(0, 2, 1, 3), Vd.permute(1, 3, 2, 0, 4).reshape(B, H, T * l, d)], dim=2)
    iq = torch.arange(T)[:, None]
    causal = torch.arange(T)[None, :] <= iq
    depth = (torch.arange(T * l)[None, :] // max(l, 1)) == iq
    mask = torch.cat([causal, depth], dim=1)
    o = F.scaled_dot_product_attention(q, kf, vf, attn_mask=mask, scale=scale)
    s = (q @ kf.transpose(-1, -2)) * scale
    lse = torch.logsumexp(s.masked_fill(~mask, float("-inf")), dim=-1)  # [B,H,T]
    return o.permute(0, 2, 1, 3), lse


@pytest.mark.parametrize("B,T,H,d,l", [(1, 1, 1, 4, 3), (2, 7, 2, 8, 4), (1, 16, 2, 8, 1), (1, 33, 1, 16, 5)])
def test_p1_flattened_masked_library_attention(B, T, H, d, l):
    rng = np.random.default_rng(10 + T)
    Q, K, V, Kd, Vd, _ = rand_inputs(rng, B, T, H, d, l)
    scale = 0.37
    O, LSE = orc.forward(Q, K, V, Kd, Vd, scale)
    o_ref, lse_ref = flattened_masked_attention(*(torch.from_numpy(x) for x in (Q, K, V, Kd, Vd)), scale)
    np.testing.assert_allclose(O, o_ref.numpy(), rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(LSE, lse_ref.numpy(), rtol=1e-12, atol=1e-12)


def test_p1_bruteforce_explicit_softmax_per_row():
    rng = np.random.default_rng(1)
    B, T, H, d, l = 2, 9, 2, 5, 3
    Q, K, V, Kd, Vd, _ = rand_inputs(rng, B, T, H, d, l)
    scale = 1.0 / np.sqrt(d)
    O, LSE = orc.forward(Q, K, V, Kd, Vd, scale)
    for b in range(B):
        for h in range(H):
            for t in range(T):
                keys = np.concatenate([K[b, : t + 1, h], Kd[:, b, t, h]], axis=0)
                vals = np.concatenate([V[b, : t + 1, h], Vd[:, b, t, h]], axis=0)
                logits = keys @ Q[b, t, h] * scale
                w = softmax(logits)
                assert w.shape == (t + 1 + l,)
                np.testing.assert_allclose(O[b, t, h], w @ vals, rtol=1e-12, atol=1e-13)
                np.testing.assert_allclose(LSE[b, h, t], logsumexp(logits), rtol=1e-12)


def test_p1_forward_rows_matches_full():
    rng = np.random.default_rng(2)
    Q, K, V, Kd, Vd, _ = rand_inputs(rng, 2, 12, 3, 4, 2)
    O, LSE = orc.forward(Q, K, V, Kd, Vd, 0.5)
    rows = np.array([[0, 0, 0], [1, 2, 11], [0, 1, 5], [1, 0, 7]], dtype=np.int32)
    o_r, lse_r = orc.forward_rows(Q, K, V, Kd, Vd, 0.5, rows)
    for n, (b, h, t) in enumerate(rows):
        np.testing.assert_array_equal(o_r[n], O[b, t, h])
        assert lse_r[n] == LSE[b, h, t]


@pytest.mark.parametrize("T,d", [(1, 4), (5, 8), (40, 16)])
def test_p2_l0_is_causal_attention(T, d):
    rng = np.random.default_rng(20 + T)
    B, H = 2, 3
    Q, K, V, _, _, dO = rand_inputs(rng, B, T, H, d, 0)
    scale = 1.0 / np.sqrt(d)
    O, LSE = orc.forward(Q, K, V, None, None, scale)
    tq, tk, tv = (torch.from_numpy(x).permute(0, 2, 1, 3).requires_grad_(True) for x in (Q, K, V))
    o_ref = F.scaled_dot_product_attention(tq, tk, tv, is_causal=True)     # default scale 1/sqrt(d)
    np.testing.assert_allclose(O, o_ref.detach().permute(0, 2, 1, 3).numpy(), rtol=1e-12, atol=1e-12)
    # textbook LSE
    s = np.einsum("bthd,bshd->bhts", Q, K) * scale
    s = np.where(np.tril(np.ones((T, T), bool)), s, -np.inf)
    np.testing.assert_allclose(LSE, logsumexp(s, axis=-1), rtol=1e-12)
    # gradients of the l = 0 case against library autograd
    o_ref.backward(torch.from_numpy(dO).permute(0, 2, 1, 3))
    dQ, dK, dV, dKd, dVd = orc.backward(Q, K, V, None, None, dO, scale)
    assert dKd.shape == (0, B, T, H, d) and dVd.shape == (0, B, T, H, d)
    for got, ref in ((dQ, tq.grad), (dK, tk.grad), (dV, tv.grad)):
        np.testing.assert_allclose(got, ref.permute(0, 2, 1, 3).numpy(), rtol=1e-10, atol=1e-12)


def test_p3_union_softmax_decomposition():
    rng = np.random.default_rng(3)
    B, T, H, d, l = 2, 11, 2, 8, 4
    Q, K, V, Kd, Vd, _ = rand_inputs(rng, B, T, H, d, l)
    scale = 0.4
    O, LSE = orc.forward(Q, K, V, Kd, Vd, scale)
    tq, tk, tv = (torch.from_numpy(x).permute(0, 2, 1, 3) for x in (Q, K, V))
    o_seq = F.scaled_dot_product_attention(tq, tk, tv, is_causal=True, scale=scale).permute(0, 2, 1, 3).numpy()
    s = np.einsum("bthd,bshd->bhts", Q, K) * scale
    lse_seq = logsumexp(np.where(np.tril(np.ones((T, T), bool)), s, -np.inf), axis=-1)   # [B,H,T]
    # depth attention: every (b,t,h) query over its own l depth keys (library SDPA, batch = B*T*H)
    qd = torch.from_numpy(Q).reshape(B * T * H, 1, 1, d)
    kd = torch.from_numpy(Kd).permute(1, 2, 3, 0, 4).reshape(B * T * H, 1, l, d)
    vd = torch.from_numpy(Vd).permute(1, 2, 3, 0, 4).reshape(B * T * H, 1, l, d)
    o_dep = F.scaled_dot_product_attention(qd, kd, vd, scale=scale).reshape(B, T, H, d).numpy()
    u = np.einsum("bthd,lbthd->bhtl", Q, Kd) * scale
    lse_dep = logsumexp(u, axis=-1)                                                         # [B,H,T]
    np.testing.assert_allclose(LSE, np.logaddexp(lse_seq, lse_dep), rtol=1e-12)
    w = np.exp(lse_seq - LSE).transpose(0, 2, 1)[..., None]                                 # [B,T,H,1]
    np.testing.assert_allclose(O, w * o_seq + (1 - w) * o_dep, rtol=1e-11, atol=1e-12)
    # the two-separate-softmaxes reading must NOT pass (guards the pin itself)
    assert np.abs(O - 0.5 * (o_seq + o_dep)).max() > 1e-3


def test_p4_closed_form_zero_queries_uniform_weights():
    rng = np.random.default_rng(4)
    B, T, H, d, l = 1, 10, 2, 6, 3
    _, K, V, Kd, Vd, _ = rand_inputs(rng, B, T, H, d, l)
    Q = np.zeros((B, T, H, d))
    O, LSE = orc.forward(Q, K, V, Kd, Vd, 1.0)
    for t in range(T):
        n = t + 1 + l
        np.testing.assert_allclose(LSE[:, :, t], np.log(n), rtol=1e-14)
        expect = (V[:, : t + 1].sum(axis=1) + Vd[:, :, t].sum(axis=0)) / n
        np.testing.assert_allclose(O[:, t], expect, rtol=1e-13, atol=1e-14)


def test_p4_t1_is_depth_attention_over_l_plus_1_keys():
    rng = np.random.default_rng(5)
    B, T, H, d, l = 3, 1, 2, 8, 6
    Q, K, V, Kd, Vd, _ = rand_inputs(rng, B, T, H, d, l)
    O, LSE = orc.forward(Q, K, V, Kd, Vd, 0.3)
    keys = np.concatenate([K[None], Kd], axis=0)[:, :, 0]      # [l+1,B,H,d]
    vals = np.concatenate([V[None], Vd], axis=0)[:, :, 0]
    logits = np.einsum("bhd,nbhd->bhn", Q[:, 0], keys) * 0.3
    w = softmax(logits, axis=-1)
    np.testing.assert_allclose(O[:, 0], np.einsum("bhn,nbhd->bhd", w, vals), rtol=1e-12)
    np.testing.assert_allclose(LSE[:, :, 0], logsumexp(logits, axis=-1), rtol=1e-13)


def test_p4_dominating_key_selects_its_value():
    rng = np.random.default_rng(6)
    B, T, H, d, l = 1, 6, 1, 4, 3
    Q, K, V, Kd, Vd, _ = rand_inputs(rng, B, T, H, d, l)
    # depth slot 1 at position 4 is aligned with the query and huge; sequence key 2 for query 5
    Kd[1, 0, 4, 0] = 200.0 * Q[0, 4, 0]
    K[0, 2, 0] = 200.0 * Q[0, 5, 0]
    O, _ = orc.forward(Q, K, V, Kd, Vd, 1.0)
    np.testing.assert_allclose(O[0, 4, 0], Vd[1, 0, 4, 0], atol=1e-9)
    np.testing.assert_allclose(O[0, 5, 0], V[0, 2, 0], atol=1e-9)
    # the causal mask is strict about the future: query 1 cannot see sequence key 2
    assert np.abs(O[0, 1, 0] - V[0, 2, 0]).max() > 1e-3


def test_p5_depth_slot_permutation_invariance():
    rng = np.random.default_rng(7)
    B, T, H, d, l = 2, 8, 2, 8, 5
    Q, K, V, Kd, Vd, dO = rand_inputs(rng, B, T, H, d, l)
    perm = rng.permutation(l)
    O, LSE = orc.forward(Q, K, V, Kd, Vd, 0.35)
    O2, LSE2 = orc.forward(Q, K, V, Kd[perm], Vd[perm], 0.35)
    np.testing.assert_allclose(O2, O, rtol=1e-13, atol=1e-14)
    np.testing.assert_allclose(LSE2, LSE, rtol=1e-14)
    g = orc.backward(Q, K, V, Kd, Vd, dO, 0.35)
    g2 = orc.backward(Q, K, V, Kd[perm], Vd[perm], dO, 0.35)
    for a, b in zip(g[:3], g2[:3]):
        np.testing.assert_allclose(b, a, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(g2[3], g[3][perm], rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(g2[4], g[4][perm], rtol=1e-12, atol=1e-14)


def test_p5_common_key_shift_and_position_locality():
    rng = np.random.default_rng(8)
    B, T, H, d, l = 1, 9, 2, 6, 3
    Q, K, V, Kd, Vd, _ = rand_inputs(rng, B, T, H, d, l)
    scale = 0.45
    O, LSE = orc.forward(Q, K, V, Kd, Vd, scale)
    c = rng.standard_normal(d)
    O2, LSE2 = orc.forward(Q, K + c, V, Kd + c, Vd, scale)
    np.testing.assert_allclose(O2, O, rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(LSE2 - LSE, scale * np.einsum("bthd,d->bht", Q, c), rtol=1e-11, atol=1e-12)
    # shifting only the sequence keys is NOT invariant (depth keys share the softmax)
    O3, _ = orc.forward(Q, K + c, V, Kd, Vd, scale)
    assert np.abs(O3 - O).max() > 1e-3
    # depth rows are position-local: swapping the depth rows of positions 2 and 6 changes only rows 2, 6
    Kd4, Vd4 = Kd.copy(), Vd.copy()
    Kd4[:, :, [2, 6]] = Kd[:, :, [6, 2]]
    Vd4[:, :, [2, 6]] = Vd[:, :, [6, 2]]
    O4, _ = orc.forward(Q, K, V, Kd4, Vd4, scale)
    changed = np.abs(O4 - O).max(axis=(0, 2, 3)) > 1e-9
    assert changed.tolist() == [t in (2, 6) for t in range(T)]


def _loss(Q, K, V, Kd, Vd, dO, scale):
    O, _ = orc.forward(Q, K, V, Kd, Vd, scale)
    return float((O * dO).sum())


def test_p6_gradients_match_finite_differences():
    rng = np.random.default_rng(9)
    B, T, H, d, l = 1, 5, 2, 3, 2
    ins = list(rand_inputs(rng, B, T, H, d, l))
    scale = 0.6
    dO = ins[5]
    grads = orc.backward(*ins[:5], dO, scale)
    eps = 1e-6
    for which, g in enumerate(grads):
        x = ins[which]
        num = np.zeros_like(x)
        it = np.nditer(x, flags=["multi_index"])
        for _ in it:
            i = it.multi_index
            old = x[i]
            x[i] = old + eps
            lp = _loss(*ins[:5], dO, scale)
            x[i] = old - eps
            lm = _loss(*ins[:5], dO, scale)
            x[i] = old
            num[i] = (lp - lm) / (2 * eps)
        err = np.abs(num - g).max() / max(np.abs(g).max(), 1e-30)
        assert err < 1e-6, (which, err)


@pytest.mark.parametrize("B,T,H,d,l", [(2, 6, 2, 4, 3), (1, 17, 1, 8, 1)])
def test_p6_gradients_match_library_autograd(B, T, H, d, l):
    rng = np.random.default_rng(11)
    Q, K, V, Kd, Vd, dO = rand_inputs(rng, B, T, H, d, l)
    scale = 0.5
    ts = [torch.from_numpy(x).clone().requires_grad_(True) for x in (Q, K, V, Kd, Vd)]
    o, _ = flattened_masked_attention(*ts, scale)
    o.backward(torch.from_numpy(dO))
    grads = orc.backward(Q, K, V, Kd, Vd, dO, scale)
    for got, t in zip(grads, ts):
        np.testing.assert_allclose(got, t.grad.numpy(), rtol=1e-10, atol=1e-12)


def test_p7_gradient_sum_identities():
    rng = np.random.default_rng(12)
    B, T, H, d, l = 2, 13, 2, 8, 4
    Q, K, V, Kd, Vd, dO = rand_inputs(rng, B, T, H, d, l)
    dQ, dK, dV, dKd, dVd = orc.backward(Q, K, V, Kd, Vd, dO, 0.3)
    # sum_j p_j + sum_i r_i = 1  =>  total value-gradient mass equals total dO mass
    np.testing.assert_allclose(dV.sum(axis=1) + dVd.sum(axis=(0, 2)), dO.sum(axis=1), rtol=1e-11, atol=1e-12)
    # sum_j ds_j + sum_i du_i = 0 per row  =>  with all queries equal, key gradients sum to zero
    Qc = np.broadcast_to(Q[:, :1], Q.shape).copy()
    _, dK2, _, dKd2, _ = orc.backward(Qc, K, V, Kd, Vd, dO, 0.3)
    np.testing.assert_allclose(dK2.sum(axis=1) + dKd2.sum(axis=(0, 2)), 0.0, atol=1e-11)


def test_p6_sampled_row_backward_matches_library_autograd_and_full_backward():
    rng = np.random.default_rng(13)
    B, T, H, d, l = 2, 19, 2, 4, 3
    Q, K, V, Kd, Vd, dO = rand_inputs(rng, B, T, H, d, l)
    scale = 0.55
    ts = [torch.from_numpy(x).clone().requires_grad_(True) for x in (Q, K, V, Kd, Vd)]
    o, _ = flattened_masked_attention(*ts, scale)
    o.backward(torch.from_numpy(dO))
    gQ, gK, gV, gKd, gVd = (t.grad.numpy() for t in ts)
    qrows = np.array([[0, 0, 0], [1, 1, 18], [0, 1, 7], [1, 0, 12]], dtype=np.int32)
    krows = np.array([[0, 0, 11], [1, 1, 18], [0, 1, 15], [0, 0, 13]], dtype=np.int32)
    dQ, dKd, dVd, dK, dV = orc.backward_rows(Q, K, V, Kd, Vd, dO, scale, qrows, krows, t_start=11)
    for n, (b, h, t) in enumerate(qrows):
        np.testing.assert_allclose(dQ[n], gQ[b, t, h], rtol=1e-10, atol=1e-12)
        np.testing.assert_allclose(dKd[n], gKd[:, b, t, h], rtol=1e-10, atol=1e-12)
        np.testing.assert_allclose(dVd[n], gVd[:, b, t, h], rtol=1e-10, atol=1e-12)
    for n, (b, h, j) in enumerate(krows):
        np.testing.assert_allclose(dK[n], gK[b, j, h], rtol=1e-10, atol=1e-12)
        np.testing.assert_allclose(dV[n], gV[b, j, h], rtol=1e-10, atol=1e-12)
    full = orc.backward(Q, K, V, Kd, Vd, dO, scale)
    np.testing.assert_allclose(dQ[1], full[0][1, 18, 1], rtol=1e-12, atol=1e-14)
    with pytest.raises(ValueError):
        orc.backward_rows(Q, K, V, Kd, Vd, dO, scale, qrows, krows, t_start=12)
