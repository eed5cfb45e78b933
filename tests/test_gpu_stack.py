"""A stack of MoDA layers through DepthStream: every layer's K, V gradient = its own sequence-attention
gradient + the depth gradients that all later layers send to its slot (checked against the oracle)."""
import numpy as np
import pytest
import torch

import paper_2603_15619_b200 as moda
from paper_2603_15619_b200 import synthetic
from oracle import moda_oracle as orc

from parity import TOL_GRAD_REL_L2, TOL_O_REL_L2, assert_same_gradients, f64, rel_l2

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("B,T,H,Hk,d,n_layers", [(1, 300, 2, 2, 64, 4), (1, 256, 4, 2, 128, 3)])
def test_stack_gradients_flow_back_through_the_depth_stream(B, T, H, Hk, d, n_layers):
    scale = d ** -0.5
    layers = []
    for i in range(n_layers):
        x = synthetic.make_gqa(B, T, H, Hk, d, 0, seed=40 + i, device="cuda")
        layers.append({k: x[k].clone().requires_grad_(k != "dO") for k in ("Q", "K", "V", "dO")})
    stream = moda.DepthStream(B, T, Hk, d, n_layers)
    loss = 0.0
    outs = []
    for L in layers:
        O = stream.attend(L["Q"], L["K"], L["V"], scale)
        outs.append(O)
        loss = loss + (O.float() * L["dO"].float()).sum()
    loss.backward()
    assert moda.moda_last_status() == 0

    # oracle: layer l sees slots 0..l-1 = K, V of the earlier layers
    dK_ref = [np.zeros((B, T, Hk, d)) for _ in range(n_layers)]
    dV_ref = [np.zeros((B, T, Hk, d)) for _ in range(n_layers)]
    for l, L in enumerate(layers):
        Kd = np.stack([f64(layers[i]["K"]) for i in range(l)]) if l else np.zeros((0, B, T, Hk, d))
        Vd = np.stack([f64(layers[i]["V"]) for i in range(l)]) if l else np.zeros((0, B, T, Hk, d))
        args = (f64(L["Q"]), f64(L["K"]), f64(L["V"]), Kd, Vd)
        O_ref, _ = orc.forward_gqa(*args, scale)
        assert rel_l2(f64(outs[l]), O_ref) <= TOL_O_REL_L2
        dQ, dK, dV, dKd, dVd = orc.backward_gqa(*args, f64(L["dO"]), scale)
        assert rel_l2(f64(L["Q"].grad), dQ) <= TOL_GRAD_REL_L2, f"dQ of layer {l}"
        dK_ref[l] += dK
        dV_ref[l] += dV
        for i in range(l):
            dK_ref[i] += dKd[i]
            dV_ref[i] += dVd[i]
    for l, L in enumerate(layers):
        assert rel_l2(f64(L["K"].grad), dK_ref[l]) <= TOL_GRAD_REL_L2, f"dK of layer {l}"
        assert rel_l2(f64(L["V"].grad), dV_ref[l]) <= TOL_GRAD_REL_L2, f"dV of layer {l}"


@pytest.mark.parametrize("B,T,H,Hk,d,l", [(1, 300, 2, 2, 64, 3), (2, 200, 3, 3, 128, 5), (1, 300, 4, 2, 64, 4),
                                          (1, 256, 16, 1, 128, 3), (1, 130, 32, 1, 64, 2),
                                          # large groups: the per-position depth kernel does the adding (16 heads: two launches)
                                          (1, 200, 8, 1, 64, 12), (2, 130, 16, 1, 64, 9), (1, 100, 8, 1, 128, 10)])
def test_accumulate_flag_adds_the_depth_gradients_to_what_the_cache_holds(B, T, H, Hk, d, l):
    """MODA_BWD_ACCUMULATE_DEPTH: slots [0, l) become bf16(old + gradient), everything else as without the flag."""
    x = synthetic.make_gqa(B, T, H, Hk, d, l, seed=77, device="cuda")
    scale = d ** -0.5
    cache = moda.alloc_depth_cache(B, T, Hk, d, l)
    for i in range(l):
        moda.moda_depth_cache_append(cache, i, x["Kd"][i].contiguous(), x["Vd"][i].contiguous())
    O, LSE = moda.moda_attn_fwd_gqa(x["Q"], x["K"], x["V"], cache, l, scale)
    plain = moda.moda_attn_bwd_gqa(x["Q"], x["K"], x["V"], cache, O, x["dO"], LSE, l, scale)
    g = torch.Generator(device="cuda").manual_seed(5)
    old = (torch.randn(plain[3].shape, generator=g, device="cuda") * plain[3].float().std()).to(torch.bfloat16)
    acc = old.clone()
    out = moda.moda_attn_bwd_gqa(x["Q"], x["K"], x["V"], cache, O, x["dO"], LSE, l, scale, d_depth_kv=acc,
                                 stages=moda.MODA_BWD_ALL_STAGES | moda.MODA_BWD_ACCUMULATE_DEPTH)
    assert moda.moda_last_status() == 0
    assert_same_gradients(out[:3], plain[:3], "with and without the accumulate flag")
    want = (old.double() + plain[3].double())
    got = acc.double()
    if H // Hk <= 8:
        ulp = torch.maximum(want.abs(), torch.tensor(1e-30, device="cuda", dtype=torch.float64)) * 2.0 ** -8
        assert bool(((got - want).abs() <= ulp).all())                       # one bf16 rounding of the exact sum
        assert float((got != want.to(torch.bfloat16).double()).double().mean()) < 1e-3   # and round-to-nearest almost everywhere
    else:
        # 16 / 32 heads per group: the groups of 8 add their shares one after the other (a rounding each),
        # while the plain call rounds the sum of the shares once
        # (the shares of the groups may be larger than their sum, so the bound is on the whole tensor)
        assert rel_l2(got.cpu().numpy(), want.cpu().numpy()) < 5e-3
    # twice more: the cache keeps collecting
    moda.moda_attn_bwd_gqa(x["Q"], x["K"], x["V"], cache, O, x["dO"], LSE, l, scale, d_depth_kv=acc,
                           stages=moda.MODA_BWD_ALL_STAGES | moda.MODA_BWD_ACCUMULATE_DEPTH)
    want2 = old.double() + 2 * plain[3].double()
    assert rel_l2(acc.double().cpu().numpy(), want2.cpu().numpy()) < 1e-2


def test_slot_written_without_attending_gets_the_gradients_of_the_layers_after_it():
    B, T, H, Hk, d = 1, 200, 4, 2, 64
    scale = d ** -0.5
    a = synthetic.make_gqa(B, T, H, Hk, d, 0, seed=3, device="cuda")
    f = synthetic.make_gqa(B, T, H, Hk, d, 0, seed=4, device="cuda")
    Kf, Vf = f["K"].clone().requires_grad_(), f["V"].clone().requires_grad_()
    Q, K, V = (a[k].clone().requires_grad_() for k in ("Q", "K", "V"))
    stream = moda.DepthStream(B, T, Hk, d, 2)
    stream.write(Kf, Vf)                                   # slot 0
    O = stream.attend(Q, K, V, scale)                      # attends to slot 0, writes slot 1
    (O.float() * a["dO"].float()).sum().backward()
    Kd, Vd = f64(Kf)[None], f64(Vf)[None]
    dQ, dK, dV, dKd, dVd = orc.backward_gqa(f64(Q), f64(K), f64(V), Kd, Vd, f64(a["dO"]), scale)
    for got, want in ((Q.grad, dQ), (K.grad, dK), (V.grad, dV), (Kf.grad, dKd[0]), (Vf.grad, dVd[0])):
        assert rel_l2(f64(got), want) <= TOL_GRAD_REL_L2


@pytest.mark.parametrize("B,T,H,Hk,d,Dm", [(1, 200, 4, 2, 64, 128), (2, 300, 2, 2, 128, 192)])
def test_slot_projected_from_a_layer_input_sends_its_gradient_to_the_input_and_the_weights(B, T, H, Hk, d, Dm):
    """FFN-side depth pair: slot 0 = projection of X (written by the projection's epilogue), then an attention layer.
    The oracle's slot gradients, pulled back through the fp64 projection, are the gradients of X, Wk, Wv."""
    scale = d ** -0.5
    a = synthetic.make_gqa(B, T, H, Hk, d, 0, seed=7, device="cuda")
    g = torch.Generator(device="cuda").manual_seed(8)
    X = torch.randn((B, T, Dm), device="cuda", generator=g).to(torch.bfloat16).requires_grad_()
    Wk = (torch.randn((Hk * d, Dm), device="cuda", generator=g) * Dm ** -0.5).to(torch.bfloat16).requires_grad_()
    Wv = (torch.randn((Hk * d, Dm), device="cuda", generator=g) * Dm ** -0.5).to(torch.bfloat16).requires_grad_()
    Q, K, V = (a[k].clone().requires_grad_() for k in ("Q", "K", "V"))
    stream = moda.DepthStream(B, T, Hk, d, 2)
    stream.project_write(X, Wk, Wv)                        # slot 0
    O = stream.attend(Q, K, V, scale)                      # attends to slot 0, writes slot 1
    (O.float() * a["dO"].float()).sum().backward()
    assert moda.moda_last_status() == 0
    # the operator sees the slot as stored (rounded to bf16); the oracle gets exactly those values
    Ks, Vs = torch.empty((B, T, Hk, d), dtype=torch.bfloat16, device="cuda"), torch.empty((B, T, Hk, d), dtype=torch.bfloat16, device="cuda")
    moda.moda_depth_cache_unpack(stream.cache, 0, Ks, Vs)
    K_ref, V_ref = orc.project_kv(f64(X), f64(Wk), f64(Wv), Hk)
    assert rel_l2(f64(Ks), K_ref) <= TOL_O_REL_L2 and rel_l2(f64(Vs), V_ref) <= TOL_O_REL_L2
    O_ref, _ = orc.forward_gqa(f64(Q), f64(K), f64(V), f64(Ks)[None], f64(Vs)[None], scale)
    assert rel_l2(f64(O), O_ref) <= TOL_O_REL_L2
    dQ, dK, dV, dKd, dVd = orc.backward_gqa(f64(Q), f64(K), f64(V), f64(Ks)[None], f64(Vs)[None], f64(a["dO"]), scale)
    gk, gv = dKd[0].reshape(B * T, Hk * d), dVd[0].reshape(B * T, Hk * d)
    x2 = f64(X).reshape(B * T, Dm)
    dX_ref = (gk @ f64(Wk) + gv @ f64(Wv)).reshape(B, T, Dm)
    for got, want, name in ((Q.grad, dQ, "dQ"), (K.grad, dK, "dK"), (V.grad, dV, "dV"), (X.grad, dX_ref, "dX"),
                            (Wk.grad, gk.T @ x2, "dWk"), (Wv.grad, gv.T @ x2, "dWv")):
        assert rel_l2(f64(got), want) <= TOL_GRAD_REL_L2, f"{name}: {rel_l2(f64(got), want):.3e}"


@pytest.mark.parametrize("B,T,H,Hk,d,l,S", [(1, 300, 2, 2, 64, 7, 3), (1, 200, 4, 2, 128, 6, 2)])
def test_window_of_the_last_slots_is_the_operator_on_those_slots(B, T, H, Hk, d, l, S):
    """Bounded depth slots: a layer that attends only to the last S of l stored slots, forward and backward."""
    x = synthetic.make_gqa(B, T, H, Hk, d, l, seed=13, device="cuda")
    scale = d ** -0.5
    cache = moda.alloc_depth_cache(B, T, Hk, d, l)
    for i in range(l):
        moda.moda_depth_cache_append(cache, i, x["Kd"][i].contiguous(), x["Vd"][i].contiguous())
    win = moda.depth_cache_window(cache, B, T, Hk, d, l - S, S)
    O, LSE = moda.moda_attn_fwd_gqa(x["Q"], x["K"], x["V"], win, S, scale)
    gcache = torch.zeros_like(cache)
    gwin = moda.depth_cache_window(gcache, B, T, Hk, d, l - S, S)
    dQ, dK, dV, _ = moda.moda_attn_bwd_gqa(x["Q"], x["K"], x["V"], win, O, x["dO"], LSE, S, scale, d_depth_kv=gwin)
    assert moda.moda_last_status() == 0
    args = (f64(x["Q"]), f64(x["K"]), f64(x["V"]), f64(x["Kd"][l - S:]), f64(x["Vd"][l - S:]))
    O_ref, LSE_ref = orc.forward_gqa(*args, scale)
    refs = orc.backward_gqa(*args, f64(x["dO"]), scale)
    assert rel_l2(f64(O), O_ref) <= TOL_O_REL_L2 and np.abs(f64(LSE) - LSE_ref).max() <= 1e-3
    dKd = torch.empty_like(x["Kd"]); dVd = torch.empty_like(x["Vd"])
    for i in range(l):
        moda.moda_depth_cache_unpack(gcache, i, dKd[i], dVd[i])
    assert float(dKd[:l - S].abs().max()) == 0.0 and float(dVd[:l - S].abs().max()) == 0.0     # slots outside the window untouched
    for got, want in ((dQ, refs[0]), (dK, refs[1]), (dV, refs[2]), (dKd[l - S:], refs[3]), (dVd[l - S:], refs[4])):
        assert rel_l2(f64(got), want) <= TOL_GRAD_REL_L2
