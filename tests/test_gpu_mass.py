"""Attention mass on the depth slots (moda_depth_slot_mass) on the GPU against the fp64 oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import paper_2603_15619_b200 as moda
from paper_2603_15619_b200 import synthetic
from oracle import moda_oracle as orc

from parity import f64

pytestmark = pytest.mark.gpu

SHAPES = [
    # B, T, H, H_kv, d, l
    (1, 128, 1, 1, 64, 1), (2, 300, 3, 3, 128, 5), (1, 1000, 4, 2, 64, 7), (1, 129, 8, 1, 128, 3), (2, 257, 2, 2, 64, 33),
    (1, 1, 2, 1, 128, 2), (1, 640, 16, 2, 64, 70), (1, 2190, 4, 4, 128, 24),
]


@pytest.mark.parametrize("B,T,H,Hk,d,l", SHAPES)
def test_mass_matches_the_oracle_and_probability_is_conserved(B, T, H, Hk, d, l):
    scale = d ** -0.5
    x = synthetic.make_gqa(B, T, H, Hk, d, l, seed=23, device="cuda")
    cache = moda.alloc_depth_cache(B, T, Hk, d, l)
    for i in range(l):
        moda.moda_depth_cache_append(cache, i, x["Kd"][i].contiguous(), x["Vd"][i].contiguous())
    O, LSE = moda.moda_attn_fwd_gqa(x["Q"], x["K"], x["V"], cache, l, scale)
    guard = torch.full((B * H * l + 64,), 7.0, dtype=torch.float32, device="cuda")
    mass = guard[32:32 + B * H * l].view(B, H, l)
    out = moda.moda_depth_slot_mass(x["Q"], cache, LSE, l, scale, H_kv=Hk, mass=mass)
    assert moda.moda_last_status() == 0 and out.data_ptr() == mass.data_ptr()
    assert bool((guard[:32] == 7.0).all()) and bool((guard[-32:] == 7.0).all()), "guard band overwritten"
    # the oracle with the same LSE the kernel was given (fp32): what is compared is the mass arithmetic alone
    ref = orc.depth_slot_mass(f64(x["Q"]), f64(x["Kd"]), f64(LSE), scale)
    got = f64(mass)
    assert np.allclose(got, ref, rtol=2e-4, atol=1e-6), f"max rel err {np.abs(got / ref - 1).max():.2e}"
    # and with the oracle's own LSE: the GPU forward's LSE (abs error <= 1e-3) moves every mass by at most that factor
    _, LSE_ref = orc.forward_gqa(*[f64(x[k]) for k in ("Q", "K", "V", "Kd", "Vd")], scale)
    ref2 = orc.depth_slot_mass(f64(x["Q"]), f64(x["Kd"]), LSE_ref, scale)
    assert np.allclose(got, ref2, rtol=2e-3, atol=1e-6)
    # bit-reproducible
    again = moda.moda_depth_slot_mass(x["Q"], cache, LSE, l, scale, H_kv=Hk)
    assert torch.equal(again, mass)


def test_top_slots_by_mass_are_the_slots_that_matter():
    # two of five slots carry keys aligned with the queries: they collect almost all of the depth mass, which is the
    # utility that a bounded slot buffer ("keep the top S") ranks by
    B, T, H, d, l = 1, 512, 2, 64, 5
    g = torch.Generator(device="cuda").manual_seed(3)
    Q = torch.randn((B, T, H, d), device="cuda", generator=g).to(torch.bfloat16)
    K = torch.randn((B, T, H, d), device="cuda", generator=g).to(torch.bfloat16)
    V = torch.randn((B, T, H, d), device="cuda", generator=g).to(torch.bfloat16)
    Kd = (0.1 * torch.randn((l, B, T, H, d), device="cuda", generator=g)).to(torch.bfloat16)
    Vd = torch.randn((l, B, T, H, d), device="cuda", generator=g).to(torch.bfloat16)
    Kd[1] = Q
    Kd[3] = (0.8 * Q.float()).to(torch.bfloat16)
    cache = moda.alloc_depth_cache(B, T, H, d, l)
    for i in range(l):
        moda.moda_depth_cache_append(cache, i, Kd[i].contiguous(), Vd[i].contiguous())
    O, LSE = moda.moda_attn_fwd(Q, K, V, cache, l, d ** -0.5)
    mass = moda.moda_depth_slot_mass(Q, cache, LSE, l, d ** -0.5)
    top = set(mass.sum(dim=(0, 1)).topk(2).indices.tolist())
    assert top == {1, 3}
    assert float(mass[:, :, [1, 3]].sum()) > 0.9 * float(mass.sum())
    assert float(mass.sum()) < B * H * T


def test_bounded_slot_buffer_driven_by_the_mass_keeps_the_useful_layers():
    """Six layers through a buffer of four slots with the top-S policy: every layer attends to the layers the buffer
    holds (checked against the oracle on exactly those layers), writes its K, V over the slot of least attention mass,
    and the two layers whose keys the queries look for survive to the end."""
    from paper_2603_15619_b200.slots import SlotBuffer
    from parity import assert_forward_close
    B, T, H, d, S, n_layers = 1, 300, 2, 64, 4, 6
    scale = d ** -0.5
    g = torch.Generator(device="cuda").manual_seed(9)
    base = torch.randn((B, T, H, d), device="cuda", generator=g)
    layers = []
    for n in range(n_layers):
        Q = (base + 0.3 * torch.randn((B, T, H, d), device="cuda", generator=g)).to(torch.bfloat16)
        # layers 0 and 2 write keys that later queries align with; the others write small random keys
        K = (base if n in (0, 2) else 0.1 * torch.randn((B, T, H, d), device="cuda", generator=g)).to(torch.bfloat16)
        V = torch.randn((B, T, H, d), device="cuda", generator=g).to(torch.bfloat16)
        layers.append((Q, K, V))
    cache = moda.alloc_depth_cache(B, T, H, d, S)
    buf = SlotBuffer(S, policy="top")
    utility = None
    for n, (Q, K, V) in enumerate(layers):
        l = buf.filled
        held = list(buf.layers())                                   # slot order
        slot = buf.next_slot(utility)
        O, LSE = moda.moda_attn_fwd_append(Q, K, V, cache, l, scale, cache, slot)
        assert moda.moda_last_status() == 0
        Kd = np.stack([f64(layers[m][1]) for m in held]) if held else np.zeros((0, B, T, H, d))
        Vd = np.stack([f64(layers[m][2]) for m in held]) if held else np.zeros((0, B, T, H, d))
        assert_forward_close(O, LSE, *orc.forward(f64(Q), f64(K), f64(V), Kd, Vd, scale), f"layer {n} over layers {held}")
        # utility of the slots this layer read (the one just overwritten holds a new layer nobody has attended to yet)
        utility = [float("inf")] * S
        if l > 0:
            mass = moda.moda_depth_slot_mass(Q, cache, LSE, l, scale).sum(dim=(0, 1)).tolist()
            utility[:l] = mass
        utility[slot] = float("inf")
        buf.record(slot, n)
    # the newest layer is always kept (nobody has attended to it yet); of the rest, the low-mass layers 1 and 3 went
    assert sorted(buf.layers()) == [0, 2, 4, 5]
