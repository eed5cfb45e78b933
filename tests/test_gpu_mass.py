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
