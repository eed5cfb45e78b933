"""Position-major depth cache for grouped-query calls: layout round trip bit for bit, and forward / backward
parity against the fp64 oracle (GPU, through the C ABI)."""
import numpy as np
import pytest
import torch

import paper_2603_15619_b200 as moda
from paper_2603_15619_b200 import synthetic
from oracle import moda_oracle as orc

from parity import TOL_GRAD_REL_L2, TOL_GRAD_ROW_REL_L2, assert_forward_close, build_cache, f64, unpack_cache, worst_row_rel_l2
from test_gpu_gqa import grad_err

pytestmark = pytest.mark.gpu


def build_cache_pm(Kd, Vd):
    l, B, T, H, d = Kd.shape
    cache = moda.alloc_depth_cache(B, T, H, d, max(l, 1), Kd.device)
    cache.fill_(7.0)                                        # every element of slots < l must be overwritten
    for i in range(l):
        moda.moda_depth_cache_append_pm(cache, i, Kd[i].contiguous(), Vd[i].contiguous())
    return cache


def unpack_cache_pm(cache, l, B, T, H, d):
    Kd = torch.empty((l, B, T, H, d), dtype=torch.bfloat16, device=cache.device)
    Vd = torch.empty_like(Kd)
    for i in range(l):
        moda.moda_depth_cache_unpack_pm(cache, i, Kd[i], Vd[i])
    return Kd, Vd


@pytest.mark.parametrize("B,T,H,d,l", [(1, 128, 1, 64, 1), (2, 300, 3, 128, 2), (1, 1000, 2, 64, 3), (1, 1, 2, 128, 1)])
def test_layout_is_position_major_and_round_trips(B, T, H, d, l):
    g = torch.Generator(device="cuda").manual_seed(4)
    Kd = torch.randn((l, B, T, H, d), device="cuda", generator=g).to(torch.bfloat16)
    Vd = torch.randn((l, B, T, H, d), device="cuda", generator=g).to(torch.bfloat16)
    cache = build_cache_pm(Kd, Vd)
    Tp = (T + 127) // 128 * 128
    c = cache[: l * B * H * Tp * 2 * d].view(l, B, H, Tp, 2, d)
    assert torch.equal(c[:, :, :, :T, 0], Kd.permute(0, 1, 3, 2, 4)), "K rows are not where the layout says"
    assert torch.equal(c[:, :, :, :T, 1], Vd.permute(0, 1, 3, 2, 4)), "V rows are not where the layout says"
    assert bool((c[:, :, :, T:] == 0).all()), "tail rows must be zero"
    Kb, Vb = unpack_cache_pm(cache, l, B, T, H, d)
    assert torch.equal(Kb, Kd) and torch.equal(Vb, Vd)


SHAPES = [
    # B, T, H, H_kv, d, l
    (1, 256, 4, 2, 64, 4), (2, 300, 4, 1, 64, 3), (1, 384, 8, 2, 128, 5), (2, 129, 2, 1, 128, 2),
    (1, 640, 6, 3, 128, 17), (1, 1, 2, 1, 64, 2), (1, 300, 8, 1, 64, 64), (1, 77, 14, 2, 64, 47),
    (1, 200, 16, 1, 64, 40), (1, 130, 32, 1, 64, 33), (1, 140, 32, 2, 128, 12), (1, 150, 8, 1, 128, 50),
    (1, 200, 4, 2, 64, 0),
]


@pytest.mark.parametrize("B,T,H,Hk,d,l", SHAPES)
def test_forward_and_backward_match_the_oracle_and_the_row_interleaved_path(B, T, H, Hk, d, l):
    scale = d ** -0.5
    x = synthetic.make_gqa(B, T, H, Hk, d, l, seed=37, device="cuda")
    cache = build_cache_pm(x["Kd"], x["Vd"]) if l > 0 else None
    O, LSE = moda.moda_attn_fwd_gqa_pm(x["Q"], x["K"], x["V"], cache, l, scale)
    assert moda.moda_last_status() == 0
    xs = [f64(x[n]) for n in ("Q", "K", "V", "Kd", "Vd")]
    O_ref, LSE_ref = orc.forward_gqa(*xs, scale)
    assert_forward_close(O, LSE, O_ref, LSE_ref, f"pm {(B, T, H, Hk, d, l)}")

    dcache = None
    if l > 0:
        dcache = moda.alloc_depth_cache(B, T, Hk, d, l)
        dcache.fill_(5.0)
    dQ, dK, dV = torch.full_like(x["Q"], 3.0), torch.full_like(x["K"], 3.0), torch.full_like(x["V"], 3.0)
    moda.moda_attn_bwd_gqa_pm(x["Q"], x["K"], x["V"], cache, O, x["dO"], LSE, l, scale, dQ=dQ, dK=dK, dV=dV, d_depth_kv_pm=dcache)
    assert moda.moda_last_status() == 0
    if l > 0:
        dKd, dVd = unpack_cache_pm(dcache, l, B, T, Hk, d)
        Tp = (T + 127) // 128 * 128
        c = dcache[: l * B * Hk * Tp * 2 * d].view(l, B, Hk, Tp, 2, d)
        assert bool((c[:, :, :, T:] == 0).all()), "tail rows of the depth gradients must be zero"
    else:
        dKd = dVd = torch.zeros((0, B, T, Hk, d), dtype=torch.bfloat16, device="cuda")
    ref = orc.backward_gqa(*xs, f64(x["dO"]), scale)
    errs = {n: grad_err(g, r) for n, g, r in zip(("dQ", "dK", "dV", "dKd", "dVd"), (dQ, dK, dV, dKd, dVd), ref)}
    bad = {n: e for n, e in errs.items() if not e <= TOL_GRAD_REL_L2}
    assert not bad, f"gradient rel-L2 over tolerance: {bad} (all: {errs})"
    rows = {n: worst_row_rel_l2(f64(g), r) for n, g, r in zip(("dQ", "dK", "dV", "dKd", "dVd"), (dQ, dK, dV, dKd, dVd), ref) if np.asarray(r).size}
    bad = {n: e for n, e in rows.items() if not e <= TOL_GRAD_ROW_REL_L2}
    assert not bad, f"worst-row gradient rel-L2 over tolerance: {bad} (all: {rows})"

    # the same per-position kernels on the row-interleaved cache, where the host would pick them, give the same bits
    if l > 0 and H // Hk == 8 and l >= 48:
        cache_rows = build_cache(x["Kd"], x["Vd"])
        O2, LSE2 = moda.moda_attn_fwd_gqa(x["Q"], x["K"], x["V"], cache_rows, l, scale)
        assert torch.equal(O, O2) and torch.equal(LSE, LSE2), "the two layouts must give identical outputs"


def test_entry_points_reject_one_head_per_group():
    w = synthetic.Workload("g1", 1, 128, 2, 64, 1)
    x = synthetic.make(w, seed=1, device="cuda")
    cache = build_cache_pm(x["Kd"], x["Vd"])
    with pytest.raises(moda.ModaError) as e:
        moda.moda_attn_fwd_gqa_pm(x["Q"], x["K"], x["V"], cache, 1, w.scale)
    assert e.value.code == -12


def test_paper_table2_shape_one_group_against_the_oracle():
    # The shape family of the paper's kernel table (B = 1, d = 64, 8 key/value heads, G = 8) at T = 8192 with 32 slots, on
    # the GPU in full with the position-major cache; the oracle checks one whole group (8 query heads on one key/value
    # head), which is a problem of its own.
    B, T, H, Hk, d, l, hk = 1, 8192, 64, 8, 64, 32, 5
    G = H // Hk
    scale = d ** -0.5
    x = synthetic.make_gqa(B, T, H, Hk, d, l, seed=2, device="cuda", k_head_norm=True)
    cache = build_cache_pm(x["Kd"], x["Vd"])
    O, LSE = moda.moda_attn_fwd_gqa_pm(x["Q"], x["K"], x["V"], cache, l, scale)
    dQ, dK, dV, dcache = moda.moda_attn_bwd_gqa_pm(x["Q"], x["K"], x["V"], cache, O, x["dO"], LSE, l, scale)
    assert moda.moda_last_status() == 0
    dKd, dVd = unpack_cache_pm(dcache, l, B, T, Hk, d)
    qs = slice(hk * G, (hk + 1) * G)
    xs = [f64(x["Q"][:, :, qs]), f64(x["K"][:, :, hk:hk + 1]), f64(x["V"][:, :, hk:hk + 1]),
          f64(x["Kd"][:, :, :, hk:hk + 1]), f64(x["Vd"][:, :, :, hk:hk + 1])]
    O_ref, LSE_ref = orc.forward_gqa(*xs, scale)
    assert_forward_close(O[:, :, qs], LSE[:, qs], O_ref, LSE_ref, "Table 2 shape, position-major cache")
    ref = orc.backward_gqa(*xs, f64(x["dO"][:, :, qs]), scale)
    got = (dQ[:, :, qs], dK[:, :, hk:hk + 1], dV[:, :, hk:hk + 1], dKd[:, :, :, hk:hk + 1], dVd[:, :, :, hk:hk + 1])
    for name, g, r in zip(("dQ", "dK", "dV", "dKd", "dVd"), got, ref):
        assert grad_err(g, r) <= TOL_GRAD_REL_L2, f"{name}: {grad_err(g, r):.3e}"
