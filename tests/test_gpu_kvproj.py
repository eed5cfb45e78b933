"""Key / value projection with the write step in its epilogue (moda_kv_project_append) on the GPU against the fp64 oracle,
through the C ABI: K = X W_K, V = X W_V, and the depth slot written by the same launch."""
import numpy as np
import pytest
import torch

import paper_2603_15619_b200 as moda
from oracle import moda_oracle as orc

from parity import TOL_O_REL_L2, f64, rel_l2, worst_row_rel_l2

pytestmark = pytest.mark.gpu


def make(B, T, Dm, Hk, d, seed):
    g = torch.Generator(device="cuda").manual_seed(seed)
    X = torch.randn((B, T, Dm), device="cuda", generator=g).to(torch.bfloat16)
    Wk = (torch.randn((Hk * d, Dm), device="cuda", generator=g) * Dm ** -0.5).to(torch.bfloat16)
    Wv = (torch.randn((Hk * d, Dm), device="cuda", generator=g) * Dm ** -0.5).to(torch.bfloat16)
    return X, Wk, Wv


SHAPES = [
    # B, T, D_model, H_kv, d
    (1, 128, 64, 1, 64), (1, 1, 64, 1, 128), (2, 300, 256, 2, 128), (1, 1000, 512, 3, 64), (1, 129, 1024, 2, 128),
    (3, 257, 320, 5, 64), (1, 640, 2048, 2, 128),     # more input features than the ring holds: it wraps several times
    # more work items than resident CTA pairs (74 on a B200): a pair takes several items, both accumulator sets are
    # reused, and (odd tile count) the last pair of each batch entry has a CTA without a tile
    (2, 2000, 256, 6, 128), (3, 2500, 128, 8, 128), (4, 1300, 192, 8, 64), (2, 2700, 64, 7, 64),
]


@pytest.mark.parametrize("B,T,Dm,Hk,d", SHAPES)
def test_projection_and_slot_match_the_oracle(B, T, Dm, Hk, d):
    X, Wk, Wv = make(B, T, Dm, Hk, d, seed=3)
    cache = moda.alloc_depth_cache(B, T, Hk, d, 3)
    cache.fill_(7.0)
    pad = 4096
    bufs = [torch.full((pad + B * T * Hk * d + pad,), 3.0, dtype=torch.bfloat16, device="cuda") for _ in range(2)]
    K_out, V_out = (bf[pad:pad + B * T * Hk * d].view(B, T, Hk, d) for bf in bufs)
    moda.moda_kv_project_append(X, Wk, Wv, Hk, cache=cache, slot=1, K_out=K_out, V_out=V_out)
    assert moda.moda_last_status() == 0
    for bf in bufs:
        assert bool((bf[:pad] == 3.0).all()) and bool((bf[-pad:] == 3.0).all()), "guard band overwritten"
    K_ref, V_ref = orc.project_kv(f64(X), f64(Wk), f64(Wv), Hk)
    for name, got, ref in (("K", K_out, K_ref), ("V", V_out, V_ref)):
        assert rel_l2(f64(got), ref) <= TOL_O_REL_L2, f"{name}: rel-L2 {rel_l2(f64(got), ref):.3e}"
        assert worst_row_rel_l2(f64(got), ref) <= 2e-2, f"{name}: worst row {worst_row_rel_l2(f64(got), ref):.3e}"
    # the slot is bit for bit what the separate append stores from the rounded K, V; the neighbouring slots are untouched
    want = moda.alloc_depth_cache(B, T, Hk, d, 3)
    want.fill_(7.0)
    moda.moda_depth_cache_append(want, 1, K_out.contiguous(), V_out.contiguous())
    assert torch.equal(cache, want)


def test_slot_only_and_projection_only_modes():
    B, T, Dm, Hk, d = 2, 300, 256, 2, 128
    X, Wk, Wv = make(B, T, Dm, Hk, d, seed=5)
    K_out, V_out = moda.moda_kv_project_append(X, Wk, Wv, Hk)                 # no cache: the projection alone
    cache = moda.alloc_depth_cache(B, T, Hk, d, 2)
    cache.fill_(7.0)
    none = moda.moda_kv_project_append(X, Wk, Wv, Hk, cache=cache, slot=0, store_kv=False)   # FFN-side: the slot alone
    assert none == (None, None) and moda.moda_last_status() == 0
    want = moda.alloc_depth_cache(B, T, Hk, d, 2)
    want.fill_(7.0)
    moda.moda_depth_cache_append(want, 0, K_out, V_out)
    assert torch.equal(cache, want)


def test_the_written_slot_feeds_the_attention():
    # layer 0 of a stack: its K, V come out of the projection, go into slot 0 in the same launch, and the next layer attends
    # to them as its depth keys; the oracle does the same with its own projection (rounded to bf16 where the tensors are)
    B, T, Dm, H, d = 1, 384, 256, 2, 64
    X, Wk, Wv = make(B, T, Dm, H, d, seed=7)
    cache = moda.alloc_depth_cache(B, T, H, d, 1)
    K0, V0 = moda.moda_kv_project_append(X, Wk, Wv, H, cache=cache, slot=0)
    g = torch.Generator(device="cuda").manual_seed(8)
    Q, K1, V1 = ((torch.randn((B, T, H, d), device="cuda", generator=g) * 0.7).to(torch.bfloat16) for _ in range(3))
    O, LSE = moda.moda_attn_fwd(Q, K1, V1, cache, 1, d ** -0.5)
    K_ref, V_ref = orc.project_kv(f64(X), f64(Wk), f64(Wv), H)
    bf = lambda a: torch.from_numpy(a).to(torch.bfloat16).double().numpy()
    O_ref, LSE_ref = orc.forward(f64(Q), f64(K1), f64(V1), bf(K_ref)[None], bf(V_ref)[None], d ** -0.5)
    from parity import assert_forward_close
    assert_forward_close(O, LSE, O_ref, LSE_ref, "attention over a projected slot")


@pytest.mark.parametrize("B,T,Dm,Hk,d", [(1, 65536, 2048, 16, 128), (2, 32768, 2048, 32, 64)])
def test_benchmark_shapes_on_sampled_outputs(B, T, Dm, Hk, d):
    """The shapes bench.py times (every resident CTA pair takes ~55 work items): sampled positions of every head against
    fp64 dot products, the slot against the separate append on whole sampled tiles, and nothing written past the tensors."""
    X, Wk, Wv = make(B, T, Dm, Hk, d, seed=11)
    cache = moda.alloc_depth_cache(B, T, Hk, d, 1)
    pad = 4096
    bufs = [torch.full((pad + B * T * Hk * d + pad,), 3.0, dtype=torch.bfloat16, device="cuda") for _ in range(2)]
    K_out, V_out = (bf[pad:pad + B * T * Hk * d].view(B, T, Hk, d) for bf in bufs)
    moda.moda_kv_project_append(X, Wk, Wv, Hk, cache=cache, slot=0, K_out=K_out, V_out=V_out)
    assert moda.moda_last_status() == 0
    for bf in bufs:
        assert bool((bf[:pad] == 3.0).all()) and bool((bf[-pad:] == 3.0).all()), "guard band overwritten"
    rng = np.random.default_rng(5)
    ts = np.unique(np.concatenate([[0, 127, 128, T - 129, T - 128, T - 1], rng.integers(0, T, size=58)]))
    Wk64, Wv64 = f64(Wk), f64(Wv)
    for b in range(B):
        x = f64(X[b, torch.from_numpy(ts).cuda()])                       # [n, Dm]
        for name, got, W in (("K", K_out, Wk64), ("V", V_out, Wv64)):
            ref = (x @ W.T).reshape(len(ts), Hk, d)
            g = f64(got[b, torch.from_numpy(ts).cuda()])
            assert rel_l2(g, ref) <= TOL_O_REL_L2, f"{name}, b = {b}: rel-L2 {rel_l2(g, ref):.3e}"
            assert worst_row_rel_l2(g, ref) <= 2e-2, f"{name}, b = {b}: worst row {worst_row_rel_l2(g, ref):.3e}"
    want = moda.alloc_depth_cache(B, T, Hk, d, 1)
    moda.moda_depth_cache_append(want, 0, K_out.contiguous(), V_out.contiguous())
    assert torch.equal(cache, want)


@pytest.mark.parametrize("B,T,Dm,Hk,d", [(1, 128, 64, 1, 64), (2, 300, 256, 2, 128), (1, 1000, 512, 3, 64), (3, 257, 320, 4, 64),
                                         (3, 2500, 128, 8, 128), (2, 2700, 64, 7, 64)])
def test_e4m3_slot_written_by_the_projection(B, T, Dm, Hk, d):
    """The slot in the e4m3 layout: codes and row scales are the oracle's quantiser applied to the bf16 K, V the same
    launch stores, byte for byte what the separate quantising append writes (tail rows: code 0, scale 1)."""
    from test_gpu_e4m3_cache import unpack_cache8
    X, Wk, Wv = make(B, T, Dm, Hk, d, seed=13)
    X[0, min(5, T - 1), :] = 0                                           # a zero row: scale 1, codes 0
    cache = moda.alloc_depth_cache_e4m3(B, T, Hk, d, 2)
    cache.fill_(0xAB)
    K_out, V_out = moda.moda_kv_project_append_e4m3(X, Wk, Wv, Hk, cache=cache, slot=1)
    assert moda.moda_last_status() == 0
    K_ref, V_ref = orc.project_kv(f64(X), f64(Wk), f64(Wv), Hk)
    assert rel_l2(f64(K_out), K_ref) <= TOL_O_REL_L2 and rel_l2(f64(V_out), V_ref) <= TOL_O_REL_L2
    want = moda.alloc_depth_cache_e4m3(B, T, Hk, d, 2)
    want.fill_(0xAB)
    moda.moda_depth_cache_append_e4m3(want, 1, K_out, V_out)
    assert torch.equal(cache, want)
    codes, scales = unpack_cache8(cache, 2, B, T, Hk, d)
    for kv, Y in enumerate((K_out, V_out)):
        ref_codes, ref_scale = orc.quantize_e4m3_rows(f64(Y))
        assert np.array_equal(scales[1, kv, :, :T], ref_scale) and np.array_equal(codes[1, kv, :, :T], ref_codes)
    # slot only (an FFN-side write): the same bytes without the K, V tensors
    only = moda.alloc_depth_cache_e4m3(B, T, Hk, d, 2)
    only.fill_(0xAB)
    assert moda.moda_kv_project_append_e4m3(X, Wk, Wv, Hk, cache=only, slot=1, store_kv=False) == (None, None)
    assert torch.equal(only, cache)
