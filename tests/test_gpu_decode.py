"""Decode step (T_q = 1) on the GPU against the fp64 oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import paper_2603_15619_b200 as moda
from paper_2603_15619_b200 import synthetic
from oracle import moda_oracle as orc

from parity import TOL_LSE_ABS, TOL_O_MAX_ABS, TOL_O_REL_L2, f64, rel_l2

pytestmark = pytest.mark.gpu

SHAPES = [
    # B, T_kv, T_cap, H, H_kv, d, l
    (1, 1, 1, 1, 1, 64, 0), (1, 1, 8, 2, 1, 128, 3), (2, 31, 31, 4, 2, 64, 2), (1, 255, 300, 2, 2, 128, 5),
    (2, 256, 256, 8, 1, 64, 4), (1, 257, 512, 6, 2, 128, 1), (3, 1000, 1024, 4, 4, 64, 7), (1, 5000, 5000, 8, 2, 128, 24),
    (2, 4097, 4100, 16, 2, 64, 64), (1, 20000, 20000, 3, 1, 128, 256), (1, 3000, 3000, 5, 1, 64, 0), (1, 777, 777, 7, 1, 128, 9),
    # many (batch, kv head) groups: few splits, so every CTA goes round its shared-memory ring several times
    (2, 1300, 1300, 32, 2, 128, 3), (1, 900, 1000, 32, 1, 64, 5), (3, 400, 400, 16, 1, 128, 2),      # G = 16, 32
    (16, 4096, 4096, 16, 8, 128, 4), (24, 6000, 6016, 16, 8, 64, 3), (40, 2500, 2500, 8, 8, 128, 2),
]


def run(x, T_kv, l, scale):
    O, LSE = moda.moda_attn_decode(x["q"], x["K"], x["V"], x["depth"] if l else None, T_kv, l, scale)
    assert moda.moda_last_status() == 0
    return O, LSE


@pytest.mark.parametrize("B,T_kv,T_cap,H,Hk,d,l", SHAPES)
def test_decode_matches_the_oracle(B, T_kv, T_cap, H, Hk, d, l):
    x = synthetic.make_decode(B, T_kv, H, Hk, d, l, seed=11, device="cuda", T_cap=T_cap)
    scale = d ** -0.5
    O, LSE = run(x, T_kv, l, scale)
    kd = f64(x["depth"][:, :, :, 0]) if l else None
    vd = f64(x["depth"][:, :, :, 1]) if l else None
    o_ref, lse_ref = orc.decode_gqa(f64(x["q"]), f64(x["K"][:, :T_kv]), f64(x["V"][:, :T_kv]), kd, vd, scale)
    assert rel_l2(f64(O), o_ref) <= TOL_O_REL_L2
    assert np.abs(f64(O) - o_ref).max() <= TOL_O_MAX_ABS
    assert np.abs(f64(LSE) - lse_ref).max() <= TOL_LSE_ABS


def test_decode_ignores_cache_rows_past_t_kv_and_is_repeatable():
    B, T_kv, T_cap, H, Hk, d, l = 2, 700, 1024, 8, 2, 128, 6
    x = synthetic.make_decode(B, T_kv, H, Hk, d, l, seed=2, device="cuda", T_cap=T_cap)
    O1, L1 = run(x, T_kv, l, d ** -0.5)
    x["K"][:, T_kv:] = float("nan")
    x["V"][:, T_kv:] = float("nan")
    O2, L2 = run(x, T_kv, l, d ** -0.5)
    assert torch.equal(O1, O2) and torch.equal(L1, L2)


def test_decode_equals_the_last_row_of_the_training_forward():
    """The same operator: the decode step of the last position reproduces the full forward's last row."""
    B, T, H, Hk, d, l = 1, 600, 4, 2, 128, 5
    x = synthetic.make_gqa(B, T, H, Hk, d, l, seed=9, device="cuda")
    scale = d ** -0.5
    cache = moda.alloc_depth_cache(B, T, Hk, d, l)
    for i in range(l):
        moda.moda_depth_cache_append(cache, i, x["Kd"][i].contiguous(), x["Vd"][i].contiguous())
    O, LSE = moda.moda_attn_fwd_gqa(x["Q"], x["K"], x["V"], cache, l, scale)
    depth = torch.stack([x["Kd"][:, :, -1], x["Vd"][:, :, -1]], dim=3).contiguous()       # [l,B,Hk,2,d]
    o, lse = moda.moda_attn_decode(x["Q"][:, -1].contiguous(), x["K"], x["V"], depth, T, l, scale)
    assert np.abs(f64(o) - f64(O[:, -1])).max() <= 2e-2
    assert np.abs(f64(lse) - f64(LSE[:, :, -1])).max() <= 2e-3


def test_decode_guard_bands_stay_intact():
    B, T_kv, H, Hk, d, l = 1, 900, 4, 1, 64, 3
    x = synthetic.make_decode(B, T_kv, H, Hk, d, l, seed=4, device="cuda")
    pad = 64
    Obuf = torch.full((B * H * d + 2 * pad,), 7.0, dtype=torch.bfloat16, device="cuda")
    Lbuf = torch.full((B * H + 2 * pad,), 7.0, dtype=torch.float32, device="cuda")
    O = Obuf[pad:pad + B * H * d].view(B, H, d)
    LSE = Lbuf[pad:pad + B * H].view(B, H)
    moda.moda_attn_decode(x["q"], x["K"], x["V"], x["depth"], T_kv, l, d ** -0.5, O=O, LSE=LSE)
    torch.cuda.synchronize()
    for buf, n in ((Obuf, B * H * d), (Lbuf, B * H)):
        assert bool((buf[:pad] == 7.0).all()) and bool((buf[pad + n:] == 7.0).all())
    assert not bool((O == 7.0).all())


def test_back_to_back_decode_steps_are_bitwise_repeatable():
    """Twenty steps queued without a host sync in between (more CTAs than SMs, ring wrapping): same bits each time."""
    B, T_kv, H, Hk, d, l = 32, 8192, 16, 8, 128, 24
    x = synthetic.make_decode(B, T_kv, H, Hk, d, l, seed=1, device="cuda")
    ws = torch.empty(moda.moda_decode_workspace_bytes(B, H, d), dtype=torch.uint8, device="cuda")
    outs = []
    for _ in range(20):
        O = torch.empty_like(x["q"])
        LSE = torch.empty((B, H), dtype=torch.float32, device="cuda")
        moda.moda_attn_decode(x["q"], x["K"], x["V"], x["depth"], T_kv, l, d ** -0.5, O=O, LSE=LSE, workspace=ws)
        outs.append((O, LSE))
    torch.cuda.synchronize()
    assert moda.moda_last_status() == 0
    for O, LSE in outs[1:]:
        assert torch.equal(O, outs[0][0]) and torch.equal(LSE, outs[0][1])
    # sampled rows against the oracle
    for b in (0, 17, 31):
        o_ref, lse_ref = orc.decode_gqa(f64(x["q"][b:b + 1]), f64(x["K"][b:b + 1]), f64(x["V"][b:b + 1]),
                                        f64(x["depth"][:, b:b + 1, :, 0]), f64(x["depth"][:, b:b + 1, :, 1]), d ** -0.5)
        assert rel_l2(f64(outs[0][0][b:b + 1]), o_ref) <= TOL_O_REL_L2
        assert np.abs(f64(outs[0][1][b:b + 1]) - lse_ref).max() <= TOL_LSE_ABS


def oracle_rows(x, lens, l, scale):
    outs = []
    for b, n in enumerate(lens):
        kd = f64(x["depth"][:, b:b + 1, :, 0]) if l else None
        vd = f64(x["depth"][:, b:b + 1, :, 1]) if l else None
        outs.append(orc.decode_gqa(f64(x["q"][b:b + 1]), f64(x["K"][b:b + 1, :n]), f64(x["V"][b:b + 1, :n]), kd, vd, scale))
    return np.concatenate([o for o, _ in outs]), np.concatenate([s for _, s in outs])


@pytest.mark.parametrize("B,T_max,H,Hk,d,l", [(5, 700, 8, 2, 128, 3), (9, 3000, 4, 4, 64, 6), (3, 130, 16, 1, 128, 0)])
def test_decode_with_a_length_per_sequence(B, T_max, H, Hk, d, l):
    x = synthetic.make_decode(B, T_max, H, Hk, d, l, seed=31, device="cuda")
    rng = np.random.default_rng(B)
    lens = [1, T_max] + [int(v) for v in rng.integers(1, T_max + 1, size=B - 2)]
    seq_lens = torch.tensor(lens, dtype=torch.int32, device="cuda")
    scale = d ** -0.5
    O, LSE = moda.moda_attn_decode_varlen(x["q"], x["K"], x["V"], seq_lens, x["depth"] if l else None, T_max, l, scale)
    assert moda.moda_last_status() == 0
    o_ref, lse_ref = oracle_rows(x, lens, l, scale)
    assert rel_l2(f64(O), o_ref) <= TOL_O_REL_L2
    assert np.abs(f64(LSE) - lse_ref).max() <= TOL_LSE_ABS


@pytest.mark.parametrize("B,T_max,H,Hk,d,l,page", [(4, 1000, 8, 2, 128, 4, 64), (6, 2500, 4, 2, 64, 2, 128), (2, 300, 16, 2, 128, 3, 256)])
def test_decode_over_a_paged_cache(B, T_max, H, Hk, d, l, page):
    """Pages scattered by a random permutation; unused page tails and unused pages poisoned with NaN."""
    x = synthetic.make_decode(B, T_max, H, Hk, d, l, seed=33, device="cuda")
    rng = np.random.default_rng(T_max)
    lens = [T_max] + [int(v) for v in rng.integers(1, T_max + 1, size=B - 1)]
    blocks = (T_max + page - 1) // page
    num_pages = B * blocks + 3
    perm = rng.permutation(num_pages)
    Kp = torch.full((num_pages, page, Hk, d), float("nan"), dtype=torch.bfloat16, device="cuda")
    Vp = torch.full_like(Kp, float("nan"))
    table = torch.full((B, blocks), -1, dtype=torch.int32, device="cuda")
    k = 0
    for b, n in enumerate(lens):
        for j in range((n + page - 1) // page):
            pg = int(perm[k]); k += 1
            m = min(page, n - j * page)
            Kp[pg, :m] = x["K"][b, j * page:j * page + m]
            Vp[pg, :m] = x["V"][b, j * page:j * page + m]
            table[b, j] = pg
    seq_lens = torch.tensor(lens, dtype=torch.int32, device="cuda")
    scale = d ** -0.5
    O, LSE = moda.moda_attn_decode_paged(x["q"], Kp, Vp, table, seq_lens, x["depth"] if l else None, T_max, l, scale)
    assert moda.moda_last_status() == 0
    o_ref, lse_ref = oracle_rows(x, lens, l, scale)
    assert rel_l2(f64(O), o_ref) <= TOL_O_REL_L2
    assert np.abs(f64(LSE) - lse_ref).max() <= TOL_LSE_ABS
    # the contiguous entry point with the same lengths gives the same bits
    O2, LSE2 = moda.moda_attn_decode_varlen(x["q"], x["K"], x["V"], seq_lens, x["depth"] if l else None, T_max, l, scale)
    assert torch.equal(O, O2) and torch.equal(LSE, LSE2)
