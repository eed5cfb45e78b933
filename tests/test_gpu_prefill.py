"""Prefill with a cache (T_q newest positions over T_kv cached keys) on the GPU against the fp64 oracle."""
import numpy as np
import pytest
import torch

import paper_2603_15619_b200 as moda
from paper_2603_15619_b200 import synthetic
from oracle import moda_oracle as orc

from parity import TOL_LSE_ABS, TOL_O_MAX_ABS, TOL_O_REL_L2, build_cache, f64, rel_l2

pytestmark = pytest.mark.gpu

SHAPES = [
    # B, T_q, T_kv, H, H_kv, d, l      (offsets: multiples of the tile, of the 64-key block, and neither)
    (1, 128, 256, 2, 2, 128, 3), (1, 128, 384, 2, 1, 64, 2), (2, 100, 164, 4, 2, 128, 4), (1, 130, 200, 2, 2, 64, 5),
    (1, 257, 300, 4, 1, 128, 0), (1, 1, 129, 2, 2, 64, 3), (1, 64, 1000, 4, 2, 128, 2), (2, 200, 777, 8, 2, 64, 1),
    (1, 300, 301, 2, 2, 128, 33), (1, 31, 95, 16, 1, 64, 2), (1, 129, 129, 2, 2, 128, 2),
    (1, 100, 300, 8, 1, 64, 40), (1, 70, 200, 16, 2, 64, 33),        # depth part through the per-position kernel
]


def inputs(B, T_q, T_kv, H, Hk, d, l, seed):
    full = synthetic.make_gqa(B, T_kv, H, Hk, d, l, seed=seed, device="cuda")
    Q = full["Q"][:, T_kv - T_q:].contiguous()
    Kd = full["Kd"][:, :, T_kv - T_q:].contiguous()
    Vd = full["Vd"][:, :, T_kv - T_q:].contiguous()
    return full, Q, Kd, Vd


@pytest.mark.parametrize("B,T_q,T_kv,H,Hk,d,l", SHAPES)
def test_prefill_matches_the_oracle(B, T_q, T_kv, H, Hk, d, l):
    full, Q, Kd, Vd = inputs(B, T_q, T_kv, H, Hk, d, l, seed=21)
    scale = d ** -0.5
    cache = build_cache(Kd, Vd) if l else None
    O, LSE = moda.moda_attn_fwd_prefill(Q, full["K"], full["V"], cache, l, scale)
    assert moda.moda_last_status() == 0
    O_ref, LSE_ref = orc.forward_prefill_gqa(f64(Q), f64(full["K"]), f64(full["V"]), f64(Kd) if l else None,
                                             f64(Vd) if l else None, scale)
    assert rel_l2(f64(O), O_ref) <= TOL_O_REL_L2
    assert np.abs(f64(O) - O_ref).max() <= TOL_O_MAX_ABS
    assert np.abs(f64(LSE) - LSE_ref).max() <= TOL_LSE_ABS


@pytest.mark.parametrize("d", [64, 128])
def test_no_cached_prefix_is_bitwise_the_training_forward(d):
    B, T, H, Hk, l = 1, 300, 4, 2, 3
    x = synthetic.make_gqa(B, T, H, Hk, d, l, seed=5, device="cuda")
    cache = build_cache(x["Kd"], x["Vd"])
    O1, L1 = moda.moda_attn_fwd_gqa(x["Q"], x["K"], x["V"], cache, l, d ** -0.5)
    O2, L2 = moda.moda_attn_fwd_prefill(x["Q"], x["K"], x["V"], cache, l, d ** -0.5)
    assert torch.equal(O1, O2) and torch.equal(L1, L2)


@pytest.mark.parametrize("d,T_q,T_kv", [(128, 2048, 8192), (64, 1000, 6000)])
def test_long_cache_rows_against_the_oracle_and_the_full_forward(d, T_q, T_kv):
    """A long cached prefix: the chunk's rows equal the same rows of the full-sequence kernel (within bf16
    rounding of different block orders) and sampled rows equal the oracle."""
    B, H, Hk, l = 1, 4, 2, 4
    full, Q, Kd, Vd = inputs(B, T_q, T_kv, H, Hk, d, l, seed=8)
    scale = d ** -0.5
    O, LSE = moda.moda_attn_fwd_prefill(Q, full["K"], full["V"], build_cache(Kd, Vd), l, scale)
    Of, Lf = moda.moda_attn_fwd_gqa(full["Q"], full["K"], full["V"], build_cache(full["Kd"], full["Vd"]), l, scale)
    assert moda.moda_last_status() == 0
    assert np.abs(f64(O) - f64(Of[:, T_kv - T_q:])).max() <= 2e-2
    assert np.abs(f64(LSE) - f64(Lf[:, :, T_kv - T_q:])).max() <= 1e-3
    for i in (0, 1, T_q // 2, T_q - 1):
        o, lse = orc.decode_gqa(f64(Q[:, i]), f64(full["K"][:, :T_kv - T_q + i + 1]), f64(full["V"][:, :T_kv - T_q + i + 1]),
                                f64(Kd[:, :, i]), f64(Vd[:, :, i]), scale)
        assert rel_l2(f64(O[:, i]), o) <= TOL_O_REL_L2
        assert np.abs(f64(LSE[:, :, i]) - lse).max() <= TOL_LSE_ABS
