"""The depth stream's write step fused into the forward (moda_attn_fwd_append), on the GPU through the C ABI:
the slot it writes is bit for bit what moda_depth_cache_append writes, O and LSE are bit for bit those of the plain
forward, and the slot that the next layer reads is really the one that was written."""
import numpy as np
import pytest
import torch

import paper_2603_15619_b200 as moda
from paper_2603_15619_b200 import binding, synthetic

from parity import assert_forward_close, build_cache, f64
from oracle import moda_oracle as orc

pytestmark = pytest.mark.gpu

SHAPES = [
    # B, T, H, H_kv, d, l
    (1, 128, 1, 1, 128, 0), (2, 300, 2, 2, 128, 3), (1, 1000, 3, 3, 64, 2), (1, 257, 4, 2, 64, 5), (2, 129, 8, 2, 128, 1),
    (1, 640, 2, 2, 128, 12),      # 2 l d >= T: the deep-ring variant of the d = 128 kernel
    (1, 1, 2, 1, 64, 0), (1, 520, 16, 2, 64, 33), (1, 130, 8, 1, 128, 50),   # grouped-query calls whose depth part is a second kernel
    # enough CTAs for the d = 128 kernel to take pairs of query tiles (432 pairs fill three waves of 148 SMs to 97 %): a
    # ragged last tile, grouped heads; and a depth-heavy shape (pairs whatever the wave count, an odd number of tiles:
    # the middle one alone) on the deep-ring variant
    (3, 2190, 16, 4, 128, 5), (13, 600, 8, 8, 128, 12),
]


@pytest.mark.parametrize("B,T,H,Hk,d,l", SHAPES)
def test_fused_write_step_is_the_separate_append_bit_for_bit(B, T, H, Hk, d, l):
    scale = d ** -0.5
    x = synthetic.make_gqa(B, T, H, Hk, d, l, seed=41, device="cuda")
    want = moda.alloc_depth_cache(B, T, Hk, d, l + 1)
    got = moda.alloc_depth_cache(B, T, Hk, d, l + 1)
    for c in (want, got):
        c.fill_(7.0)
        for i in range(l):
            moda.moda_depth_cache_append(c, i, x["Kd"][i].contiguous(), x["Vd"][i].contiguous())
    moda.moda_depth_cache_append(want, l, x["K"], x["V"])
    O0, LSE0 = moda.moda_attn_fwd_gqa(x["Q"], x["K"], x["V"], want, l, scale)
    O1, LSE1 = moda.moda_attn_fwd_append(x["Q"], x["K"], x["V"], got, l, scale, got, l)
    assert moda.moda_last_status() == 0
    assert torch.equal(got, want), "slot written by the forward differs from moda_depth_cache_append"
    assert torch.equal(O0, O1) and torch.equal(LSE0, LSE1)
    xs = [f64(x[n]) for n in ("Q", "K", "V", "Kd", "Vd")]
    assert_forward_close(O1, LSE1, *orc.forward_gqa(*xs, scale), "forward with the fused write step")


@pytest.mark.parametrize("d,T,H", [(128, 300, 2), (64, 520, 3), (128, 2190, 16)])
def test_fixed_size_slot_buffer_with_in_place_eviction_is_a_sliding_window(d, T, H):
    # A buffer of S slots: layer i attends to the slots that are filled and then writes its own K, V over the oldest
    # one, in the same launch.  Against the oracle run on the last S layers' K, V (any order: pin P5).
    B, S, layers = (3 if T == 2190 else 1), 3, 6      # the last shape is large enough for the forward to take tile pairs
    scale = d ** -0.5
    g = torch.Generator(device="cuda").manual_seed(77)
    mk = lambda: (torch.randn((B, T, H, d), device="cuda", generator=g) * 0.7).to(torch.bfloat16)
    buf = moda.alloc_depth_cache(B, T, H, d, S)
    buf.fill_(0.0)
    history = []
    for i in range(layers):
        Q, K, V = mk(), mk(), mk()
        l = min(i, S)
        O, LSE = moda.moda_attn_fwd_append(Q, K, V, buf, l, scale, buf, i % S)
        assert moda.moda_last_status() == 0
        window = history[-S:]
        Kd = np.stack([f64(k) for k, _ in window]) if window else np.zeros((0, B, T, H, d))
        Vd = np.stack([f64(v) for _, v in window]) if window else np.zeros((0, B, T, H, d))
        O_ref, LSE_ref = orc.forward(f64(Q), f64(K), f64(V), Kd, Vd, scale)
        assert_forward_close(O, LSE, O_ref, LSE_ref, f"layer {i} of a {S}-slot buffer")
        history.append((K, V))


def test_in_place_eviction_is_rejected_for_grouped_heads():
    B, T, H, Hk, d, l = 1, 128, 4, 2, 64, 2
    x = synthetic.make_gqa(B, T, H, Hk, d, l, seed=3, device="cuda")
    cache = build_cache(x["Kd"], x["Vd"])
    with pytest.raises(moda.ModaError) as e:
        moda.moda_attn_fwd_append(x["Q"], x["K"], x["V"], cache, l, d ** -0.5, cache, 0)
    assert e.value.code == -6
