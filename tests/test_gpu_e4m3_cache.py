"""Depth cache in e4m3 with a scale per row: the quantiser bit for bit, and forward / backward parity against the
oracle run on the dequantised slots (GPU, through the C ABI)."""
import numpy as np
import pytest
import torch

import paper_2603_15619_b200 as moda
from paper_2603_15619_b200 import synthetic
from oracle import moda_oracle as orc

from parity import assert_forward_close, f64
from test_gpu_bwd import assert_grads_close

pytestmark = pytest.mark.gpu


def build_cache8(Kd, Vd):
    l, B, T, H, d = Kd.shape
    cache = moda.alloc_depth_cache_e4m3(B, T, H, d, max(l, 1), Kd.device)
    cache.fill_(0xAB)                                       # every byte of slots < l must be overwritten
    for i in range(l):
        moda.moda_depth_cache_append_e4m3(cache, i, Kd[i].contiguous(), Vd[i].contiguous())
    return cache


def unpack_cache8(cache, l, B, T, H, d):
    """(codes uint8 [l, 2, B, Tpad, H, d], scales fp32 [l, 2, B, Tpad, H]) read back from the cache's bytes."""
    nt = (T + 127) // 128
    blk = 128 * d + 512
    raw = cache[: l * B * H * nt * 2 * blk].cpu().numpy().reshape(l, B, H, nt, 2, blk)
    codes = raw[..., : 128 * d].reshape(l, B, H, nt, 2, d // 16, 128, 16)
    codes = codes.transpose(0, 4, 1, 3, 6, 2, 5, 7).reshape(l, 2, B, nt * 128, H, d)       # [l, kv, B, t, H, d]
    scales = np.ascontiguousarray(raw[..., 128 * d:]).view(np.float32).reshape(l, B, H, nt, 2, 128)
    scales = scales.transpose(0, 4, 1, 3, 5, 2).reshape(l, 2, B, nt * 128, H)
    return codes, scales


def oracle_cache8(Kd, Vd):
    """The oracle's codes, scales and dequantised slots of bf16 depth tensors [l, B, T, H, d]."""
    out = []
    for X in (Kd, Vd):
        codes, scale = orc.quantize_e4m3_rows(f64(X))
        out.append((codes, scale, orc.dequantize_e4m3_rows(codes, scale)))
    return out


@pytest.mark.parametrize("B,T,H,d,l", [(1, 128, 1, 64, 1), (2, 300, 3, 128, 2), (1, 1000, 2, 64, 3), (1, 1, 1, 128, 1)])
def test_quantiser_matches_the_oracle_bit_for_bit(B, T, H, d, l):
    w = synthetic.Workload("q", B, T, H, d, l)
    x = synthetic.make(w, seed=5, device="cuda")
    Kd, Vd = x["Kd"].clone(), x["Vd"].clone()
    # rows that exercise the corners: all zero, one huge entry (everything else underflows to subnormal codes or zero),
    # exact ties, a negative zero
    Kd[0, 0, 0, 0, :] = 0
    if T > 2:
        Kd[0, 0, 1, 0, :] = 1e-3
        Kd[0, 0, 1, 0, 0] = 300.0
        Vd[0, 0, 2, 0, :] = torch.linspace(-448, 448, d, device="cuda").to(torch.bfloat16)
        Vd[0, 0, 2, 0, 1] = -0.0
    cache = build_cache8(Kd, Vd)
    codes, scales = unpack_cache8(cache, l, B, T, H, d)
    for kv, X in enumerate((Kd, Vd)):
        ref_codes, ref_scale = orc.quantize_e4m3_rows(f64(X))
        assert np.array_equal(scales[:, kv, :, :T], ref_scale), "row scales differ"
        assert np.array_equal(codes[:, kv, :, :T], ref_codes), "codes differ"
        if T % 128:
            assert (codes[:, kv, :, T:] == 0).all() and (scales[:, kv, :, T:] == 1.0).all(), "tail rows must be code 0, scale 1"


CASES = [(1, 128, 1, 64, 1), (2, 257, 3, 128, 3), (1, 640, 2, 64, 5), (1, 1000, 1, 128, 8), (2, 255, 1, 64, 32),
         (1, 200, 2, 128, 33), (1, 130, 1, 64, 70), (1, 65, 2, 128, 2)]


@pytest.mark.parametrize("B,T,H,d,l", CASES)
def test_forward_and_backward_match_the_oracle_on_the_dequantised_slots(B, T, H, d, l):
    w = synthetic.Workload("e", B, T, H, d, l)
    x = synthetic.make(w, seed=17, device="cuda")
    cache = build_cache8(x["Kd"], x["Vd"])
    (_, _, Kd_hat), (_, _, Vd_hat) = oracle_cache8(x["Kd"], x["Vd"])
    O_ref, LSE_ref = orc.forward(f64(x["Q"]), f64(x["K"]), f64(x["V"]), Kd_hat, Vd_hat, w.scale)
    O, LSE = moda.moda_attn_fwd_e4m3(x["Q"], x["K"], x["V"], cache, l, w.scale)
    assert moda.moda_last_status() == 0
    assert_forward_close(O, LSE, O_ref, LSE_ref, f"e4m3 {(B, T, H, d, l)}")
    # the quantisation is part of the operands, not of the error budget: against the unquantised slots the
    # forward must differ by more than the parity tolerance would hide only if the cache mattered at all
    ref = orc.backward(f64(x["Q"]), f64(x["K"]), f64(x["V"]), Kd_hat, Vd_hat, f64(x["dO"]), w.scale)
    dcache = moda.alloc_depth_cache(B, T, H, d, l)
    dcache.fill_(5.0)
    dQ, dK, dV, dcache = moda.moda_attn_bwd_e4m3(x["Q"], x["K"], x["V"], cache, O, x["dO"], LSE, l, w.scale, d_depth_kv=dcache)
    assert moda.moda_last_status() == 0
    from parity import unpack_cache
    dKd, dVd = unpack_cache(dcache, l, B, T, H, d)
    assert_grads_close((dQ, dK, dV, dKd, dVd), ref, f"e4m3 {(B, T, H, d, l)}")


def test_forward_with_enough_ctas_for_tile_pairs():
    # 432 pairs of query tiles fill three waves of 148 SMs to 97 %: the d = 128 kernel then takes two tiles per CTA
    B, T, H, d, l = 3, 2190, 16, 128, 3
    w = synthetic.Workload("p", B, T, H, d, l)
    x = synthetic.make(w, seed=19, device="cuda")
    cache = build_cache8(x["Kd"], x["Vd"])
    (_, _, Kd_hat), (_, _, Vd_hat) = oracle_cache8(x["Kd"], x["Vd"])
    O_ref, LSE_ref = orc.forward(f64(x["Q"]), f64(x["K"]), f64(x["V"]), Kd_hat, Vd_hat, w.scale)
    O, LSE = moda.moda_attn_fwd_e4m3(x["Q"], x["K"], x["V"], cache, l, w.scale)
    assert moda.moda_last_status() == 0
    assert_forward_close(O, LSE, O_ref, LSE_ref, "e4m3, tile pairs")


def test_the_e4m3_path_reads_the_codes_not_the_original_slots():
    # Slots with a wide dynamic range inside each row: the dequantised slots differ from the originals by far more
    # than the parity tolerance, so a kernel that somehow saw bf16 values (or dropped the scales) fails here.
    B, T, H, d, l = 1, 384, 2, 64, 4
    w = synthetic.Workload("r", B, T, H, d, l)
    x = synthetic.make(w, seed=23, device="cuda")
    g = torch.Generator(device="cuda").manual_seed(3)
    boost = torch.exp2(torch.randint(-6, 3, x["Kd"].shape, device="cuda", generator=g).float())
    Kd = (x["Kd"].float() * boost).to(torch.bfloat16)
    Vd = (x["Vd"].float() * boost).to(torch.bfloat16)
    cache = build_cache8(Kd, Vd)
    (_, _, Kd_hat), (_, _, Vd_hat) = oracle_cache8(Kd, Vd)
    Q, K, V = f64(x["Q"]), f64(x["K"]), f64(x["V"])
    O_hat, LSE_hat = orc.forward(Q, K, V, Kd_hat, Vd_hat, w.scale)
    O_raw, _ = orc.forward(Q, K, V, f64(Kd), f64(Vd), w.scale)
    O, LSE = moda.moda_attn_fwd_e4m3(x["Q"], x["K"], x["V"], cache, l, w.scale)
    assert_forward_close(O, LSE, O_hat, LSE_hat, "wide-range rows")
    gap = np.linalg.norm(O_hat - O_raw) / np.linalg.norm(O_raw)
    assert gap > 1.5e-2, f"the case does not separate quantised from unquantised slots (gap {gap:.2e})"


@pytest.mark.parametrize("B,T,H,Hk,d,l", [(1, 300, 4, 2, 64, 3), (2, 200, 8, 1, 128, 2), (1, 256, 6, 2, 64, 40)])
def test_grouped_query_forward(B, T, H, Hk, d, l):
    w = synthetic.Workload("g", B, T, H, d, l)
    x = synthetic.make(w, seed=29, device="cuda")
    K, V = x["K"][:, :, :Hk].contiguous(), x["V"][:, :, :Hk].contiguous()
    Kd, Vd = x["Kd"][:, :, :, :Hk].contiguous(), x["Vd"][:, :, :, :Hk].contiguous()
    cache = build_cache8(Kd, Vd)
    (_, _, Kd_hat), (_, _, Vd_hat) = oracle_cache8(Kd, Vd)
    O_ref, LSE_ref = orc.forward_gqa(f64(x["Q"]), f64(K), f64(V), Kd_hat, Vd_hat, w.scale)
    O, LSE = moda.moda_attn_fwd_e4m3(x["Q"], K, V, cache, l, w.scale)
    assert moda.moda_last_status() == 0
    assert_forward_close(O, LSE, O_ref, LSE_ref, f"e4m3 gqa {(B, T, H, Hk, d, l)}")


def test_depth_zero_ignores_the_cache_pointer():
    w = synthetic.Workload("z", 1, 200, 2, 64, 0)
    x = synthetic.make(w, seed=1, device="cuda")
    O, LSE = moda.moda_attn_fwd_e4m3(x["Q"], x["K"], x["V"], None, 0, w.scale)
    O2, LSE2 = moda.moda_attn_fwd(x["Q"], x["K"], x["V"], None, 0, w.scale)
    assert torch.equal(O, O2) and torch.equal(LSE, LSE2)


def test_c3_full_size_one_head_slice():
    # The benchmark's T = 8192 shape (c3 with 16 slots) at full size through the e4m3 entry points; heads are independent, so
    # one complete (b, h) slice is checked against the oracle run on that slice alone, with the oracle's own quantiser.
    from parity import unpack_cache
    w = synthetic.WORKLOADS["c3"].with_l(16)
    B, T, H, d, l = w.B, w.T, w.H, w.d, w.l
    x = {n: synthetic.tensor(w, n, 0, 0, "cuda") for n in ("Q", "K", "V", "dO")}
    cache = moda.alloc_depth_cache_e4m3(B, T, H, d, l)
    b, h = B - 1, H // 2
    Kd_h, Vd_h = [], []
    for i in range(l):
        kd, vd = synthetic.tensor(w, "Kd", 0, i, "cuda"), synthetic.tensor(w, "Vd", 0, i, "cuda")
        moda.moda_depth_cache_append_e4m3(cache, i, kd, vd)
        Kd_h.append(f64(kd[b:b + 1, :, h:h + 1]))
        Vd_h.append(f64(vd[b:b + 1, :, h:h + 1]))
        del kd, vd
    O, LSE = moda.moda_attn_fwd_e4m3(x["Q"], x["K"], x["V"], cache, l, w.scale)
    dQ, dK, dV, dcache = moda.moda_attn_bwd_e4m3(x["Q"], x["K"], x["V"], cache, O, x["dO"], LSE, l, w.scale)
    assert moda.moda_last_status() == 0
    (_, _, Kd_hat), (_, _, Vd_hat) = [(None, None, orc.dequantize_e4m3_rows(*orc.quantize_e4m3_rows(np.stack(a)))) for a in (Kd_h, Vd_h)]
    sl = lambda t: f64(t[b:b + 1, :, h:h + 1])
    O_ref, LSE_ref = orc.forward(sl(x["Q"]), sl(x["K"]), sl(x["V"]), Kd_hat, Vd_hat, w.scale)
    assert_forward_close(O[b:b + 1, :, h:h + 1], LSE[b:b + 1, h:h + 1], O_ref, LSE_ref, "c3 l = 16, e4m3 cache")
    ref = orc.backward(sl(x["Q"]), sl(x["K"]), sl(x["V"]), Kd_hat, Vd_hat, sl(x["dO"]), w.scale)
    dKd, dVd = unpack_cache(dcache, l, B, T, H, d)
    got = (dQ[b:b + 1, :, h:h + 1], dK[b:b + 1, :, h:h + 1], dV[b:b + 1, :, h:h + 1],
           dKd[:, b:b + 1, :, h:h + 1], dVd[:, b:b + 1, :, h:h + 1])
    assert_grads_close(got, ref, "c3 l = 16, e4m3 cache")


@pytest.mark.parametrize("B,T,H,Hk,d,l", [(1, 128, 1, 1, 64, 0), (2, 300, 2, 2, 128, 3), (1, 1000, 4, 2, 64, 5), (1, 257, 8, 1, 128, 2),
                                          (3, 2190, 16, 16, 128, 3), (1, 640, 3, 3, 64, 33),
                                          # from 32768 positions on the quantiser runs inside the forward kernel (ragged tail, grouped heads)
                                          (1, 32768 + 70, 2, 1, 128, 2), (1, 32768, 2, 2, 64, 3)])
def test_forward_writes_its_own_slot_in_e4m3(B, T, H, Hk, d, l):
    """moda_attn_fwd_append_e4m3: same output as moda_attn_fwd_e4m3, and the slot holds byte for byte what the quantising
    append stores from K, V (tail rows of a ragged last tile: code 0, scale 1); the other slots are untouched."""
    scale = d ** -0.5
    x = synthetic.make_gqa(B, T, H, Hk, d, l, seed=29, device="cuda")
    want = moda.alloc_depth_cache_e4m3(B, T, Hk, d, l + 1)
    got = moda.alloc_depth_cache_e4m3(B, T, Hk, d, l + 1)
    for c in (want, got):
        c.fill_(0xAB)
        for i in range(l):
            moda.moda_depth_cache_append_e4m3(c, i, x["Kd"][i].contiguous(), x["Vd"][i].contiguous())
    moda.moda_depth_cache_append_e4m3(want, l, x["K"], x["V"])
    O0, LSE0 = moda.moda_attn_fwd_e4m3(x["Q"], x["K"], x["V"], want, l, scale)
    O1, LSE1 = moda.moda_attn_fwd_append_e4m3(x["Q"], x["K"], x["V"], got, l, scale, got, l)
    assert moda.moda_last_status() == 0
    assert torch.equal(got, want), "slot written by the forward differs from moda_depth_cache_append_e4m3"
    assert torch.equal(O0, O1) and torch.equal(LSE0, LSE1)


def test_e4m3_slot_buffer_with_in_place_eviction():
    # a buffer of two e4m3 slots as a sliding window: every layer attends to the two layers before it and writes its own
    # K, V over the older one in the same launch; checked against the oracle on the dequantised slots
    B, T, H, d, S, n_layers = 1, 300, 2, 128, 2, 5
    scale = d ** -0.5
    layers = [synthetic.make_gqa(B, T, H, H, d, 0, seed=60 + n, device="cuda") for n in range(n_layers)]
    cache = moda.alloc_depth_cache_e4m3(B, T, H, d, S)
    owner = {}                                            # slot -> layer it holds
    for n, x in enumerate(layers):
        l = len(owner)
        slot = n % S
        held = [owner[i] for i in range(l)]               # in slot order (the operator does not depend on it)
        O, LSE = moda.moda_attn_fwd_append_e4m3(x["Q"], x["K"], x["V"], cache, l, scale, cache, slot)
        assert moda.moda_last_status() == 0
        deq = lambda t: orc.dequantize_e4m3_rows(*orc.quantize_e4m3_rows(f64(t)))
        Kd = np.stack([deq(layers[m]["K"]) for m in held]) if held else np.zeros((0, B, T, H, d))
        Vd = np.stack([deq(layers[m]["V"]) for m in held]) if held else np.zeros((0, B, T, H, d))
        O_ref, LSE_ref = orc.forward(f64(x["Q"]), f64(x["K"]), f64(x["V"]), Kd, Vd, scale)
        assert_forward_close(O, LSE, O_ref, LSE_ref, f"layer {n} over layers {held}")
        owner[slot] = n
    assert sorted(owner.values()) == [n_layers - 2, n_layers - 1]


def test_quantiser_is_bit_exact_over_a_wide_range_of_rows_and_on_ties():
    """The kernels take the quotient x / scale as a reciprocal and two fused steps; the codes must still be those of the
    IEEE quotient that the oracle rounds.  16 M values: rows scaled by powers of two from 2^-100 to 2^100 (the tiny ones
    take the kernels' IEEE fallback), rows whose scale is a power of two and whose entries sit on rounding ties of the
    format, rows with one entry far above the rest, and plain Gaussian rows."""
    B, T, H, d, l = 2, 4096, 4, 128, 2
    g = torch.Generator(device="cuda").manual_seed(77)
    X = torch.randn((2, l, B, T, H, d), device="cuda", generator=g)
    expo = torch.randint(-100, 101, (2, l, B, T, H, 1), device="cuda", generator=g).float()
    X = X * torch.exp2(expo)
    # ties: row maximum 448 * 2^k (scale exactly 2^k), entries = midpoints between neighbouring e4m3 values times 2^k
    mids = torch.tensor([0.0009765625 * (2 * i + 1) for i in range(8)] + [1.0625 + 0.125 * i for i in range(8)] +
                        [17.0, 19.0, 21.0, 23.0, 25.0, 27.0, 29.0, 31.0, 208.0 + 8, 240.0 + 8, 416.0 + 16, 448.0 - 16],
                        device="cuda")
    tie_rows = mids[torch.randint(0, mids.numel(), (T // 4, d), device="cuda", generator=g)]
    tie_rows = tie_rows * (torch.randint(0, 2, tie_rows.shape, device="cuda", generator=g).float() * 2 - 1)
    tie_rows[:, 0] = 448.0
    X[0, 0, 0, : T // 4, 0, :] = tie_rows * torch.exp2(torch.randint(-20, 21, (T // 4, 1), device="cuda", generator=g).float())
    X[1, 1, 1, :, 1, 5] = 3.0e4                                           # one dominant entry per row
    Kd, Vd = X[0].to(torch.bfloat16), X[1].to(torch.bfloat16)
    cache = build_cache8(Kd, Vd)
    codes, scales = unpack_cache8(cache, l, B, T, H, d)
    for kv, Y in enumerate((Kd, Vd)):
        ref_codes, ref_scale = orc.quantize_e4m3_rows(f64(Y))
        assert np.array_equal(scales[:, kv], ref_scale), "row scales differ"
        bad = np.argwhere(codes[:, kv] != ref_codes)
        assert bad.size == 0, f"{len(bad)} codes differ, first at {bad[0]}: got {codes[:, kv][tuple(bad[0])]}, want {ref_codes[tuple(bad[0])]}"
