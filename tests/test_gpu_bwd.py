"""Backward parity of the CUDA path against the fp64 oracle (GPU, through the C ABI)."""
import numpy as np
import pytest
import torch

import paper_2603_15619_b200 as moda
from paper_2603_15619_b200 import synthetic

from parity import (TOL_GRAD_REL_L2, TOL_GRAD_ROW_REL_L2, assert_same_gradients, build_cache, f64, oracle_backward, rel_l2,
                    unpack_cache, worst_row_rel_l2)

# Both forms of the backward are checked against the oracle: the fused form (the default: five
# contractions, dQ through an fp32 accumulator) and the split, bit-reproducible form.
FORMS = ["fused", "split"]


def stages_of(form):
    return None if form == "fused" else moda.MODA_BWD_ALL_STAGES | moda.MODA_BWD_DETERMINISTIC

pytestmark = pytest.mark.gpu


def run_fwd_bwd(x, w, form="fused"):
    B, T, H, d = x["Q"].shape
    cache = build_cache(x["Kd"], x["Vd"]) if w.l > 0 else None
    O, LSE = moda.moda_attn_fwd(x["Q"], x["K"], x["V"], cache, w.l, w.scale)
    pad = 4096
    n = x["Q"].numel()
    bufs = [torch.full((pad + n + pad,), 3.0, dtype=torch.bfloat16, device="cuda") for _ in range(3)]
    dQ, dK, dV = (bf[pad:pad + n].view(B, T, H, d) for bf in bufs)
    dcache = None
    if w.l > 0:
        dcache = moda.alloc_depth_cache(B, T, H, d, w.l)
        dcache.fill_(5.0)                                  # every element of slots < l must be overwritten
    moda.moda_attn_bwd(x["Q"], x["K"], x["V"], cache, O, x["dO"], LSE, w.l, w.scale,
                       dQ=dQ, dK=dK, dV=dV, d_depth_kv=dcache, stages=stages_of(form))
    assert moda.moda_last_status() == 0
    for bf in bufs:
        assert bool((bf[:pad] == 3.0).all()) and bool((bf[-pad:] == 3.0).all()), "guard band overwritten"
    if w.l > 0:
        dKd, dVd = unpack_cache(dcache, w.l, B, T, H, d)
        nt = (T + 127) // 128
        c = dcache.view(w.l, B, H, nt, 2, d // 8, 128, 8)
        if T % 128:
            assert bool((c[:, :, :, -1, :, :, T % 128:, :] == 0).all()), "tail rows of the depth gradients must be zero"
    else:
        dKd = dVd = torch.zeros((0, B, T, H, d), dtype=torch.bfloat16, device="cuda")
    return dQ, dK, dV, dKd, dVd


def assert_grads_close(got, ref, what):
    names = ("dQ", "dK", "dV", "dKd", "dVd")
    errs = {}
    for n, g, r in zip(names, got, ref):
        if r.size == 0:
            continue
        # relative L2; the 1e-5-per-element floor only matters where the exact gradient vanishes
        # identically (a single visible key makes dQ and dK exactly zero)
        diff = np.linalg.norm(f64(g) - r)
        errs[n] = float(diff / (np.linalg.norm(r) + 1e-5 * np.sqrt(r.size)))
    bad = {n: e for n, e in errs.items() if not e <= TOL_GRAD_REL_L2}
    assert not bad, f"{what}: gradient rel-L2 over tolerance: {bad} (all: {errs})"
    # no single row may hide in the tensor norm
    rows = {n: worst_row_rel_l2(f64(g), r) for n, g, r in zip(names, got, ref) if r.size}
    bad = {n: e for n, e in rows.items() if not e <= TOL_GRAD_ROW_REL_L2}
    assert not bad, f"{what}: worst-row gradient rel-L2 over tolerance: {bad} (all: {rows})"
    return errs


@pytest.mark.parametrize("form", FORMS)
def test_c1_tiny_config_full_parity(form):
    w = synthetic.WORKLOADS["c1"]
    x = synthetic.make(w, seed=0, device="cuda")
    got = run_fwd_bwd(x, w, form)
    assert_grads_close(got, oracle_backward(x, w.scale), "c1")
    got2 = run_fwd_bwd(x, w, form)
    if form == "split":
        for a, b in zip(got, got2):
            assert torch.equal(a, b), "the split form must be deterministic"
    else:
        assert_same_gradients(got, got2, "c1")


SMALL = [
    (1, 1, 1, 64, 0), (1, 1, 1, 64, 3), (1, 2, 1, 128, 1), (2, 127, 2, 64, 1), (1, 128, 1, 128, 0),
    (1, 129, 2, 128, 3), (2, 255, 1, 64, 32), (2, 257, 3, 128, 32), (1, 300, 2, 64, 8), (1, 640, 2, 128, 5),
    (1, 64, 1, 64, 2), (1, 65, 1, 128, 2), (1, 192, 2, 64, 0), (1, 1000, 1, 64, 2),
    # more than 32 depth slots: the forward's online softmax over groups of 32 slots
    (1, 200, 2, 64, 33), (1, 257, 1, 128, 64), (1, 130, 1, 64, 100), (1, 128, 1, 128, 256),
]


# Shapes whose depth streams wrap their shared-memory ring several times, in both dQ kernel variants
# (d = 128 picks the deeper ring when l d / T is large).  A ring stage handed back to the bulk copy
# too early shows up as a few dQ / dKd rows that change from run to run, so repeat and compare bits.
@pytest.mark.parametrize("form", FORMS)
@pytest.mark.parametrize("B,T,H,d,l", [(2, 640, 3, 128, 5), (2, 640, 3, 128, 8), (1, 256, 2, 64, 4), (2, 255, 1, 64, 32)])
def test_backward_is_repeatable_when_the_depth_ring_wraps(B, T, H, d, l, form):
    w = synthetic.Workload("rep", B, T, H, d, l)
    x = synthetic.make(w, seed=22, device="cuda")
    first = run_fwd_bwd(x, w, form)
    assert_grads_close(first, oracle_backward(x, w.scale), f"{(B, T, H, d, l)}")
    for rep in range(30):
        again = run_fwd_bwd(x, w, form)
        if form == "split":
            for name, a, b in zip(("dQ", "dK", "dV", "dKd", "dVd"), first, again):
                assert torch.equal(a, b), f"{name} changed on repeat {rep}"
        else:
            assert_same_gradients(first, again, f"repeat {rep}")


@pytest.mark.parametrize("form", FORMS)
@pytest.mark.parametrize("B,T,H,d,l", SMALL)
def test_small_and_ragged_shapes(B, T, H, d, l, form):
    w = synthetic.Workload("s", B, T, H, d, l)
    x = synthetic.make(w, seed=12, device="cuda")
    got = run_fwd_bwd(x, w, form)
    assert_grads_close(got, oracle_backward(x, w.scale), f"{(B, T, H, d, l)}")


def test_gradient_sum_identities_at_c2_size():
    # sum_s dV_s + sum_{t,i} dVd_i[t] = sum_t dO_t for every (b, h): holds at any size, cheap to check
    w = synthetic.WORKLOADS["c2"]
    x = synthetic.make(w, seed=0, device="cuda")
    dQ, dK, dV, dKd, dVd = run_fwd_bwd(x, w)
    lhs = dV.float().sum(dim=1) + dVd.float().sum(dim=(0, 2))
    rhs = x["dO"].float().sum(dim=1)
    err = float((lhs - rhs).norm() / rhs.norm())
    assert err < 2e-2, err


@pytest.mark.parametrize("form", FORMS)
def test_c2_one_head_slice_full_parity(form):
    # heads are independent (one KV head per query head), so a complete (b, h) slice of the
    # full-size launch can be checked exactly against the oracle run on that slice alone
    w = synthetic.WORKLOADS["c2"]
    x = synthetic.make(w, seed=0, device="cuda")
    got = run_fwd_bwd(x, w, form)
    for (b, h) in ((0, 0), (w.B - 1, w.H - 1)):
        xs = {k: (v[:, b:b + 1, :, h:h + 1] if k in ("Kd", "Vd") else v[b:b + 1, :, h:h + 1]) for k, v in x.items()}
        ref = oracle_backward(xs, w.scale)
        gs = [g[:, b:b + 1, :, h:h + 1] if g.dim() == 5 else g[b:b + 1, :, h:h + 1] for g in got]
        assert_grads_close(gs, ref, f"c2 slice b={b} h={h}")


def test_side_stream_call_with_allocations_interleaved_on_the_default_stream():
    # The wrappers allocate the outputs and the workspace they are not given.  Those blocks must belong
    # to the stream the kernels run on: here the calls go to a side stream while the default stream keeps
    # allocating and scribbling over fresh blocks of the same sizes, which would land in a workspace that
    # had been handed back to the allocator while the backward kernels were still queued.
    w = synthetic.Workload("side", 2, 640, 3, 128, 5)
    x = synthetic.make(w, seed=31, device="cuda")
    cache = build_cache(x["Kd"], x["Vd"])
    ref = oracle_backward(x, w.scale)
    side = torch.cuda.Stream()
    ws_bytes = moda.moda_bwd_workspace_bytes(w.B, w.T, w.H, w.d, w.l)
    for rep in range(5):
        side.wait_stream(torch.cuda.current_stream())
        O, LSE = moda.moda_attn_fwd(x["Q"], x["K"], x["V"], cache, w.l, w.scale, stream=side)
        dQ, dK, dV, dcache = moda.moda_attn_bwd(x["Q"], x["K"], x["V"], cache, O, x["dO"], LSE, w.l, w.scale, stream=side)
        for _ in range(8):                                    # default stream: same-sized blocks, filled at once
            torch.empty(ws_bytes, dtype=torch.uint8, device="cuda").fill_(0x7f)
            torch.empty_like(x["Q"]).fill_(7.0)
        side.synchronize()
        torch.cuda.synchronize()
        dKd, dVd = unpack_cache(dcache, w.l, w.B, w.T, w.H, w.d)
        assert_grads_close((dQ, dK, dV, dKd, dVd), ref, f"side stream, repeat {rep}")


@pytest.mark.parametrize("scale", [1e-6, 0.3])
def test_small_and_large_scales(scale):
    # a tiny scale makes every visible key nearly equally likely, a large one concentrates on the few largest scores; the fused
    # backward carries LSE / scale inside its score contractions
    w = synthetic.Workload("sc", 1, 300, 2, 128, 3)
    x = synthetic.make(w, seed=44, device="cuda")
    cache = build_cache(x["Kd"], x["Vd"])
    O, LSE = moda.moda_attn_fwd(x["Q"], x["K"], x["V"], cache, w.l, scale)
    dQ, dK, dV, dcache = moda.moda_attn_bwd(x["Q"], x["K"], x["V"], cache, O, x["dO"], LSE, w.l, scale)
    assert moda.moda_last_status() == 0
    dKd, dVd = unpack_cache(dcache, w.l, w.B, w.T, w.H, w.d)
    assert_grads_close((dQ, dK, dV, dKd, dVd), oracle_backward(x, scale), f"scale {scale}")
