"""moda_attn_bwd_static_scratch: the backward entry point for callers that cannot supply scratch.

Some users of the library are never in a position to allocate: a plug-in that a host framework
only hands input and output tensors, or a server that fixed its device-memory plan at start-up and
must not call cudaMalloc while serving.  For them the library carries its own 4 MiB scratch array.
This test drives that entry point through the C ABI and checks its gradients against the fp64 oracle
and against what the ordinary moda_attn_bwd returns, on calls in a row (each later call runs on top of
the earlier call's leftovers in the shared array); that the device's free memory is the same before
and after the call (nothing was allocated on its behalf); and that it refuses problems larger than the
built-in array.

The file name sorts last so that a run that stops at the first failure has already run every other
test; the test is self-contained and also passes when run alone in a fresh process.
"""
import ctypes

import pytest
import torch

import paper_2603_15619_b200 as moda
from paper_2603_15619_b200 import binding, synthetic

from parity import TOL_GRAD_REL_L2, build_cache, f64, oracle_backward, rel_l2, unpack_cache

pytestmark = pytest.mark.gpu


def _problem(B, T, H, d, l, seed):
    w = synthetic.Workload("na", B, T, H, d, l)
    x = synthetic.make(w, seed=seed, device="cuda")
    cache = build_cache(x["Kd"], x["Vd"]) if l > 0 else None
    O, LSE = moda.moda_attn_fwd(x["Q"], x["K"], x["V"], cache, l, w.scale)
    return w, x, cache, O, LSE


def _compare(w, x, cache, O, LSE):
    # the built-in scratch holds the row terms only, so the entry point runs the split (reproducible) form
    ref = moda.moda_attn_bwd(x["Q"], x["K"], x["V"], cache, O, x["dO"], LSE, w.l, w.scale,
                             stages=moda.MODA_BWD_ALL_STAGES | moda.MODA_BWD_DETERMINISTIC)
    outs = [torch.full_like(x["Q"], 9.0) for _ in range(3)]
    dcache = None
    if w.l > 0:
        dcache = moda.alloc_depth_cache(w.B, w.T, w.H, w.d, w.l)
        dcache.fill_(9.0)
    # Outputs are the caller's; the binding only marshals pointers.  Free device memory as the driver
    # reports it must not move across the call (a cudaMalloc anywhere below would lower it).
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    got = moda.moda_attn_bwd_static_scratch(x["Q"], x["K"], x["V"], cache, O, x["dO"], LSE, w.l, w.scale,
                                            outs[0], outs[1], outs[2], dcache)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before, "device memory was allocated during the call"
    assert moda.moda_last_status() == 0
    # against the oracle, like every other backward test
    refs = oracle_backward(x, w.scale)
    grads = [got[0], got[1], got[2]]
    if w.l > 0:
        grads += list(unpack_cache(got[3], w.l, w.B, w.T, w.H, w.d))
    for n, g, r in zip(("dQ", "dK", "dV", "dKd", "dVd"), grads, refs):
        err = rel_l2(f64(g), r)
        assert err <= TOL_GRAD_REL_L2, f"{n}: rel-L2 {err:.3e} against the oracle"
    names = ("dQ", "dK", "dV", "d_depth_kv")
    for n, g, r in zip(names, got, ref):
        if r is None:
            assert g is None
            continue
        err = rel_l2(f64(g), f64(r))
        assert err <= TOL_GRAD_REL_L2, f"{n}: rel-L2 {err:.3e} against moda_attn_bwd"
        # same kernels, same inputs: in fact the bits agree
        assert torch.equal(g, r), n


def test_static_scratch_matches_workspace_variant_on_two_calls_in_a_row():
    # first call: a small problem; second call: a different, larger one that reuses (and outgrows)
    # whatever the first call left in the shared array
    _compare(*_problem(1, 300, 2, 64, 3, seed=21))
    _compare(*_problem(2, 640, 3, 128, 5, seed=22))
    # and the first problem again, now on top of the second one's leftovers
    _compare(*_problem(1, 300, 2, 64, 3, seed=21))


def test_static_scratch_rejects_oversized_problems_without_launching():
    lib = binding.load()
    p = ctypes.c_void_p(4096)      # never dereferenced: the size check comes before any device work
    rows_over = binding.MODA_STATIC_SCRATCH_ROWS + 128
    rc = lib.moda_attn_bwd_static_scratch(p, p, p, None, p, p, p, 1, rows_over, 1, 64, 0, ctypes.c_float(0.125),
                                          p, p, p, None, None)
    assert rc == -11
    assert "scratch" in binding.strerror(rc)
    assert moda.moda_last_status() == 0
