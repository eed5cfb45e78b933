"""Shared helpers of the GPU parity tests: tolerances, error metrics, oracle marshalling."""
import numpy as np
import torch

import paper_2603_15619_b200 as moda
from oracle import moda_oracle as orc

# Tolerances fixed by the benchmark spec for bf16 inputs with fp32 accumulation.
TOL_O_REL_L2 = 1e-2
TOL_O_MAX_ABS = 2e-2
TOL_LSE_ABS = 1e-3
TOL_GRAD_REL_L2 = 2e-2
# Companion to the per-tensor gradient norm: the worst single row (last axis = features).  A tensor
# norm over millions of rows cannot see a handful of wrong rows; a wrong (missing, stale, misplaced)
# row is off by about its whole norm.  A correct row is a bf16-rounded sum of bf16-rounded products
# (P and dS are rounded to bf16 before their second contraction): a few times 2^-9 of the magnitude of
# its *terms*.  Rows whose terms cancel (dU_i = R_i (<dO, vd_i> - D_t) with the two close, D_t taken
# from the bf16 O) are small with an error set by the terms, so a row is measured against the larger of
# its own norm and the tensor's RMS row norm.
TOL_GRAD_ROW_REL_L2 = 5e-2


def rel_l2(got, ref):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    return float(np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-300))


def max_abs(got, ref):
    return float(np.abs(np.asarray(got, dtype=np.float64) - np.asarray(ref, dtype=np.float64)).max())


def worst_row_rel_l2(got, ref):
    """Largest per-row relative L2 error; rows are the vectors along the last axis."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    if ref.size == 0:
        return 0.0
    got = got.reshape(-1, got.shape[-1])
    ref = ref.reshape(-1, ref.shape[-1])
    norms = np.linalg.norm(ref, axis=1)
    # the absolute part only matters where the exact gradient vanishes identically (one visible key)
    floor = float(np.sqrt(np.mean(norms ** 2))) + 1e-4 * np.sqrt(ref.shape[-1])
    err = np.linalg.norm(got - ref, axis=1) / np.maximum(norms, floor)
    return float(err.max())


def f64(t):
    """Exact conversion of a (bf16) torch tensor to a numpy float64 array."""
    return t.detach().to("cpu", torch.float64).numpy()


def build_cache(Kd, Vd):
    """Pack logical depth tensors [l,B,T,H,d] into the library's cache layout, slot by slot."""
    l, B, T, H, d = Kd.shape
    cache = moda.alloc_depth_cache(B, T, H, d, max(l, 1), Kd.device)
    for i in range(l):
        moda.moda_depth_cache_append(cache, i, Kd[i].contiguous(), Vd[i].contiguous())
    return cache


def unpack_cache(cache, l, B, T, H, d):
    Kd = torch.empty((l, B, T, H, d), dtype=torch.bfloat16, device=cache.device)
    Vd = torch.empty_like(Kd)
    for i in range(l):
        moda.moda_depth_cache_unpack(cache, i, Kd[i], Vd[i])
    return Kd, Vd


def oracle_forward(x, scale):
    return orc.forward(f64(x["Q"]), f64(x["K"]), f64(x["V"]), f64(x["Kd"]), f64(x["Vd"]), scale)


def oracle_backward(x, scale):
    return orc.backward(f64(x["Q"]), f64(x["K"]), f64(x["V"]), f64(x["Kd"]), f64(x["Vd"]), f64(x["dO"]), scale)


def assert_forward_close(O, LSE, O_ref, LSE_ref, what=""):
    e_rel, e_abs = rel_l2(f64(O), O_ref), max_abs(f64(O), O_ref)
    e_lse = max_abs(f64(LSE), LSE_ref)
    assert e_rel <= TOL_O_REL_L2, f"{what}: O rel-L2 {e_rel:.3e}"
    assert e_abs <= TOL_O_MAX_ABS, f"{what}: O max-abs {e_abs:.3e}"
    assert e_lse <= TOL_LSE_ABS, f"{what}: LSE abs {e_lse:.3e}"
    return e_rel, e_abs, e_lse


def assert_same_gradients(a, b, what=""):
    """Two backward calls on the same inputs: dK, dV and the depth gradients agree bit for bit (they
    are accumulated on chip in a fixed order).  dQ tiles are summed into an fp32 accumulator with
    floating-point atomics, so its last fp32 bits depend on the order of arrival and a few of its bf16
    values may round the other way: it must agree to far below the parity tolerance."""
    names = ("dQ", "dK", "dV", "d_depth_kv", "d_depth_v")
    for n, s, t in zip(names, a, b):
        if s is None or t is None:
            assert s is None and t is None, n
            continue
        if n == "dQ":
            err = rel_l2(f64(s), f64(t))
            assert err <= 1e-3, f"{what} dQ differs between identical calls by rel-L2 {err:.3e}"
        else:
            assert torch.equal(s, t), f"{what} {n} changed between identical calls"
