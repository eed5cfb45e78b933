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


def rel_l2(got, ref):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    return float(np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-300))


def max_abs(got, ref):
    return float(np.abs(np.asarray(got, dtype=np.float64) - np.asarray(ref, dtype=np.float64)).max())


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
