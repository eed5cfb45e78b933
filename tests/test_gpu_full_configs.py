"""Parity at the full sizes of the benchmark workloads (c3, c4, c5), in the launch configuration
bench.py times.  The oracle cannot run whole tensors of this size, so it computes

  * forward rows (O_t, LSE_t) one by one for sampled positions of EVERY (b, h),
  * backward rows: dQ_t, dKd_i[t], dVd_i[t] for sampled positions, and dK_j, dV_j for sampled keys
    in the last 256 positions (their sums run over few queries),
  * one complete (b, h) slice, forward and backward, per config (c3 at l = 32, c4, c5),

and a property that holds at any size covers the rest: sum_s dV_s + sum_{t,i} dVd_i[t] = sum_t dO_t.
Depth tensors are regenerated slot by slot from their seeds, so the logical [l,B,T,H,d] tensors
never exist in memory; the oracle receives zero-filled depth arrays with only the sampled rows set.
"""
import numpy as np
import pytest
import torch

import paper_2603_15619_b200 as moda
from paper_2603_15619_b200 import synthetic

from parity import TOL_GRAD_REL_L2, TOL_GRAD_ROW_REL_L2, assert_forward_close, f64, rel_l2, worst_row_rel_l2
from oracle import moda_oracle as orc

pytestmark = pytest.mark.gpu
SEED = 0


def run_gpu(w):
    x = {n: synthetic.tensor(w, n, SEED, 0, "cuda") for n in ("Q", "K", "V", "dO")}
    cache = dcache = None
    if w.l > 0:
        cache = moda.alloc_depth_cache(w.B, w.T, w.H, w.d, w.l)
        dcache = moda.alloc_depth_cache(w.B, w.T, w.H, w.d, w.l)
        for i in range(w.l):
            moda.moda_depth_cache_append(cache, i, synthetic.tensor(w, "Kd", SEED, i, "cuda"),
                                         synthetic.tensor(w, "Vd", SEED, i, "cuda"))
    O, LSE = moda.moda_attn_fwd(x["Q"], x["K"], x["V"], cache, w.l, w.scale)
    dQ, dK, dV, dcache = moda.moda_attn_bwd(x["Q"], x["K"], x["V"], cache, O, x["dO"], LSE, w.l, w.scale,
                                            d_depth_kv=dcache)
    assert moda.moda_last_status() == 0
    return x, cache, dcache, O, LSE, dQ, dK, dV


def depth_rows(w, cache_like, ts_by_head):
    """Rows of the logical depth tensors read back from a cache-layout buffer:
    {(b,h): (K rows [l, n, d], V rows [l, n, d])} as float64 (bf16 values are exact in float64)."""
    nt = (w.T + 127) // 128
    c = cache_like.view(w.l, w.B, w.H, nt, 2, w.d // 8, 128, 8)
    out = {}
    for (b, h), ts in ts_by_head.items():
        tt = torch.as_tensor(ts, device="cuda")
        blk = c[:, b, h, tt // 128, :, :, tt % 128, :]            # [n, l, 2, d/8, 8] (advanced indices first)
        blk = blk.permute(1, 0, 2, 3, 4).reshape(w.l, len(ts), 2, w.d)
        out[(b, h)] = (f64(blk[:, :, 0]), f64(blk[:, :, 1]))
    return out


def regenerated_depth_rows(w, ts_by_head):
    """The same rows taken from the seeded generator directly (independent of the cache kernels)."""
    out = {k: (np.zeros((w.l, len(ts), w.d)), np.zeros((w.l, len(ts), w.d))) for k, ts in ts_by_head.items()}
    for i in range(w.l):
        kd = synthetic.tensor(w, "Kd", SEED, i, "cuda")
        vd = synthetic.tensor(w, "Vd", SEED, i, "cuda")
        for (b, h), ts in ts_by_head.items():
            tt = torch.as_tensor(ts, device="cuda")
            out[(b, h)][0][i] = f64(kd[b, tt, h])
            out[(b, h)][1][i] = f64(vd[b, tt, h])
        del kd, vd
    return out


def check_config(w, heads_bwd=4, rows_per_head=6, tail=256, seed=1):
    x, cache, dcache, O, LSE, dQ, dK, dV = run_gpu(w)
    rng = np.random.default_rng(seed)
    fixed = sorted({0, 1, 127, 128, w.T // 2 - 1, w.T // 2 + 1, w.T - 1})
    ts_by_head = {(b, h): fixed + sorted(rng.integers(0, w.T, size=rows_per_head).tolist())
                  for b in range(w.B) for h in range(w.H)}
    drows = regenerated_depth_rows(w, ts_by_head) if w.l else {}
    bwd_heads = [(0, 0), (w.B - 1, w.H - 1)] + [(int(rng.integers(w.B)), int(rng.integers(w.H))) for _ in range(heads_bwd - 2)]
    if w.l:
        g_rows = depth_rows(w, dcache, ts_by_head)
    worst = {}
    for (b, h), ts in ts_by_head.items():
        sl = lambda t: f64(t[b:b + 1, :, h:h + 1])
        Qs, Ks, Vs, dOs = sl(x["Q"]), sl(x["K"]), sl(x["V"]), sl(x["dO"])
        Kd = np.zeros((w.l, 1, w.T, 1, w.d))
        Vd = np.zeros((w.l, 1, w.T, 1, w.d))
        if w.l:
            Kd[:, 0, ts, 0] = drows[(b, h)][0]
            Vd[:, 0, ts, 0] = drows[(b, h)][1]
        rows = np.array([(0, 0, t) for t in ts], dtype=np.int32)
        O_ref, LSE_ref = orc.forward_rows(Qs, Ks, Vs, Kd, Vd, w.scale, rows)
        tt = torch.tensor(ts, device="cuda")
        e = assert_forward_close(O[b, tt, h], LSE[b, h, tt], O_ref, LSE_ref, f"{w.name} b={b} h={h}")
        worst["O"] = max(worst.get("O", 0), e[0])
        if (b, h) not in bwd_heads:
            continue
        # backward rows; key rows from the last `tail` positions (depth rows of that window are needed too)
        t0 = w.T - tail
        kts = sorted({w.T - 1, w.T - 2, t0, t0 + 1, t0 + 127, t0 + 128} | set(rng.integers(t0, w.T, size=4).tolist()))
        if w.l:
            win = {(b, h): list(range(t0, w.T))}
            wr = regenerated_depth_rows(w, win)[(b, h)]
            Kd[:, 0, t0:, 0] = wr[0]
            Vd[:, 0, t0:, 0] = wr[1]
        krows = np.array([(0, 0, j) for j in kts], dtype=np.int32)
        dQ_r, dKd_r, dVd_r, dK_r, dV_r = orc.backward_rows(Qs, Ks, Vs, Kd, Vd, dOs, w.scale, rows, krows, t_start=t0)
        kt = torch.tensor(kts, device="cuda")
        errs = {"dQ": rel_l2(f64(dQ[b, tt, h]), dQ_r), "dK": rel_l2(f64(dK[b, kt, h]), dK_r),
                "dV": rel_l2(f64(dV[b, kt, h]), dV_r)}
        if w.l:
            gk, gv = g_rows[(b, h)]                         # [l, n, d]
            errs["dKd"] = rel_l2(gk.transpose(1, 0, 2), dKd_r)
            errs["dVd"] = rel_l2(gv.transpose(1, 0, 2), dVd_r)
        bad = {n: v for n, v in errs.items() if not v <= TOL_GRAD_REL_L2}
        assert not bad, f"{w.name} b={b} h={h}: {bad} (all {errs})"
        rerrs = {"dQ": worst_row_rel_l2(f64(dQ[b, tt, h]), dQ_r), "dK": worst_row_rel_l2(f64(dK[b, kt, h]), dK_r),
                 "dV": worst_row_rel_l2(f64(dV[b, kt, h]), dV_r)}
        if w.l:
            rerrs["dKd"] = worst_row_rel_l2(gk.transpose(1, 0, 2), dKd_r)
            rerrs["dVd"] = worst_row_rel_l2(gv.transpose(1, 0, 2), dVd_r)
        bad = {n: v for n, v in rerrs.items() if not v <= TOL_GRAD_ROW_REL_L2}
        assert not bad, f"{w.name} b={b} h={h}: worst sampled row {bad} (all {rerrs})"
        for n, v in errs.items():
            worst[n] = max(worst.get(n, 0), v)
    # property at full size
    lhs = dV.float().sum(dim=1)
    if w.l:
        nt = (w.T + 127) // 128
        c = dcache.view(w.l, w.B, w.H, nt, 2, w.d // 8, 128, 8)
        lhs = lhs + c[:, :, :, :, 1].float().sum(dim=(0, 3, 5)).reshape(w.B, w.H, w.d)
    rhs = x["dO"].float().sum(dim=1)
    err = float((lhs - rhs).norm() / rhs.norm())
    assert err < 2e-2, f"{w.name}: value-gradient mass identity off by {err:.3e}"
    return x, (O, LSE, dQ, dK, dV, dcache), worst


def check_slice(w, x, outs, b, h):
    """One complete (b, h) slice, forward and backward, against the oracle run on that slice alone."""
    O, LSE, dQ, dK, dV, dcache = outs
    sl = lambda t: f64(t[b:b + 1, :, h:h + 1])
    Kd = np.zeros((w.l, 1, w.T, 1, w.d))
    Vd = np.zeros((w.l, 1, w.T, 1, w.d))
    for i in range(w.l):
        Kd[i, 0, :, 0] = f64(synthetic.tensor(w, "Kd", SEED, i, "cuda")[b, :, h])
        Vd[i, 0, :, 0] = f64(synthetic.tensor(w, "Vd", SEED, i, "cuda")[b, :, h])
    args = (sl(x["Q"]), sl(x["K"]), sl(x["V"]), Kd, Vd)
    O_ref, LSE_ref = orc.forward(*args, w.scale)
    assert_forward_close(O[b:b + 1, :, h:h + 1], LSE[b:b + 1, h:h + 1], O_ref, LSE_ref, f"{w.name} slice")
    refs = orc.backward(*args, sl(x["dO"]), w.scale)
    pairs = {"dQ": (sl(dQ), refs[0]), "dK": (sl(dK), refs[1]), "dV": (sl(dV), refs[2])}
    if w.l:
        all_t = {(b, h): list(range(w.T))}
        gk, gv = depth_rows(w, dcache, all_t)[(b, h)]        # [l, T, d]
        pairs["dKd"] = (gk, refs[3][:, 0, :, 0])
        pairs["dVd"] = (gv, refs[4][:, 0, :, 0])
    errs = {n: rel_l2(g, r) for n, (g, r) in pairs.items()}
    bad = {n: v for n, v in errs.items() if not v <= TOL_GRAD_REL_L2}
    assert not bad, f"{w.name} slice b={b} h={h}: {bad} (all {errs})"
    # every row of the slice on its own: dK / dV rows near j = 0 are sums over the whole sequence (the
    # longest inner loops of the dK/dV pass), rows near T - 1 over a few queries
    rerrs = {n: worst_row_rel_l2(g, r) for n, (g, r) in pairs.items()}
    bad = {n: v for n, v in rerrs.items() if not v <= TOL_GRAD_ROW_REL_L2}
    assert not bad, f"{w.name} slice b={b} h={h}: worst row {bad} (all {rerrs})"
    return errs, rerrs


@pytest.mark.parametrize("l", list(synthetic.C3_DEPTHS))
def test_c3_depth_sweep_points(l):
    w = synthetic.WORKLOADS["c3"].with_l(l)
    x, outs, _ = check_config(w, heads_bwd=3)
    if l == 32:
        check_slice(w, x, outs, w.B - 1, 3)


def test_c4_long_context_64k():
    w = synthetic.WORKLOADS["c4"]
    x, outs, _ = check_config(w, heads_bwd=3)
    # One complete head at T = 65536: every dK / dV row, including those of the first key tiles whose
    # sums run over all 65536 queries, and every dQ / depth-gradient row, against the oracle.
    check_slice(w, x, outs, 0, 5)


def test_c5_narrow_heads_deep_stack():
    w = synthetic.WORKLOADS["c5"]
    x, outs, _ = check_config(w, heads_bwd=3, rows_per_head=3)
    check_slice(w, x, outs, 1, 17)


@pytest.mark.parametrize("d", [128, 64])
def test_twice_the_longest_configured_context(d):
    # T = 131072 (1024 query tiles per head), beyond every configured workload: index arithmetic,
    # barrier phases over very long loops and the causal imbalance at its largest
    w = synthetic.Workload("t128k", 1, 131072, 2, d, 4)
    check_config(w, heads_bwd=2, rows_per_head=3)
