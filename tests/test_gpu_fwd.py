"""Forward parity of the CUDA path against the fp64 oracle (GPU, through the C ABI)."""
import numpy as np
import pytest
import torch

import paper_2603_15619_b200 as moda
from paper_2603_15619_b200 import synthetic

from parity import assert_forward_close, build_cache, f64, oracle_forward
from oracle import moda_oracle as orc

pytestmark = pytest.mark.gpu


def run_forward(x, w):
    cache = build_cache(x["Kd"], x["Vd"]) if w.l > 0 else None
    B, T, H, d = x["Q"].shape
    # guard bands: poisoned pads around O and LSE must stay untouched
    pad = 4096
    Obuf = torch.full((pad + x["Q"].numel() + pad,), 3.0, dtype=torch.bfloat16, device="cuda")
    Lbuf = torch.full((pad + B * H * T + pad,), 3.0, dtype=torch.float32, device="cuda")
    O = Obuf[pad:pad + x["Q"].numel()].view(B, T, H, d)
    LSE = Lbuf[pad:pad + B * H * T].view(B, H, T)
    moda.moda_attn_fwd(x["Q"], x["K"], x["V"], cache, w.l, w.scale, O=O, LSE=LSE)
    assert moda.moda_last_status() == 0
    for buf in (Obuf, Lbuf):
        assert bool((buf[:pad] == 3.0).all()) and bool((buf[-pad:] == 3.0).all()), "guard band overwritten"
    return O, LSE


def test_c1_tiny_config_full_parity():
    w = synthetic.WORKLOADS["c1"]
    x = synthetic.make(w, seed=0, device="cuda")
    O, LSE = run_forward(x, w)
    O_ref, LSE_ref = oracle_forward(x, w.scale)
    assert_forward_close(O, LSE, O_ref, LSE_ref, "c1")
    # deterministic: a second launch gives the same bits
    O2, LSE2 = run_forward(x, w)
    assert torch.equal(O, O2) and torch.equal(LSE, LSE2)


SMALL = [
    (1, 1, 1, 64, 0), (1, 1, 1, 64, 3), (1, 2, 1, 128, 1), (2, 127, 2, 64, 1), (1, 128, 1, 128, 0),
    (1, 129, 2, 128, 3), (2, 255, 1, 64, 32), (2, 257, 3, 128, 32), (1, 300, 2, 64, 8), (1, 640, 2, 128, 5),
    (1, 1024, 1, 128, 0), (1, 1000, 1, 64, 2),
    # more than 32 depth slots: several groups of the online softmax over the depth keys
    (1, 200, 2, 64, 33), (1, 257, 1, 128, 64), (1, 130, 1, 64, 100), (1, 128, 1, 128, 256), (2, 300, 2, 64, 65),
    # tile pairs in the d = 128 kernel: 432 pairs (three waves of 148 SMs filled to 97 %), with and without depth slots, and
    # a depth-heavy shape with an odd number of tiles
    (3, 2190, 16, 128, 3), (3, 2304, 16, 128, 0), (3, 2100, 12, 128, 40),
]


@pytest.mark.parametrize("B,T,H,d,l", SMALL)
def test_small_and_ragged_shapes(B, T, H, d, l):
    w = synthetic.Workload("s", B, T, H, d, l)
    x = synthetic.make(w, seed=11, device="cuda")
    O, LSE = run_forward(x, w)
    O_ref, LSE_ref = oracle_forward(x, w.scale)
    assert_forward_close(O, LSE, O_ref, LSE_ref, f"{(B, T, H, d, l)}")


def test_large_scores_exercise_rescaling():
    # growing key norms along the sequence force the running maximum up by more than the lazy
    # threshold several times; K scaled per position
    w = synthetic.Workload("r", 1, 1024, 2, 128, 4)
    x = synthetic.make(w, seed=5, device="cuda")
    ramp = torch.linspace(0.2, 3.0, w.T, device="cuda").view(1, w.T, 1, 1)
    x["K"] = (x["K"].float() * ramp).to(torch.bfloat16)
    O, LSE = run_forward(x, w)
    O_ref, LSE_ref = oracle_forward(x, w.scale)
    assert_forward_close(O, LSE, O_ref, LSE_ref, "ramp")


@pytest.mark.parametrize("d,direction", [(64, 1), (128, 1), (64, -1)])
def test_depth_slot_groups_rescale_each_other(d, direction):
    # 80 depth slots = three groups of the online softmax over the depth keys; key norms grow (or
    # shrink) with the slot index, so that later groups raise the running maximum and the partial
    # output of earlier groups must be rescaled (or later groups arrive far below the maximum)
    w = synthetic.Workload("g", 1, 200, 2, d, 80)
    x = synthetic.make(w, seed=8, device="cuda")
    ramp = torch.linspace(0.2, 3.0, w.l, device="cuda")
    if direction < 0:
        ramp = ramp.flip(0)
    x["Kd"] = (x["Kd"].float() * ramp.view(w.l, 1, 1, 1, 1)).to(torch.bfloat16)
    O, LSE = run_forward(x, w)
    O_ref, LSE_ref = oracle_forward(x, w.scale)
    assert_forward_close(O, LSE, O_ref, LSE_ref, "depth ramp")


def test_l0_matches_l_gt0_with_far_away_depth_keys():
    # depth keys with hugely negative scores contribute nothing: l = 0 kernel path == l > 0 path
    w = synthetic.Workload("z", 1, 384, 2, 64, 2)
    x = synthetic.make(w, seed=6, device="cuda")
    x["Kd"] = (-40.0 * x["Q"].float()).to(torch.bfloat16).unsqueeze(0).repeat(2, 1, 1, 1, 1)
    O, LSE = run_forward(x, w)
    w0 = w.with_l(0)
    x0 = dict(x, Kd=x["Kd"][:0], Vd=x["Vd"][:0])
    O0, LSE0 = run_forward(x0, w0)
    assert torch.equal(O, O0)
    assert float((LSE - LSE0).abs().max()) < 1e-5


def check_sampled_rows(w, x, O, LSE, rows_per_head=8, seed=0):
    """Forward rows of every (b, h), computed one by one by the oracle on that head's slice."""
    rng = np.random.default_rng(seed)
    fixed = sorted({0, 1, min(127, w.T - 1), min(128, w.T - 1), w.T // 2 - 1, w.T // 2 + 1, w.T - 1})
    worst = [0.0, 0.0, 0.0]
    for b in range(w.B):
        for h in range(w.H):
            ts = fixed + rng.integers(0, w.T, size=rows_per_head).tolist()
            rows = np.array([(0, 0, t) for t in ts], dtype=np.int32)
            sl = lambda t: f64(t[b:b + 1, :, h:h + 1])
            sld = lambda t: f64(t[:, b:b + 1, :, h:h + 1])
            O_ref, LSE_ref = orc.forward_rows(sl(x["Q"]), sl(x["K"]), sl(x["V"]), sld(x["Kd"]), sld(x["Vd"]),
                                              w.scale, rows)
            tt = torch.tensor(ts, device="cuda")
            e = assert_forward_close(O[b, tt, h], LSE[b, h, tt], O_ref, LSE_ref, f"{w.name} b={b} h={h}")
            worst = [max(a, c) for a, c in zip(worst, e)]
    return worst


def test_c2_full_size_sampled_rows_every_head():
    w = synthetic.WORKLOADS["c2"]
    x = synthetic.make(w, seed=0, device="cuda")
    O, LSE = run_forward(x, w)
    check_sampled_rows(w, x, O, LSE)
