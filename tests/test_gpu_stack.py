"""A stack of MoDA layers through DepthStream: every layer's K, V gradient = its own sequence-attention
gradient + the depth gradients that all later layers send to its slot (checked against the oracle)."""
import numpy as np
import pytest
import torch

import paper_2603_15619_b200 as moda
from paper_2603_15619_b200 import synthetic
from oracle import moda_oracle as orc

from parity import TOL_GRAD_REL_L2, TOL_O_REL_L2, f64, rel_l2

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("B,T,H,Hk,d,n_layers", [(1, 300, 2, 2, 64, 4), (1, 256, 4, 2, 128, 3)])
def test_stack_gradients_flow_back_through_the_depth_stream(B, T, H, Hk, d, n_layers):
    scale = d ** -0.5
    layers = []
    for i in range(n_layers):
        x = synthetic.make_gqa(B, T, H, Hk, d, 0, seed=40 + i, device="cuda")
        layers.append({k: x[k].clone().requires_grad_(k != "dO") for k in ("Q", "K", "V", "dO")})
    stream = moda.DepthStream(B, T, Hk, d, n_layers)
    loss = 0.0
    outs = []
    for L in layers:
        O = stream.attend(L["Q"], L["K"], L["V"], scale)
        outs.append(O)
        loss = loss + (O.float() * L["dO"].float()).sum()
    loss.backward()
    assert moda.moda_last_status() == 0

    # oracle: layer l sees slots 0..l-1 = K, V of the earlier layers
    dK_ref = [np.zeros((B, T, Hk, d)) for _ in range(n_layers)]
    dV_ref = [np.zeros((B, T, Hk, d)) for _ in range(n_layers)]
    for l, L in enumerate(layers):
        Kd = np.stack([f64(layers[i]["K"]) for i in range(l)]) if l else np.zeros((0, B, T, Hk, d))
        Vd = np.stack([f64(layers[i]["V"]) for i in range(l)]) if l else np.zeros((0, B, T, Hk, d))
        args = (f64(L["Q"]), f64(L["K"]), f64(L["V"]), Kd, Vd)
        O_ref, _ = orc.forward_gqa(*args, scale)
        assert rel_l2(f64(outs[l]), O_ref) <= TOL_O_REL_L2
        dQ, dK, dV, dKd, dVd = orc.backward_gqa(*args, f64(L["dO"]), scale)
        assert rel_l2(f64(L["Q"].grad), dQ) <= TOL_GRAD_REL_L2, f"dQ of layer {l}"
        dK_ref[l] += dK
        dV_ref[l] += dV
        for i in range(l):
            dK_ref[i] += dKd[i]
            dV_ref[i] += dVd[i]
    for l, L in enumerate(layers):
        assert rel_l2(f64(L["K"].grad), dK_ref[l]) <= TOL_GRAD_REL_L2, f"dK of layer {l}"
        assert rel_l2(f64(L["V"].grad), dV_ref[l]) <= TOL_GRAD_REL_L2, f"dV of layer {l}"
