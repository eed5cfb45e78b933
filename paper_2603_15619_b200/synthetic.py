"""Seeded synthetic inputs for the MoDA operator (shapes and value recipes only).

This module holds no arithmetic of the method: it draws Gaussian tensors with the
shapes of the workloads and rounds them to bf16 once.  Both the CUDA path and the CPU
oracle are fed from the tensors made here, so the two sides always see identical bits.

Workloads (B batch, T positions, H heads, d head width, l depth slots per position):

    c1  tiny             B=1 T=256   H=2  d=64  l=4   N(0,1)
    c2  1.5B-shaped      B=4 T=4096  H=16 d=128 l=23  N(0,1); Q, K, depth K times 0.5
    c3  depth sweep      B=2 T=8192  H=16 d=128 l in {0,1,8,16,24,32}  N(0,1)
    c4  long context     B=1 T=65536 H=16 d=128 l=24  N(0,1)
    c5  narrow deep      B=2 T=32768 H=32 d=64  l=32  N(0,1); every K row of head h is
                         multiplied by r[h] ~ U[0.5, 2]; depth slot i uses its own r_i[h]

The paper's own inputs are activations of trained language models; attention cost does
not depend on the values, so i.i.d. Gaussians of the same shapes stand in for them.

Each tensor is drawn from its own generator seeded by (seed, tensor name, slot), so a
single depth slot or a slice of a large workload can be regenerated without holding the
rest.  The generator of the requested device is used (the CUDA bits differ from the CPU
bits; whichever tensor is made is the one handed to both sides).
"""
from __future__ import annotations

import dataclasses
import math
import zlib

import torch


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    B: int
    T: int
    H: int
    d: int
    l: int
    qk_mul: float = 1.0          # multiplier on Q, K and depth K before bf16 rounding
    k_head_norm: bool = False    # c5: per-head random K row-norm multiplier in [0.5, 2]

    @property
    def scale(self) -> float:
        return 1.0 / math.sqrt(self.d)

    def with_l(self, l: int) -> "Workload":
        return dataclasses.replace(self, l=l, name=f"{self.name.split('_l')[0]}_l{l}")


WORKLOADS = {
    "c1": Workload("c1", B=1, T=256, H=2, d=64, l=4),
    "c2": Workload("c2", B=4, T=4096, H=16, d=128, l=23, qk_mul=0.5),
    "c3": Workload("c3", B=2, T=8192, H=16, d=128, l=32),
    "c4": Workload("c4", B=1, T=65536, H=16, d=128, l=24),
    "c5": Workload("c5", B=2, T=32768, H=32, d=64, l=32, k_head_norm=True),
}
C3_DEPTHS = (0, 1, 8, 16, 24, 32)


def _gen(seed: int, name: str, slot: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed((int(seed) * 1000003 + zlib.crc32(name.encode()) * 97 + slot + 1) % (2 ** 63 - 1))
    return g


def tensor(w: Workload, name: str, seed: int = 0, slot: int = 0, device="cpu") -> torch.Tensor:
    """One bf16 tensor [B, T, H, d] of workload ``w``.

    ``name`` is one of "Q", "K", "V", "dO", "Kd", "Vd"; ``slot`` selects the depth slot
    for "Kd"/"Vd" (ignored otherwise)."""
    if name not in ("Q", "K", "V", "dO", "Kd", "Vd"):
        raise ValueError(name)
    dev = torch.device(device)
    g = _gen(seed, name, slot if name in ("Kd", "Vd") else 0, dev)
    x = torch.randn((w.B, w.T, w.H, w.d), generator=g, device=dev, dtype=torch.float32)
    if name in ("Q", "K", "Kd") and w.qk_mul != 1.0:
        x *= w.qk_mul
    if w.k_head_norm and name in ("K", "Kd"):
        gr = _gen(seed, name + "/headnorm", slot if name == "Kd" else 0, torch.device("cpu"))
        r = 0.5 + 1.5 * torch.rand((w.H,), generator=gr, dtype=torch.float32)
        x *= r.to(dev).view(1, 1, w.H, 1)
    return x.to(torch.bfloat16)


def make(w: Workload, seed: int = 0, device="cpu") -> dict:
    """All inputs of one workload: Q, K, V, dO [B,T,H,d]; Kd, Vd [l,B,T,H,d] (bf16)."""
    out = {n: tensor(w, n, seed, 0, device) for n in ("Q", "K", "V", "dO")}
    shape = (w.l, w.B, w.T, w.H, w.d)
    Kd = torch.empty(shape, dtype=torch.bfloat16, device=device)
    Vd = torch.empty(shape, dtype=torch.bfloat16, device=device)
    for i in range(w.l):
        Kd[i] = tensor(w, "Kd", seed, i, device)
        Vd[i] = tensor(w, "Vd", seed, i, device)
    out["Kd"], out["Vd"] = Kd, Vd
    return out


def make_gqa(B: int, T: int, H: int, H_kv: int, d: int, l: int, seed: int = 0, device="cpu", **kw) -> dict:
    """Inputs of a grouped-query problem: Q, dO [B,T,H,d]; K, V [B,T,H_kv,d]; Kd, Vd [l,B,T,H_kv,d]."""
    wq = Workload("gqa/q", B, T, H, d, l, **kw)
    wk = Workload("gqa/kv", B, T, H_kv, d, l, **kw)
    out = make(wk, seed, device)
    out["Q"] = tensor(wq, "Q", seed, 0, device)
    out["dO"] = tensor(wq, "dO", seed, 0, device)
    return out


def make_decode(B: int, T_kv: int, H: int, H_kv: int, d: int, l: int, seed: int = 0, device="cpu", T_cap=None, **kw) -> dict:
    """Inputs of a decode step: q [B,H,d]; K, V [B,T_cap,H_kv,d] (the KV cache of one layer, positions
    < T_kv meaningful); depth [l,B,H_kv,2,d] (key row, value row of the token's depth pairs).  Same
    distributions as the training-shape tensors."""
    T_cap = T_kv if T_cap is None else T_cap
    wk = Workload("decode/kv", B, T_cap, H_kv, d, l, **kw)
    wq = Workload("decode/q", B, 1, H, d, l, **kw)
    wd = Workload("decode/depth", B, 1, H_kv, d, l, **kw)
    out = {"q": tensor(wq, "Q", seed, 0, device)[:, 0].contiguous(),
           "K": tensor(wk, "K", seed, 0, device), "V": tensor(wk, "V", seed, 0, device)}
    depth = torch.empty((l, B, H_kv, 2, d), dtype=torch.bfloat16, device=device)
    for i in range(l):
        depth[i, :, :, 0] = tensor(wd, "Kd", seed, i, device)[:, 0]
        depth[i, :, :, 1] = tensor(wd, "Vd", seed, i, device)[:, 0]
    out["depth"] = depth
    return out
