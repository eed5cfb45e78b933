"""FLOP and byte accounting of the MoDA operator (host arithmetic for the reported metric).

Conventions (a multiply-add counts as 2 FLOPs):

* sequence part, forward: two contractions (QK^T and PV) over the causal half of the
  T x T score matrix, counted as 4 * B * H * d * T^2 / 2 (the usual causal convention;
  the exact number of visible pairs is T (T + 1) / 2);
* depth part, forward: two length-d products per (query, depth slot):
  4 * B * H * T * l * d.  This is the prefilling depth-attention cost of the paper's
  Table 1 (2 G T L^2 H_k d + 2 G T L H_k d summed over a stack = 4 T D sum_l l);
* backward = 2.5 x forward (five contractions against two), forward+backward = 3.5 x.

Algorithmic HBM bytes (what the method itself must move, every tensor once):
forward reads Q, K, V (3E bf16), the depth cache (2 l E bf16), writes O (E bf16) and LSE
(B H T fp32); backward reads Q, K, V, O, dO, LSE and the depth cache again and writes
dQ, dK, dV and the depth gradients (2 l E bf16); E = B T H d.
"""
from __future__ import annotations


def fwd_flops(B: int, T: int, H: int, d: int, l: int) -> float:
    return 4.0 * B * H * d * T * T / 2.0 + depth_fwd_flops(B, T, H, d, l)


def depth_fwd_flops(B: int, T: int, H: int, d: int, l: int) -> float:
    return 4.0 * B * H * T * l * d


def bwd_flops(B: int, T: int, H: int, d: int, l: int) -> float:
    return 2.5 * fwd_flops(B, T, H, d, l)


def fwd_bwd_flops(B: int, T: int, H: int, d: int, l: int) -> float:
    return 3.5 * fwd_flops(B, T, H, d, l)


def fwd_bytes(B: int, T: int, H: int, d: int, l: int) -> float:
    E = B * T * H * d
    return 2.0 * (4 * E + 2 * l * E) + 4.0 * B * H * T


def bwd_bytes(B: int, T: int, H: int, d: int, l: int) -> float:
    E = B * T * H * d
    # reads Q K V O dO + depth cache, writes dQ dK dV + depth gradients; LSE read
    return 2.0 * (8 * E + 4 * l * E) + 4.0 * B * H * T


def depth_bytes_fwd(B: int, T: int, H: int, d: int, l: int) -> float:
    return 2.0 * 2 * l * B * T * H * d


def stack_depth_fwd_flops(T: int, D: int, n_layers: int) -> float:
    """Depth-part forward FLOPs of a whole stack in which layer i (0-based) sees the i
    preceding attention layers' K, V as depth slots: sum_i 4 T D i, D = H_q d."""
    return sum(depth_fwd_flops(1, T, 1, D, i) for i in range(n_layers))
