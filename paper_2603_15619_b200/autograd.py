"""torch.autograd wrapper around the C ABI: one differentiable call per attention layer.

Plumbing only: forward and backward are single calls into the CUDA library (moda_attn_fwd_gqa /
moda_attn_bwd_gqa; plain multi-head attention is the H_kv == H case).  The depth cache is passed
and differentiated in cache layout: the gradient of ``depth_kv`` has the layout of the cache
(kv = 0 holds dKd, kv = 1 holds dVd, slots >= l are zero), so that a stack of layers can add it to
the gradients of the layers that wrote those slots (moda_depth_cache_unpack turns a slot back into
[B, T, H_kv, d] tensors).
"""
from __future__ import annotations

import torch

from . import binding


class _ModaAttention(torch.autograd.Function):
    @staticmethod
    def forward(ctx, Q, K, V, depth_kv, l, scale):
        Q, K, V = Q.contiguous(), K.contiguous(), V.contiguous()
        O, LSE = binding.moda_attn_fwd_gqa(Q, K, V, depth_kv if l > 0 else None, l, scale)
        ctx.save_for_backward(Q, K, V, depth_kv if l > 0 else None, O, LSE)
        ctx.l, ctx.scale = int(l), float(scale)
        ctx.mark_non_differentiable(LSE)
        return O, LSE

    @staticmethod
    def backward(ctx, dO, _dLSE):
        Q, K, V, depth_kv, O, LSE = ctx.saved_tensors
        B, T, H, d = Q.shape
        Hk = K.shape[2]
        l = ctx.l
        d_cache = None
        if l > 0:
            # slots >= l of the caller's cache get no gradient: start from zeros of the cache's size
            d_cache = torch.zeros_like(depth_kv)
        dQ, dK, dV, _ = binding.moda_attn_bwd_gqa(Q, K, V, depth_kv, O, dO.contiguous(), LSE, l, ctx.scale,
                                                  d_depth_kv=d_cache)
        return dQ, dK, dV, d_cache, None, None


def moda_attention(Q, K, V, depth_kv=None, l=0, scale=None):
    """Differentiable MoDA attention of one layer.

    Q [B,T,H,d]; K, V [B,T,H_kv,d] (H_kv divides H); ``depth_kv`` a depth cache with H_kv heads
    holding at least ``l`` slots (see alloc_depth_cache / moda_depth_cache_append).  Returns
    O [B,T,H,d] and LSE [B,H,T] (LSE is not differentiable)."""
    if scale is None:
        scale = Q.shape[-1] ** -0.5
    if l > 0 and depth_kv is None:
        raise ValueError("depth_kv is required when l > 0")
    if depth_kv is None:
        depth_kv = Q.new_empty(0)
    return _ModaAttention.apply(Q, K, V, depth_kv, int(l), float(scale))
