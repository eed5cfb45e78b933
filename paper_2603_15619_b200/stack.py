"""Depth stream of a stack of attention layers, differentiable end to end.

In a MoDA model (paper Sec. 2.2, the "write" step) every attention layer appends its own K, V to
the depth stream after attending, and layer l attends to the l slots written before it.  So K_i, V_i
of layer i receive gradient from layer i's own sequence attention and, as depth slot i, from every
later layer.  ``DepthStream`` owns the depth cache and one gradient cache of the same layout and
wires those contributions together around the C-ABI calls (the backward call's accumulate flag adds
each layer's depth gradients into the shared gradient cache); it is plumbing: no arithmetic of the
operator happens here beyond adding a slot's gradient to its layer's K, V gradient.

    stream = DepthStream(B, T, H_kv, d, n_layers)
    for layer in layers:
        q, k, v = layer.project(x)               # [B,T,H,d], [B,T,H_kv,d], [B,T,H_kv,d]
        o = stream.attend(q, k, v)               # attends to the slots so far, then appends k, v
        x = layer.rest(x, o)

Backward runs the layers in reverse (a token tensor chains the calls so that autograd keeps that
order even if the layers' inputs are unrelated): layer l adds its depth gradients into slots < l of
the gradient cache, and the gradient of its own K, V is its sequence-attention gradient plus slot l
of that cache, which by then holds the contributions of all later layers.
"""
from __future__ import annotations

import torch

from . import binding


class _Attend(torch.autograd.Function):
    @staticmethod
    def forward(ctx, Q, K, V, token, stream, l, scale):
        Q, K, V = Q.contiguous(), K.contiguous(), V.contiguous()
        # attention and the "write" step (slot l = this layer's K, V) in one launch
        O, LSE = binding.moda_attn_fwd_append(Q, K, V, stream.cache if l > 0 else None, l, scale, stream.cache, l)
        ctx.save_for_backward(Q, K, V, O, LSE)
        ctx.stream, ctx.l, ctx.scale = stream, l, scale
        return O, token + 0

    @staticmethod
    def backward(ctx, dO, dtoken):
        Q, K, V, O, LSE = ctx.saved_tensors
        stream, l = ctx.stream, ctx.l
        B, T, H, d = Q.shape
        Hk = K.shape[2]
        # slots < l of the gradient cache receive this layer's share (added in place by the kernel)
        dQ, dK, dV, _ = binding.moda_attn_bwd_gqa(
            Q, K, V, stream.cache if l > 0 else None, O, dO.contiguous(), LSE, l, ctx.scale,
            d_depth_kv=stream.grad_cache if l > 0 else None,
            stages=binding.MODA_BWD_ALL_STAGES | binding.MODA_BWD_ACCUMULATE_DEPTH)
        if stream.slot_has_grad(l):                                     # later layers attended to slot l
            dKs = torch.empty_like(K)
            dVs = torch.empty_like(V)
            binding.moda_depth_cache_unpack(stream.grad_cache, l, dKs, dVs)
            dK += dKs
            dV += dVs
        return dQ, dK, dV, dtoken, None, None, None


class _Write(torch.autograd.Function):
    """A slot written without attending (the FFN-side depth K/V of Sec. 2.2): its gradient is the
    slot of the gradient cache that the later layers filled."""

    @staticmethod
    def forward(ctx, K, V, token, stream, slot):
        K, V = K.contiguous(), V.contiguous()
        binding.moda_depth_cache_append(stream.cache, slot, K, V)
        ctx.stream, ctx.slot = stream, slot
        ctx.save_for_backward(K, V)
        return token + 0

    @staticmethod
    def backward(ctx, dtoken):
        K, V = ctx.saved_tensors
        dK, dV = torch.zeros_like(K), torch.zeros_like(V)
        if ctx.stream.slot_has_grad(ctx.slot):
            binding.moda_depth_cache_unpack(ctx.stream.grad_cache, ctx.slot, dK, dV)
        return dK, dV, dtoken, None, None


class _ProjectWrite(torch.autograd.Function):
    """A slot produced by a key / value projection of X (Sec. 2.2: an FFN layer obtains its depth pair through a KV
    projection of its input) and written by the projection's own epilogue: one launch, K and V never stored.  Backward:
    the slot of the gradient cache is dK, dV; dX = dK Wk + dV Wv and dW = dK^T X are plain library GEMMs."""

    @staticmethod
    def forward(ctx, X, Wk, Wv, token, stream, slot):
        X, Wk, Wv = X.contiguous(), Wk.contiguous(), Wv.contiguous()
        binding.moda_kv_project_append(X, Wk, Wv, stream.shape[2], cache=stream.cache, slot=slot, store_kv=False)
        ctx.stream, ctx.slot = stream, slot
        ctx.save_for_backward(X, Wk, Wv)
        return token + 0

    @staticmethod
    def backward(ctx, dtoken):
        X, Wk, Wv = ctx.saved_tensors
        B, T, Hk, d = ctx.stream.shape
        if not ctx.stream.slot_has_grad(ctx.slot):
            return torch.zeros_like(X), torch.zeros_like(Wk), torch.zeros_like(Wv), dtoken, None, None
        dK = torch.empty((B, T, Hk, d), dtype=X.dtype, device=X.device)
        dV = torch.empty_like(dK)
        binding.moda_depth_cache_unpack(ctx.stream.grad_cache, ctx.slot, dK, dV)
        dK2, dV2, X2 = dK.view(B * T, Hk * d), dV.view(B * T, Hk * d), X.view(B * T, -1)
        dX = torch.addmm(dK2 @ Wk, dV2, Wv).view_as(X)
        return dX, dK2.t() @ X2, dV2.t() @ X2, dtoken, None, None


class DepthStream:
    """Depth cache of one forward pass through a stack (and its gradient cache)."""

    def __init__(self, B, T, H_kv, d, n_layers, device="cuda"):
        self.shape = (B, T, H_kv, d)
        self.n_layers = int(n_layers)
        self.cache = binding.alloc_depth_cache(B, T, H_kv, d, n_layers, device)
        self.grad_cache = torch.zeros_like(self.cache)
        self.n_written = 0
        self.token = torch.zeros((), device=device, requires_grad=True)

    def slot_has_grad(self, l):
        return l < self.n_written - 1

    def attend(self, Q, K, V, scale=None):
        """MoDA attention of the next layer: attends to the slots written so far, then appends K, V."""
        l = self.n_written
        if l >= self.n_layers:
            raise ValueError("more layers than the stream was sized for")
        if scale is None:
            scale = Q.shape[-1] ** -0.5
        O, self.token = _Attend.apply(Q, K, V, self.token, self, l, float(scale))
        self.n_written = l + 1
        return O

    def write(self, K, V):
        """Appends K, V [B,T,H_kv,d] as the next slot without attending (e.g. an FFN layer's depth K/V)."""
        slot = self.n_written
        if slot >= self.n_layers:
            raise ValueError("more slots than the stream was sized for")
        self.token = _Write.apply(K, V, self.token, self, slot)
        self.n_written = slot + 1

    def project_write(self, X, Wk, Wv):
        """Appends K = X Wk^T, V = X Wv^T (X [B,T,D_model], W [H_kv d, D_model]) as the next slot without attending:
        the projection kernel writes the slot from its epilogue."""
        slot = self.n_written
        if slot >= self.n_layers:
            raise ValueError("more slots than the stream was sized for")
        self.token = _ProjectWrite.apply(X, Wk, Wv, self.token, self, slot)
        self.n_written = slot + 1
