"""ctypes binding of libmoda_b200.so: same names as the C ABI in include/moda.h.

Argument marshalling only -- every step of the operator runs in the CUDA kernels behind
the C entry points.  Tensors are torch CUDA tensors (PyTorch supplies device memory and
streams, nothing else).  There is no CPU fallback: if the library cannot be loaded, or a
call returns an error code, a ``ModaError`` is raised.
"""
from __future__ import annotations

import ctypes
import os

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libmoda_b200.so")

MODA_MAX_DEPTH = 256
SYMBOLS = (
    "moda_version", "moda_strerror", "moda_last_cuda_error", "moda_last_status", "moda_selftest_wait_timeout",
    "moda_depth_cache_bytes", "moda_depth_cache_append", "moda_depth_cache_unpack",
    "moda_attn_fwd", "moda_bwd_workspace_bytes", "moda_attn_bwd", "moda_attn_bwd_stages",
    "moda_attn_bwd_static_scratch",
    "moda_attn_fwd_gqa", "moda_bwd_workspace_bytes_gqa", "moda_attn_bwd_gqa", "moda_attn_bwd_gqa_stages",
    "moda_decode_workspace_bytes", "moda_attn_decode", "moda_attn_fwd_prefill", "moda_attn_fwd_append",
    "moda_attn_decode_varlen", "moda_attn_decode_paged",
    "moda_depth_cache_e4m3_bytes", "moda_depth_cache_append_e4m3", "moda_attn_fwd_e4m3", "moda_attn_bwd_e4m3",
    "moda_depth_cache_append_pm", "moda_depth_cache_unpack_pm", "moda_attn_fwd_gqa_pm", "moda_attn_bwd_gqa_pm",
    "moda_kv_project_append",
    "moda_kv_project_append_e4m3",
    "moda_attn_fwd_append_e4m3",
    "moda_depth_slot_mass_workspace_bytes",
    "moda_depth_slot_mass",
)
MODA_STATIC_SCRATCH_ROWS = 1 << 20
MODA_BWD_STAGE_ROWTERMS, MODA_BWD_STAGE_DQ, MODA_BWD_STAGE_DKDV, MODA_BWD_ALL_STAGES = 1, 2, 4, 7
MODA_BWD_STAGE_ROWS, MODA_BWD_STAGE_SEQ, MODA_BWD_STAGE_FINISH = 1, 2, 4
MODA_BWD_ACCUMULATE_DEPTH = 8      # ORed into a stages mask: depth gradients are added to d_depth_kv
MODA_BWD_DETERMINISTIC = 16        # ORed into a stages mask: the split, bit-reproducible form of the backward


class ModaError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what} failed: [{code}] {strerror(code)}"
                         + (f" (cudaError {last_cuda_error()})" if code == -9 else ""))
        self.code = code


_lib = None


def load() -> ctypes.CDLL:
    """Load the CUDA library (raises if it has not been built: there is no fallback)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2603_15619_b200.build` "
            "(or __graft_entry__.build()). The MoDA operator has no CPU or PyTorch fallback.")
    lib = ctypes.CDLL(LIB_PATH)
    vp, ci, cf, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_size_t
    lib.moda_version.restype = ci
    lib.moda_strerror.restype = ctypes.c_char_p
    lib.moda_strerror.argtypes = [ci]
    lib.moda_last_cuda_error.restype = ci
    lib.moda_last_status.restype = ci
    lib.moda_last_status.argtypes = [ci]
    lib.moda_selftest_wait_timeout.restype = ci
    lib.moda_selftest_wait_timeout.argtypes = [vp]
    lib.moda_depth_cache_bytes.restype = sz
    lib.moda_depth_cache_bytes.argtypes = [ci] * 5
    lib.moda_depth_cache_append.restype = ci
    lib.moda_depth_cache_append.argtypes = [vp, ci, ci, ci, ci, ci, vp, vp, vp]
    lib.moda_depth_cache_unpack.restype = ci
    lib.moda_depth_cache_unpack.argtypes = [vp, ci, ci, ci, ci, ci, vp, vp, vp]
    lib.moda_attn_fwd.restype = ci
    lib.moda_attn_fwd.argtypes = [vp, vp, vp, vp, ci, ci, ci, ci, ci, cf, vp, vp, vp]
    lib.moda_bwd_workspace_bytes.restype = sz
    lib.moda_bwd_workspace_bytes.argtypes = [ci] * 5
    lib.moda_attn_bwd.restype = ci
    lib.moda_attn_bwd.argtypes = [vp] * 7 + [ci] * 5 + [cf] + [vp] * 5 + [sz, vp]
    lib.moda_attn_bwd_stages.restype = ci
    lib.moda_attn_bwd_stages.argtypes = [vp] * 7 + [ci] * 5 + [cf] + [vp] * 5 + [sz, ci, vp]
    lib.moda_attn_bwd_static_scratch.restype = ci
    lib.moda_attn_bwd_static_scratch.argtypes = [vp] * 7 + [ci] * 5 + [cf] + [vp] * 4 + [vp]
    lib.moda_attn_fwd_gqa.restype = ci
    lib.moda_attn_fwd_gqa.argtypes = [vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, cf, vp, vp, vp]
    lib.moda_attn_fwd_append.restype = ci
    lib.moda_attn_fwd_append.argtypes = [vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, cf, vp, vp, vp, ci, vp]
    lib.moda_attn_fwd_append_e4m3.restype = ci
    lib.moda_attn_fwd_append_e4m3.argtypes = [vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, cf, vp, vp, vp, ci, vp]
    lib.moda_bwd_workspace_bytes_gqa.restype = sz
    lib.moda_bwd_workspace_bytes_gqa.argtypes = [ci] * 6
    lib.moda_attn_bwd_gqa.restype = ci
    lib.moda_attn_bwd_gqa.argtypes = [vp] * 7 + [ci] * 6 + [cf] + [vp] * 5 + [sz, vp]
    lib.moda_attn_bwd_gqa_stages.restype = ci
    lib.moda_attn_bwd_gqa_stages.argtypes = [vp] * 7 + [ci] * 6 + [cf] + [vp] * 5 + [sz, ci, vp]
    lib.moda_attn_decode_varlen.restype = ci
    lib.moda_attn_decode_varlen.argtypes = [vp] * 5 + [ci] * 7 + [cf] + [vp] * 3 + [sz, vp]
    lib.moda_attn_decode_paged.restype = ci
    lib.moda_attn_decode_paged.argtypes = [vp] * 6 + [ci] * 9 + [cf] + [vp] * 3 + [sz, vp]
    lib.moda_attn_fwd_prefill.restype = ci
    lib.moda_attn_fwd_prefill.argtypes = [vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, ci, cf, vp, vp, vp]
    lib.moda_decode_workspace_bytes.restype = sz
    lib.moda_decode_workspace_bytes.argtypes = [ci] * 3
    lib.moda_attn_decode.restype = ci
    lib.moda_attn_decode.argtypes = [vp] * 4 + [ci] * 7 + [cf] + [vp] * 3 + [sz, vp]
    lib.moda_depth_cache_e4m3_bytes.restype = sz
    lib.moda_depth_cache_e4m3_bytes.argtypes = [ci] * 5
    lib.moda_depth_cache_append_e4m3.restype = ci
    lib.moda_depth_cache_append_e4m3.argtypes = [vp, ci, ci, ci, ci, ci, vp, vp, vp]
    lib.moda_attn_fwd_e4m3.restype = ci
    lib.moda_attn_fwd_e4m3.argtypes = [vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, cf, vp, vp, vp]
    lib.moda_attn_bwd_e4m3.restype = ci
    lib.moda_attn_bwd_e4m3.argtypes = [vp] * 7 + [ci] * 5 + [cf] + [vp] * 5 + [sz, vp]
    lib.moda_depth_cache_append_pm.restype = ci
    lib.moda_depth_cache_append_pm.argtypes = [vp, ci, ci, ci, ci, ci, vp, vp, vp]
    lib.moda_depth_cache_unpack_pm.restype = ci
    lib.moda_depth_cache_unpack_pm.argtypes = [vp, ci, ci, ci, ci, ci, vp, vp, vp]
    lib.moda_attn_fwd_gqa_pm.restype = ci
    lib.moda_attn_fwd_gqa_pm.argtypes = [vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, cf, vp, vp, vp]
    lib.moda_attn_bwd_gqa_pm.restype = ci
    lib.moda_attn_bwd_gqa_pm.argtypes = [vp] * 7 + [ci] * 6 + [cf] + [vp] * 5 + [sz, vp]
    lib.moda_kv_project_append.restype = ci
    lib.moda_kv_project_append.argtypes = [vp, vp, vp, ci, ci, ci, ci, ci, vp, vp, vp, ci, vp]
    lib.moda_depth_slot_mass_workspace_bytes.restype = ctypes.c_size_t
    lib.moda_depth_slot_mass_workspace_bytes.argtypes = [ci, ci, ci, ci]
    lib.moda_depth_slot_mass.restype = ci
    lib.moda_depth_slot_mass.argtypes = [vp, vp, vp, ci, ci, ci, ci, ci, ci, ctypes.c_float, vp, vp, ctypes.c_size_t, vp]
    lib.moda_kv_project_append_e4m3.restype = ci
    lib.moda_kv_project_append_e4m3.argtypes = [vp, vp, vp, ci, ci, ci, ci, ci, vp, vp, vp, ci, vp]
    _lib = lib
    return lib


def _ptr(t):
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError("device (CUDA) tensors required")
    if not t.is_contiguous():
        raise ValueError("contiguous tensors required")
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def _new(shape, dtype, device, stream):
    """Buffer the wrapper allocates on the caller's behalf.  It is allocated with `stream` current, so
    torch's caching allocator ties the block to the stream the kernels run on: when the Python
    reference is dropped while those kernels are still queued, the block is only handed out again
    to work that is ordered after them (a block made on another stream could be reused at once)."""
    if stream is None:
        return torch.empty(shape, dtype=dtype, device=device)
    with torch.cuda.stream(stream):
        return torch.empty(shape, dtype=dtype, device=device)


def _new_like(t, stream):
    return _new(t.shape, t.dtype, t.device, stream)


def _check(rc: int, what: str):
    if rc != 0:
        raise ModaError(rc, what)


def _bthd(t, name):
    if t.dtype != torch.bfloat16 or t.dim() != 4:
        raise ValueError(f"{name} must be a bf16 [B, T, H, d] tensor")
    return tuple(t.shape)


def moda_version() -> int:
    return int(load().moda_version())


def strerror(code: int) -> str:
    return load().moda_strerror(int(code)).decode()


def last_cuda_error() -> int:
    return int(load().moda_last_cuda_error())


def moda_last_status(clear: bool = False) -> int:
    """Device status word (0 = no kernel gave up a wait). Synchronises the device."""
    return int(load().moda_last_status(int(clear)))


MODA_ERR_DEVICE_TIMEOUT = -10
MODA_SELFTEST_WAIT_STATUS = (255 << 8) | 1


def moda_selftest_wait_timeout(stream=None):
    """Launch the kernel whose only wait runs out after about 1 ms (self-test of the failure reporting)."""
    _check(load().moda_selftest_wait_timeout(_stream(stream)), "moda_selftest_wait_timeout")


def moda_depth_cache_bytes(B, T, H, d, l_max) -> int:
    return int(load().moda_depth_cache_bytes(B, T, H, d, l_max))


def alloc_depth_cache(B, T, H, d, l_max, device="cuda", stream=None) -> torch.Tensor:
    """Caller-side helper: a bf16 buffer of moda_depth_cache_bytes() bytes (uninitialised)."""
    n = moda_depth_cache_bytes(B, T, H, d, l_max)
    if n == 0 and l_max != 0:
        raise ValueError("bad depth-cache shape")
    return _new((max(n // 2, 8),), torch.bfloat16, device, stream)


def depth_cache_window(cache, B, T, H, d, first_slot, n_slots=None):
    """View of slots [first_slot, first_slot + n_slots) of a depth cache (to its end when n_slots is None).

    The cache is slot-major, so a window of consecutive slots is itself a cache: passing the view with
    ``l = n_slots`` makes a layer attend only to those slots (e.g. the last S layers instead of all
    preceding ones, the bounded depth-slot idea of the paper's discussion), and the same view of a
    gradient cache receives exactly their gradients."""
    slot = moda_depth_cache_bytes(B, T, H, d, 1) // 2
    if first_slot < 0 or first_slot * slot > cache.numel():
        raise ValueError("window starts outside the cache")
    end = cache.numel() if n_slots is None else (first_slot + n_slots) * slot
    if end > cache.numel():
        raise ValueError("window ends outside the cache")
    return cache[first_slot * slot:end]


def moda_depth_cache_append(cache, slot, K_i, V_i, stream=None):
    B, T, H, d = _bthd(K_i, "K_i")
    assert _bthd(V_i, "V_i") == (B, T, H, d)
    _check(load().moda_depth_cache_append(_ptr(cache), B, T, H, d, int(slot), _ptr(K_i), _ptr(V_i), _stream(stream)),
           "moda_depth_cache_append")


def moda_depth_cache_unpack(cache, slot, K_i, V_i, stream=None):
    ref = K_i if K_i is not None else V_i
    B, T, H, d = _bthd(ref, "K_i/V_i")
    _check(load().moda_depth_cache_unpack(_ptr(cache), B, T, H, d, int(slot), _ptr(K_i), _ptr(V_i), _stream(stream)),
           "moda_depth_cache_unpack")


def moda_depth_cache_e4m3_bytes(B, T, H, d, l_max) -> int:
    return int(load().moda_depth_cache_e4m3_bytes(B, T, H, d, l_max))


def alloc_depth_cache_e4m3(B, T, H, d, l_max, device="cuda", stream=None) -> torch.Tensor:
    """Caller-side helper: a uint8 buffer of moda_depth_cache_e4m3_bytes() bytes (uninitialised)."""
    n = moda_depth_cache_e4m3_bytes(B, T, H, d, l_max)
    if n == 0 and l_max != 0:
        raise ValueError("bad depth-cache shape")
    return _new((max(n, 16),), torch.uint8, device, stream)


def moda_depth_cache_append_e4m3(cache, slot, K_i, V_i, stream=None):
    """Quantise K_i, V_i (bf16 [B,T,H,d]) into slot ``slot`` of an e4m3 depth cache (codes + one fp32 scale per row)."""
    B, T, H, d = _bthd(K_i, "K_i")
    assert _bthd(V_i, "V_i") == (B, T, H, d)
    _check(load().moda_depth_cache_append_e4m3(_ptr(cache), B, T, H, d, int(slot), _ptr(K_i), _ptr(V_i), _stream(stream)),
           "moda_depth_cache_append_e4m3")


def moda_attn_fwd_e4m3(Q, K, V, depth_kv_e4m3, l, scale, O=None, LSE=None, stream=None):
    """moda_attn_fwd_gqa with the depth slots read from an e4m3 cache."""
    B, T, H, Hk, d = _gqa_shapes(Q, K, V)
    if O is None:
        O = _new_like(Q, stream)
    if LSE is None:
        LSE = _new((B, H, T), torch.float32, Q.device, stream)
    _check(load().moda_attn_fwd_e4m3(_ptr(Q), _ptr(K), _ptr(V), _ptr(depth_kv_e4m3) if l > 0 else None,
                                     B, T, H, Hk, d, int(l), float(scale), _ptr(O), _ptr(LSE), _stream(stream)),
           "moda_attn_fwd_e4m3")
    return O, LSE


def moda_attn_fwd_append_e4m3(Q, K, V, depth_kv_e4m3, l, scale, append_cache_e4m3, append_slot, O=None, LSE=None, stream=None):
    """moda_attn_fwd_e4m3 that also quantises K, V into slot ``append_slot`` of an e4m3 cache in the same launch."""
    B, T, H, Hk, d = _gqa_shapes(Q, K, V)
    if O is None:
        O = _new_like(Q, stream)
    if LSE is None:
        LSE = _new((B, H, T), torch.float32, Q.device, stream)
    _check(load().moda_attn_fwd_append_e4m3(_ptr(Q), _ptr(K), _ptr(V), _ptr(depth_kv_e4m3) if l > 0 else None,
                                            B, T, H, Hk, d, int(l), float(scale), _ptr(O), _ptr(LSE),
                                            _ptr(append_cache_e4m3), int(append_slot), _stream(stream)),
           "moda_attn_fwd_append_e4m3")
    return O, LSE


def moda_attn_bwd_e4m3(Q, K, V, depth_kv_e4m3, O, dO, LSE, l, scale,
                       dQ=None, dK=None, dV=None, d_depth_kv=None, workspace=None, stream=None):
    """moda_attn_bwd with the depth slots read from an e4m3 cache; the depth gradients come back in the bf16 cache layout."""
    B, T, H, d = _bthd(Q, "Q")
    dQ = _new_like(Q, stream) if dQ is None else dQ
    dK = _new_like(K, stream) if dK is None else dK
    dV = _new_like(V, stream) if dV is None else dV
    if l > 0 and d_depth_kv is None:
        d_depth_kv = alloc_depth_cache(B, T, H, d, l, Q.device, stream)
    if workspace is None:
        workspace = _new((moda_bwd_workspace_bytes(B, T, H, d, l),), torch.uint8, Q.device, stream)
    _check(load().moda_attn_bwd_e4m3(_ptr(Q), _ptr(K), _ptr(V), _ptr(depth_kv_e4m3) if l > 0 else None,
                                     _ptr(O), _ptr(dO), _ptr(LSE), B, T, H, d, int(l), float(scale),
                                     _ptr(dQ), _ptr(dK), _ptr(dV), _ptr(d_depth_kv) if l > 0 else None,
                                     _ptr(workspace), workspace.numel() * workspace.element_size(), _stream(stream)),
           "moda_attn_bwd_e4m3")
    return dQ, dK, dV, d_depth_kv


def moda_depth_cache_append_pm(cache, slot, K_i, V_i, stream=None):
    """moda_depth_cache_append for the position-major layout (grouped-query calls through the *_pm entry points)."""
    B, T, H, d = _bthd(K_i, "K_i")
    assert _bthd(V_i, "V_i") == (B, T, H, d)
    _check(load().moda_depth_cache_append_pm(_ptr(cache), B, T, H, d, int(slot), _ptr(K_i), _ptr(V_i), _stream(stream)),
           "moda_depth_cache_append_pm")


def moda_depth_cache_unpack_pm(cache, slot, K_i, V_i, stream=None):
    ref = K_i if K_i is not None else V_i
    B, T, H, d = _bthd(ref, "K_i/V_i")
    _check(load().moda_depth_cache_unpack_pm(_ptr(cache), B, T, H, d, int(slot), _ptr(K_i), _ptr(V_i), _stream(stream)),
           "moda_depth_cache_unpack_pm")


def moda_attn_fwd_gqa_pm(Q, K, V, depth_kv_pm, l, scale, O=None, LSE=None, stream=None):
    """moda_attn_fwd_gqa with the depth slots in the position-major layout (H_kv < H)."""
    B, T, H, Hk, d = _gqa_shapes(Q, K, V)
    if O is None:
        O = _new_like(Q, stream)
    if LSE is None:
        LSE = _new((B, H, T), torch.float32, Q.device, stream)
    _check(load().moda_attn_fwd_gqa_pm(_ptr(Q), _ptr(K), _ptr(V), _ptr(depth_kv_pm) if l > 0 else None,
                                       B, T, H, Hk, d, int(l), float(scale), _ptr(O), _ptr(LSE), _stream(stream)),
           "moda_attn_fwd_gqa_pm")
    return O, LSE


def moda_attn_bwd_gqa_pm(Q, K, V, depth_kv_pm, O, dO, LSE, l, scale,
                         dQ=None, dK=None, dV=None, d_depth_kv_pm=None, workspace=None, stream=None):
    """moda_attn_bwd_gqa with the depth slots and the depth gradients in the position-major layout."""
    B, T, H, Hk, d = _gqa_shapes(Q, K, V)
    dQ = _new_like(Q, stream) if dQ is None else dQ
    dK = _new_like(K, stream) if dK is None else dK
    dV = _new_like(V, stream) if dV is None else dV
    if l > 0 and d_depth_kv_pm is None:
        d_depth_kv_pm = alloc_depth_cache(B, T, Hk, d, l, Q.device, stream)
    if workspace is None:
        workspace = _new((moda_bwd_workspace_bytes_gqa(B, T, H, Hk, d, l),), torch.uint8, Q.device, stream)
    _check(load().moda_attn_bwd_gqa_pm(_ptr(Q), _ptr(K), _ptr(V), _ptr(depth_kv_pm) if l > 0 else None,
                                       _ptr(O), _ptr(dO), _ptr(LSE), B, T, H, Hk, d, int(l), float(scale),
                                       _ptr(dQ), _ptr(dK), _ptr(dV), _ptr(d_depth_kv_pm) if l > 0 else None,
                                       _ptr(workspace), workspace.numel() * workspace.element_size(), _stream(stream)),
           "moda_attn_bwd_gqa_pm")
    return dQ, dK, dV, d_depth_kv_pm


def moda_kv_project_append(X, Wk, Wv, H_kv, cache=None, slot=0, store_kv=True, K_out=None, V_out=None, stream=None,
                           e4m3=False):
    """K, V [B,T,H_kv,d] = X [B,T,D_model] times the key / value projections Wk, Wv [H_kv d, D_model]; with ``cache`` the
    same launch writes them as depth slot ``slot``.  ``store_kv=False`` (FFN-side projection) writes the slot only.
    ``e4m3=True``: ``cache`` is an e4m3 cache (alloc_depth_cache_e4m3) and the call is moda_kv_project_append_e4m3."""
    if X.dim() != 3 or X.dtype != torch.bfloat16:
        raise ValueError("X must be a bf16 [B, T, D_model] tensor")
    B, T, Dm = X.shape
    n = Wk.shape[0]
    if Wk.shape != (n, Dm) or Wv.shape != (n, Dm) or n % H_kv or Wk.dtype != torch.bfloat16 or Wv.dtype != torch.bfloat16:
        raise ValueError("Wk, Wv must be bf16 [H_kv d, D_model] tensors matching X")
    d = n // H_kv
    if store_kv:
        K_out = _new((B, T, H_kv, d), torch.bfloat16, X.device, stream) if K_out is None else K_out
        V_out = _new((B, T, H_kv, d), torch.bfloat16, X.device, stream) if V_out is None else V_out
    else:
        K_out = V_out = None
    fn = load().moda_kv_project_append_e4m3 if e4m3 else load().moda_kv_project_append
    _check(fn(_ptr(X), _ptr(Wk), _ptr(Wv), B, T, Dm, int(H_kv), d, _ptr(K_out), _ptr(V_out),
              _ptr(cache), int(slot), _stream(stream)), "moda_kv_project_append_e4m3" if e4m3 else "moda_kv_project_append")
    return K_out, V_out


def moda_kv_project_append_e4m3(X, Wk, Wv, H_kv, cache=None, slot=0, store_kv=True, K_out=None, V_out=None, stream=None):
    """moda_kv_project_append with the slot written as e4m3 codes and row scales."""
    return moda_kv_project_append(X, Wk, Wv, H_kv, cache, slot, store_kv, K_out, V_out, stream, e4m3=True)


def moda_depth_slot_mass(Q, depth_kv, LSE, l, scale, H_kv=None, mass=None, workspace=None, stream=None):
    """mass [B,H,l] fp32: the probability that the rows of every query head give to each depth slot, summed over the
    positions (Q and LSE of the forward call; the bf16 row-interleaved cache it read)."""
    B, T, H, d = _bthd(Q, "Q")
    H_kv = H if H_kv is None else int(H_kv)
    if mass is None:
        mass = _new((B, H, int(l)), torch.float32, Q.device, stream)
    need = int(load().moda_depth_slot_mass_workspace_bytes(B, T, H, int(l)))
    if workspace is None:
        workspace = _new((max(need, 16),), torch.uint8, Q.device, stream)
    _check(load().moda_depth_slot_mass(_ptr(Q), _ptr(depth_kv) if l > 0 else None, _ptr(LSE), B, T, H, H_kv, d, int(l),
                                       float(scale), _ptr(mass), _ptr(workspace), workspace.numel() * workspace.element_size(),
                                       _stream(stream)), "moda_depth_slot_mass")
    return mass


def moda_attn_fwd(Q, K, V, depth_kv, l, scale, O=None, LSE=None, stream=None):
    """O [B,T,H,d] bf16 and LSE [B,H,T] fp32 of the MoDA operator (outputs allocated if not given)."""
    B, T, H, d = _bthd(Q, "Q")
    assert _bthd(K, "K") == (B, T, H, d) and _bthd(V, "V") == (B, T, H, d)
    if O is None:
        O = _new_like(Q, stream)
    if LSE is None:
        LSE = _new((B, H, T), torch.float32, Q.device, stream)
    _check(load().moda_attn_fwd(_ptr(Q), _ptr(K), _ptr(V), _ptr(depth_kv) if l > 0 else None,
                                B, T, H, d, int(l), float(scale), _ptr(O), _ptr(LSE), _stream(stream)),
           "moda_attn_fwd")
    return O, LSE


def moda_bwd_workspace_bytes(B, T, H, d, l) -> int:
    return int(load().moda_bwd_workspace_bytes(B, T, H, d, l))


def moda_attn_bwd(Q, K, V, depth_kv, O, dO, LSE, l, scale,
                  dQ=None, dK=None, dV=None, d_depth_kv=None, workspace=None, stream=None, stages=None):
    """dQ, dK, dV [B,T,H,d] bf16 and the depth gradients (cache layout, slots < l).

    With ``stages`` (a MODA_BWD_STAGE_* mask) the call goes through moda_attn_bwd_stages."""
    B, T, H, d = _bthd(Q, "Q")
    dQ = _new_like(Q, stream) if dQ is None else dQ
    dK = _new_like(Q, stream) if dK is None else dK
    dV = _new_like(Q, stream) if dV is None else dV
    if l > 0 and d_depth_kv is None:
        d_depth_kv = alloc_depth_cache(B, T, H, d, l, Q.device, stream)
    need = moda_bwd_workspace_bytes(B, T, H, d, l)
    if workspace is None:
        workspace = _new((need,), torch.uint8, Q.device, stream)
    args = [_ptr(Q), _ptr(K), _ptr(V), _ptr(depth_kv) if l > 0 else None,
            _ptr(O), _ptr(dO), _ptr(LSE), B, T, H, d, int(l), float(scale),
            _ptr(dQ), _ptr(dK), _ptr(dV), _ptr(d_depth_kv) if l > 0 else None,
            _ptr(workspace), workspace.numel() * workspace.element_size()]
    if stages is None:
        _check(load().moda_attn_bwd(*args, _stream(stream)), "moda_attn_bwd")
    else:
        _check(load().moda_attn_bwd_stages(*args, int(stages), _stream(stream)), "moda_attn_bwd_stages")
    return dQ, dK, dV, d_depth_kv


def moda_attn_bwd_stages(*args, stages, **kwargs):
    """moda_attn_bwd restricted to the launches selected by the ``stages`` bit mask."""
    return moda_attn_bwd(*args, stages=stages, **kwargs)


def moda_attn_bwd_static_scratch(Q, K, V, depth_kv, O, dO, LSE, l, scale, dQ, dK, dV, d_depth_kv=None, stream=None):
    """Backward for callers that cannot hand over a scratch buffer (a plug-in that only receives its
    tensors, a server that may not call cudaMalloc once it is running).  Same results as
    moda_attn_bwd; the per-row terms live in a 4 MiB array built into the library, so this call
    takes no workspace and allocates nothing -- which is why every output must be passed in.

    Limit: B*H*T <= MODA_STATIC_SCRATCH_ROWS (error -11 beyond it).  Calls on one device share that
    array: do not let two of them overlap on the GPU."""
    B, T, H, d = _bthd(Q, "Q")
    if l > 0 and d_depth_kv is None:
        raise ValueError("d_depth_kv must be provided: this entry point allocates nothing")
    _check(load().moda_attn_bwd_static_scratch(
        _ptr(Q), _ptr(K), _ptr(V), _ptr(depth_kv) if l > 0 else None, _ptr(O), _ptr(dO), _ptr(LSE),
        B, T, H, d, int(l), float(scale), _ptr(dQ), _ptr(dK), _ptr(dV), _ptr(d_depth_kv) if l > 0 else None,
        _stream(stream)), "moda_attn_bwd_static_scratch")
    return dQ, dK, dV, d_depth_kv


def moda_bwd_workspace_bytes_gqa(B, T, H, H_kv, d, l) -> int:
    return int(load().moda_bwd_workspace_bytes_gqa(B, T, H, H_kv, d, l))


def _gqa_shapes(Q, K, V):
    B, T, H, d = _bthd(Q, "Q")
    Bk, Tk, Hk, dk = _bthd(K, "K")
    if (Bk, Tk, dk) != (B, T, d) or _bthd(V, "V") != (B, T, Hk, d):
        raise ValueError("K and V must be bf16 [B, T, H_kv, d] tensors matching Q's B, T and d")
    return B, T, H, Hk, d


def moda_attn_fwd_gqa(Q, K, V, depth_kv, l, scale, O=None, LSE=None, stream=None):
    """Grouped-query forward: Q [B,T,H,d], K, V [B,T,H_kv,d], depth cache with H_kv heads.

    Returns O [B,T,H,d] bf16 and LSE [B,H,T] fp32 (allocated if not given)."""
    B, T, H, Hk, d = _gqa_shapes(Q, K, V)
    if O is None:
        O = _new_like(Q, stream)
    if LSE is None:
        LSE = _new((B, H, T), torch.float32, Q.device, stream)
    _check(load().moda_attn_fwd_gqa(_ptr(Q), _ptr(K), _ptr(V), _ptr(depth_kv) if l > 0 else None,
                                    B, T, H, Hk, d, int(l), float(scale), _ptr(O), _ptr(LSE), _stream(stream)),
           "moda_attn_fwd_gqa")
    return O, LSE


def moda_attn_fwd_append(Q, K, V, depth_kv, l, scale, append_cache, append_slot, O=None, LSE=None, stream=None):
    """moda_attn_fwd_gqa that also stores K, V into slot ``append_slot`` of ``append_cache`` (cache layout, H_kv heads)
    in the same launch: the depth stream's write step without a separate pass over K and V."""
    B, T, H, Hk, d = _gqa_shapes(Q, K, V)
    if O is None:
        O = _new_like(Q, stream)
    if LSE is None:
        LSE = _new((B, H, T), torch.float32, Q.device, stream)
    _check(load().moda_attn_fwd_append(_ptr(Q), _ptr(K), _ptr(V), _ptr(depth_kv) if l > 0 else None,
                                       B, T, H, Hk, d, int(l), float(scale), _ptr(O), _ptr(LSE),
                                       _ptr(append_cache), int(append_slot), _stream(stream)),
           "moda_attn_fwd_append")
    return O, LSE


def moda_attn_bwd_gqa(Q, K, V, depth_kv, O, dO, LSE, l, scale,
                      dQ=None, dK=None, dV=None, d_depth_kv=None, workspace=None, stream=None, stages=None):
    """Grouped-query backward: dQ [B,T,H,d], dK, dV [B,T,H_kv,d], depth gradients (cache layout, H_kv heads).

    With ``stages`` (a MODA_BWD_STAGE_* mask) the call goes through moda_attn_bwd_gqa_stages."""
    B, T, H, Hk, d = _gqa_shapes(Q, K, V)
    dQ = _new_like(Q, stream) if dQ is None else dQ
    dK = _new_like(K, stream) if dK is None else dK
    dV = _new_like(V, stream) if dV is None else dV
    if l > 0 and d_depth_kv is None:
        d_depth_kv = alloc_depth_cache(B, T, Hk, d, l, Q.device, stream)
    if workspace is None:
        workspace = _new((moda_bwd_workspace_bytes_gqa(B, T, H, Hk, d, l),), torch.uint8, Q.device, stream)
    args = [_ptr(Q), _ptr(K), _ptr(V), _ptr(depth_kv) if l > 0 else None,
            _ptr(O), _ptr(dO), _ptr(LSE), B, T, H, Hk, d, int(l), float(scale),
            _ptr(dQ), _ptr(dK), _ptr(dV), _ptr(d_depth_kv) if l > 0 else None,
            _ptr(workspace), workspace.numel() * workspace.element_size()]
    if stages is None:
        _check(load().moda_attn_bwd_gqa(*args, _stream(stream)), "moda_attn_bwd_gqa")
    else:
        _check(load().moda_attn_bwd_gqa_stages(*args, int(stages), _stream(stream)), "moda_attn_bwd_gqa_stages")
    return dQ, dK, dV, d_depth_kv


def moda_attn_bwd_gqa_stages(*args, stages, **kwargs):
    """moda_attn_bwd_gqa restricted to the launches selected by the ``stages`` bit mask."""
    return moda_attn_bwd_gqa(*args, stages=stages, **kwargs)


def moda_decode_workspace_bytes(B, H, d) -> int:
    return int(load().moda_decode_workspace_bytes(B, H, d))


def moda_attn_decode(q, K, V, depth_kv_token, T_kv, l, scale, O=None, LSE=None, workspace=None, stream=None):
    """Decode step: q [B,H,d], K, V [B,T_cap,H_kv,d] (positions < T_kv read), depth pairs of the token
    [l,B,H_kv,2,d] (key row, value row).  Returns O [B,H,d] bf16 and LSE [B,H] fp32."""
    if q.dtype != torch.bfloat16 or q.dim() != 3:
        raise ValueError("q must be a bf16 [B, H, d] tensor")
    B, H, d = q.shape
    Bk, T_cap, Hk, dk = _bthd(K, "K")
    if (Bk, dk) != (B, d) or tuple(V.shape) != tuple(K.shape) or V.dtype != torch.bfloat16:
        raise ValueError("K and V must be bf16 [B, T_cap, H_kv, d] tensors matching q's B and d")
    if l > 0 and (depth_kv_token is None or tuple(depth_kv_token.shape) != (l, B, Hk, 2, d)
                  or depth_kv_token.dtype != torch.bfloat16):
        raise ValueError("depth_kv_token must be a bf16 [l, B, H_kv, 2, d] tensor")
    if O is None:
        O = _new_like(q, stream)
    if LSE is None:
        LSE = _new((B, H), torch.float32, q.device, stream)
    if workspace is None:
        workspace = _new((moda_decode_workspace_bytes(B, H, d),), torch.uint8, q.device, stream)
    _check(load().moda_attn_decode(_ptr(q), _ptr(K), _ptr(V), _ptr(depth_kv_token) if l > 0 else None,
                                   B, int(T_kv), T_cap, H, Hk, d, int(l), float(scale), _ptr(O), _ptr(LSE),
                                   _ptr(workspace), workspace.numel() * workspace.element_size(), _stream(stream)),
           "moda_attn_decode")
    return O, LSE


def moda_attn_fwd_prefill(Q, K, V, depth_kv, l, scale, O=None, LSE=None, stream=None):
    """Prefill with a cache: Q [B,T_q,H,d] (the newest positions), K, V [B,T_kv,H_kv,d] with T_kv >= T_q,
    depth cache over the T_q positions.  Returns O [B,T_q,H,d] bf16 and LSE [B,H,T_q] fp32."""
    B, T_q, H, d = _bthd(Q, "Q")
    Bk, T_kv, Hk, dk = _bthd(K, "K")
    if (Bk, dk) != (B, d) or _bthd(V, "V") != (B, T_kv, Hk, d):
        raise ValueError("K and V must be bf16 [B, T_kv, H_kv, d] tensors matching Q's B and d")
    if O is None:
        O = _new_like(Q, stream)
    if LSE is None:
        LSE = _new((B, H, T_q), torch.float32, Q.device, stream)
    _check(load().moda_attn_fwd_prefill(_ptr(Q), _ptr(K), _ptr(V), _ptr(depth_kv) if l > 0 else None,
                                        B, T_q, T_kv, H, Hk, d, int(l), float(scale), _ptr(O), _ptr(LSE),
                                        _stream(stream)), "moda_attn_fwd_prefill")
    return O, LSE


def _decode_outputs(q, O, LSE, workspace, stream):
    B, H, d = q.shape
    if O is None:
        O = _new_like(q, stream)
    if LSE is None:
        LSE = _new((B, H), torch.float32, q.device, stream)
    if workspace is None:
        workspace = _new((moda_decode_workspace_bytes(B, H, d),), torch.uint8, q.device, stream)
    return O, LSE, workspace


def _int32(t, name, shape):
    if t.dtype != torch.int32 or tuple(t.shape) != tuple(shape):
        raise ValueError(f"{name} must be an int32 tensor of shape {tuple(shape)}")
    return t


def moda_attn_decode_varlen(q, K, V, seq_lens, depth_kv_token, max_seq_len, l, scale, O=None, LSE=None,
                            workspace=None, stream=None):
    """Decode step with a length per sequence: seq_lens int32 [B] (device), each in [1, max_seq_len]."""
    B, H, d = q.shape
    _, T_cap, Hk, _ = _bthd(K, "K")
    _int32(seq_lens, "seq_lens", (B,))
    O, LSE, workspace = _decode_outputs(q, O, LSE, workspace, stream)
    _check(load().moda_attn_decode_varlen(_ptr(q), _ptr(K), _ptr(V), _ptr(seq_lens), _ptr(depth_kv_token) if l > 0 else None,
                                          B, int(max_seq_len), T_cap, H, Hk, d, int(l), float(scale), _ptr(O), _ptr(LSE),
                                          _ptr(workspace), workspace.numel() * workspace.element_size(), _stream(stream)),
           "moda_attn_decode_varlen")
    return O, LSE


def moda_attn_decode_paged(q, K_pages, V_pages, block_table, seq_lens, depth_kv_token, max_seq_len, l, scale,
                           O=None, LSE=None, workspace=None, stream=None):
    """Decode step over a paged KV cache: K_pages, V_pages [num_pages, page_size, H_kv, d]; block_table int32
    [B, max_blocks]; seq_lens int32 [B]."""
    B, H, d = q.shape
    num_pages, page_size, Hk, _ = _bthd(K_pages, "K_pages")
    _int32(seq_lens, "seq_lens", (B,))
    if block_table.dtype != torch.int32 or block_table.dim() != 2 or block_table.shape[0] != B:
        raise ValueError("block_table must be an int32 [B, max_blocks] tensor")
    O, LSE, workspace = _decode_outputs(q, O, LSE, workspace, stream)
    _check(load().moda_attn_decode_paged(_ptr(q), _ptr(K_pages), _ptr(V_pages), _ptr(block_table), _ptr(seq_lens),
                                         _ptr(depth_kv_token) if l > 0 else None,
                                         B, int(max_seq_len), page_size, num_pages, block_table.shape[1], H, Hk, d, int(l),
                                         float(scale), _ptr(O), _ptr(LSE), _ptr(workspace),
                                         workspace.numel() * workspace.element_size(), _stream(stream)),
           "moda_attn_decode_paged")
    return O, LSE
