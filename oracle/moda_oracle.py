"""ctypes front end of the fp64 CPU oracle (``moda_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, by ``__graft_entry__.smoke()`` and by
the CPU-baseline / ``--impl reference`` legs of ``bench.py``.  Nothing in the product
package imports this module, and this module imports nothing from the product package.

All arrays are numpy float64, C-contiguous, in the logical layouts of the paper's
statement of the operator (Sec. 2.2, Alg. 1 input/output lines):

    Q, K, V, O, dO, dQ, dK, dV : [B, T, H, d]
    Kd, Vd, dKd, dVd           : [l, B, T, H, d]   (depth slot i = layer i's K, V)
    LSE                        : [B, H, T]         (natural log, over sequence+depth keys)
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "moda_oracle.c")
_LIB = os.path.join(_HERE, "libmoda_oracle.so")
_lock = threading.Lock()
_lib = None

_dp = ctypes.POINTER(ctypes.c_double)
_ip = ctypes.POINTER(ctypes.c_int)


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain -O2, OpenMP; no fast-math). Returns the .so path."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + f".tmp{os.getpid()}"
            cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"]
            subprocess.run(cmd, check=True)
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.moda_oracle_threads.restype = ctypes.c_int
        lib.moda_oracle_fwd.restype = ctypes.c_int
        lib.moda_oracle_fwd.argtypes = [_dp] * 5 + [ctypes.c_int] * 5 + [ctypes.c_double, _dp, _dp]
        lib.moda_oracle_fwd_rows.restype = ctypes.c_int
        lib.moda_oracle_fwd_rows.argtypes = (
            [_dp] * 5 + [ctypes.c_int] * 5 + [ctypes.c_double, _ip, ctypes.c_int, _dp, _dp]
        )
        lib.moda_oracle_bwd.restype = ctypes.c_int
        lib.moda_oracle_bwd.argtypes = [_dp] * 6 + [ctypes.c_int] * 5 + [ctypes.c_double] + [_dp] * 5
        lib.moda_oracle_bwd_rows.restype = ctypes.c_int
        lib.moda_oracle_bwd_rows.argtypes = (
            [_dp] * 6 + [ctypes.c_int] * 5 + [ctypes.c_double, _ip, ctypes.c_int, _ip, ctypes.c_int, ctypes.c_int]
            + [_dp] * 5
        )
        lib.moda_oracle_base_time.restype = ctypes.c_int
        lib.moda_oracle_base_time.argtypes = [ctypes.c_int, ctypes.c_int]
        lib.moda_oracle_fwd_gqa.restype = ctypes.c_int
        lib.moda_oracle_fwd_gqa.argtypes = [_dp] * 5 + [ctypes.c_int] * 6 + [ctypes.c_double, _dp, _dp]
        lib.moda_oracle_bwd_gqa.restype = ctypes.c_int
        lib.moda_oracle_bwd_gqa.argtypes = [_dp] * 6 + [ctypes.c_int] * 6 + [ctypes.c_double] + [_dp] * 5
        _lib = lib
    return _lib


def threads() -> int:
    """Number of OpenMP threads the oracle will use."""
    return int(_load().moda_oracle_threads())


def _f64(a, shape):
    a = np.ascontiguousarray(a, dtype=np.float64)
    if a.shape != tuple(shape):
        raise ValueError(f"expected shape {tuple(shape)}, got {a.shape}")
    return a


def _ptr(a):
    return a.ctypes.data_as(_dp)


def _prep(Q, K, V, Kd, Vd):
    Q = np.ascontiguousarray(Q, dtype=np.float64)
    if Q.ndim != 4:
        raise ValueError("Q must be [B, T, H, d]")
    B, T, H, d = Q.shape
    K = _f64(K, (B, T, H, d))
    V = _f64(V, (B, T, H, d))
    l = 0 if Kd is None else int(np.shape(Kd)[0])
    if l == 0:
        Kd = np.zeros((0, B, T, H, d))
        Vd = np.zeros((0, B, T, H, d))
    Kd = _f64(Kd, (l, B, T, H, d))
    Vd = _f64(Vd, (l, B, T, H, d))
    return Q, K, V, Kd, Vd, (B, T, H, d, l)


def forward(Q, K, V, Kd, Vd, scale):
    """O [B,T,H,d] and LSE [B,H,T] of the MoDA operator (definition, fp64)."""
    Q, K, V, Kd, Vd, (B, T, H, d, l) = _prep(Q, K, V, Kd, Vd)
    O = np.empty((B, T, H, d))
    LSE = np.empty((B, H, T))
    rc = _load().moda_oracle_fwd(_ptr(Q), _ptr(K), _ptr(V), _ptr(Kd), _ptr(Vd),
                                 B, T, H, d, l, float(scale), _ptr(O), _ptr(LSE))
    if rc != 0:
        raise MemoryError("oracle scratch allocation failed")
    return O, LSE


def forward_rows(Q, K, V, Kd, Vd, scale, rows):
    """Forward for sampled rows only. ``rows`` is an int array [n, 3] of (b, h, t).

    Returns O_rows [n, d] and LSE_rows [n]."""
    Q, K, V, Kd, Vd, (B, T, H, d, l) = _prep(Q, K, V, Kd, Vd)
    rows = np.ascontiguousarray(rows, dtype=np.int32).reshape(-1, 3)
    if rows.size and not ((rows >= 0).all() and (rows[:, 0] < B).all()
                          and (rows[:, 1] < H).all() and (rows[:, 2] < T).all()):
        raise ValueError("row index out of range")
    n = rows.shape[0]
    O = np.empty((n, d))
    LSE = np.empty((n,))
    rc = _load().moda_oracle_fwd_rows(_ptr(Q), _ptr(K), _ptr(V), _ptr(Kd), _ptr(Vd),
                                      B, T, H, d, l, float(scale),
                                      rows.ctypes.data_as(_ip), n, _ptr(O), _ptr(LSE))
    if rc != 0:
        raise MemoryError("oracle scratch allocation failed")
    return O, LSE


def backward(Q, K, V, Kd, Vd, dO, scale):
    """dQ, dK, dV [B,T,H,d] and dKd, dVd [l,B,T,H,d] for upstream gradient dO."""
    Q, K, V, Kd, Vd, (B, T, H, d, l) = _prep(Q, K, V, Kd, Vd)
    dO = _f64(dO, (B, T, H, d))
    dQ = np.empty((B, T, H, d))
    dK = np.empty((B, T, H, d))
    dV = np.empty((B, T, H, d))
    dKd = np.empty((l, B, T, H, d))
    dVd = np.empty((l, B, T, H, d))
    rc = _load().moda_oracle_bwd(_ptr(Q), _ptr(K), _ptr(V), _ptr(Kd), _ptr(Vd), _ptr(dO),
                                 B, T, H, d, l, float(scale),
                                 _ptr(dQ), _ptr(dK), _ptr(dV), _ptr(dKd), _ptr(dVd))
    if rc != 0:
        raise MemoryError("oracle scratch allocation failed")
    return dQ, dK, dV, dKd, dVd


def backward_rows(Q, K, V, Kd, Vd, dO, scale, qrows, krows=None, t_start=None):
    """Backward for sampled rows.

    ``qrows`` [n_q, 3] of (b, h, t): returns dQ_rows [n_q, d], dKd_rows, dVd_rows [n_q, l, d].
    ``krows`` [n_k, 3] of (b, h, j), all j >= ``t_start`` (default: the smallest j): returns
    dK_rows, dV_rows [n_k, d].  The cost of the key rows is (T - t_start) forward rows per head."""
    Q, K, V, Kd, Vd, (B, T, H, d, l) = _prep(Q, K, V, Kd, Vd)
    dO = _f64(dO, (B, T, H, d))
    qrows = np.ascontiguousarray(qrows if qrows is not None else np.zeros((0, 3)), dtype=np.int32).reshape(-1, 3)
    krows = np.ascontiguousarray(krows if krows is not None else np.zeros((0, 3)), dtype=np.int32).reshape(-1, 3)
    for rows in (qrows, krows):
        if rows.size and not ((rows >= 0).all() and (rows[:, 0] < B).all()
                              and (rows[:, 1] < H).all() and (rows[:, 2] < T).all()):
            raise ValueError("row index out of range")
    if t_start is None:
        t_start = int(krows[:, 2].min()) if krows.size else T
    n_q, n_k = qrows.shape[0], krows.shape[0]
    dQ = np.empty((n_q, d)); dKd = np.empty((n_q, l, d)); dVd = np.empty((n_q, l, d))
    dK = np.empty((n_k, d)); dV = np.empty((n_k, d))
    rc = _load().moda_oracle_bwd_rows(_ptr(Q), _ptr(K), _ptr(V), _ptr(Kd), _ptr(Vd), _ptr(dO),
                                      B, T, H, d, l, float(scale),
                                      qrows.ctypes.data_as(_ip), n_q, krows.ctypes.data_as(_ip), n_k, int(t_start),
                                      _ptr(dQ), _ptr(dKd), _ptr(dVd), _ptr(dK), _ptr(dV))
    if rc == -2:
        raise ValueError("every key row must be >= t_start")
    if rc != 0:
        raise MemoryError("oracle scratch allocation failed")
    return dQ, dKd, dVd, dK, dV


# ---------------------------------------------------------------------------------------
# Grouped-query form (Sec. 3, group-aware depth KV): Q, O, dO, dQ have Hq heads; K, V and the
# depth K, V have Hk = Hq / G heads; query head hq uses KV head hq // G.
# ---------------------------------------------------------------------------------------
def base_time(i_q: int, G: int) -> int:
    """Base-time index of flattened query row i_q = t * G + g."""
    return int(_load().moda_oracle_base_time(int(i_q), int(G)))


def _prep_gqa(Q, K, V, Kd, Vd):
    Q = np.ascontiguousarray(Q, dtype=np.float64)
    K = np.ascontiguousarray(K, dtype=np.float64)
    if Q.ndim != 4 or K.ndim != 4:
        raise ValueError("Q must be [B, T, Hq, d] and K [B, T, Hk, d]")
    B, T, Hq, d = Q.shape
    Hk = K.shape[2]
    if K.shape != (B, T, Hk, d) or Hk < 1 or Hq % Hk:
        raise ValueError("K must be [B, T, Hk, d] with Hk dividing Hq")
    V = _f64(V, (B, T, Hk, d))
    l = 0 if Kd is None else int(np.shape(Kd)[0])
    if l == 0:
        Kd = np.zeros((0, B, T, Hk, d)); Vd = np.zeros((0, B, T, Hk, d))
    Kd = _f64(Kd, (l, B, T, Hk, d)); Vd = _f64(Vd, (l, B, T, Hk, d))
    return Q, K, V, Kd, Vd, (B, T, Hq, Hk, d, l)


def forward_gqa(Q, K, V, Kd, Vd, scale):
    """O [B,T,Hq,d] and LSE [B,Hq,T] of the grouped-query MoDA operator (definition, fp64)."""
    Q, K, V, Kd, Vd, (B, T, Hq, Hk, d, l) = _prep_gqa(Q, K, V, Kd, Vd)
    O = np.empty((B, T, Hq, d)); LSE = np.empty((B, Hq, T))
    rc = _load().moda_oracle_fwd_gqa(_ptr(Q), _ptr(K), _ptr(V), _ptr(Kd), _ptr(Vd),
                                     B, T, Hq, Hk, d, l, float(scale), _ptr(O), _ptr(LSE))
    if rc != 0:
        raise MemoryError("oracle scratch allocation failed")
    return O, LSE


def backward_gqa(Q, K, V, Kd, Vd, dO, scale):
    """dQ [B,T,Hq,d], dK, dV [B,T,Hk,d], dKd, dVd [l,B,T,Hk,d] (sums over the heads of a group)."""
    Q, K, V, Kd, Vd, (B, T, Hq, Hk, d, l) = _prep_gqa(Q, K, V, Kd, Vd)
    dO = _f64(dO, (B, T, Hq, d))
    dQ = np.empty((B, T, Hq, d)); dK = np.empty((B, T, Hk, d)); dV = np.empty((B, T, Hk, d))
    dKd = np.empty((l, B, T, Hk, d)); dVd = np.empty((l, B, T, Hk, d))
    rc = _load().moda_oracle_bwd_gqa(_ptr(Q), _ptr(K), _ptr(V), _ptr(Kd), _ptr(Vd), _ptr(dO),
                                     B, T, Hq, Hk, d, l, float(scale),
                                     _ptr(dQ), _ptr(dK), _ptr(dV), _ptr(dKd), _ptr(dVd))
    if rc != 0:
        raise MemoryError("oracle scratch allocation failed")
    return dQ, dK, dV, dKd, dVd


# ---------------------------------------------------------------------------------------
# Decode step (T_q = 1): the newest token of every sequence attends to the T_kv sequence keys of
# this layer's KV cache (its own included) and to its own l depth key/value pairs, the
# 2 l H_k d values per token of the paper's complexity table (Table 1, "decoding cache").
# Written straight from the definition in numpy float64: for the last position the causal mask
# of Eq. 2 admits every cached key, so the row is one plain softmax over T_kv + l keys.
# ---------------------------------------------------------------------------------------
def decode_gqa(q, K, V, kd, vd, scale):
    """o [B,Hq,d] and lse [B,Hq] for q [B,Hq,d], K, V [B,T_kv,Hk,d], kd, vd [l,B,Hk,d] (or None)."""
    q = np.ascontiguousarray(q, dtype=np.float64)
    K = np.ascontiguousarray(K, dtype=np.float64)
    V = np.ascontiguousarray(V, dtype=np.float64)
    if q.ndim != 3 or K.ndim != 4 or V.shape != K.shape:
        raise ValueError("q must be [B, Hq, d]; K, V [B, T_kv, Hk, d]")
    B, Hq, d = q.shape
    _, Tkv, Hk, _ = K.shape
    if K.shape[0] != B or K.shape[3] != d or Hk < 1 or Hq % Hk or Tkv < 1:
        raise ValueError("K must be [B, T_kv >= 1, Hk, d] with Hk dividing Hq")
    G = Hq // Hk
    l = 0 if kd is None else int(np.shape(kd)[0])
    kd = np.zeros((0, B, Hk, d)) if l == 0 else _f64(kd, (l, B, Hk, d))
    vd = np.zeros((0, B, Hk, d)) if l == 0 else _f64(vd, (l, B, Hk, d))
    o = np.empty((B, Hq, d)); lse = np.empty((B, Hq))
    for b in range(B):
        for h in range(Hq):
            hk = h // G
            keys = np.concatenate([K[b, :, hk, :], kd[:, b, hk, :]], axis=0)      # [T_kv + l, d]
            vals = np.concatenate([V[b, :, hk, :], vd[:, b, hk, :]], axis=0)
            s = (keys @ q[b, h]) * float(scale)
            m = s.max()
            p = np.exp(s - m)
            z = p.sum()
            o[b, h] = (p / z) @ vals
            lse[b, h] = m + np.log(z)
    return o, lse


# ---------------------------------------------------------------------------------------
# Prefill with a cache (1 <= T_q <= T_kv): the T_q newest positions of a sequence whose layer
# already caches T_kv - T_q earlier keys.  Query row i (0-based among the new positions) sits at
# absolute position i + (T_kv - T_q): the causal mask of Eq. 2 admits sequence keys
# j <= i + (T_kv - T_q), and its depth keys are those stored for its own position (slot arrays
# are indexed by the new positions only).  Definition written out in numpy float64.
# ---------------------------------------------------------------------------------------
def forward_prefill_gqa(Q, K, V, Kd, Vd, scale):
    """O [B,T_q,Hq,d], LSE [B,Hq,T_q] for Q [B,T_q,Hq,d], K, V [B,T_kv,Hk,d], Kd, Vd [l,B,T_q,Hk,d] (or None)."""
    Q = np.ascontiguousarray(Q, dtype=np.float64)
    K = np.ascontiguousarray(K, dtype=np.float64)
    V = np.ascontiguousarray(V, dtype=np.float64)
    if Q.ndim != 4 or K.ndim != 4 or V.shape != K.shape:
        raise ValueError("Q must be [B, T_q, Hq, d]; K, V [B, T_kv, Hk, d]")
    B, Tq, Hq, d = Q.shape
    _, Tkv, Hk, _ = K.shape
    if K.shape[0] != B or K.shape[3] != d or Hk < 1 or Hq % Hk or Tq < 1 or Tkv < Tq:
        raise ValueError("need T_kv >= T_q >= 1 and Hk dividing Hq")
    G = Hq // Hk
    off = Tkv - Tq
    l = 0 if Kd is None else int(np.shape(Kd)[0])
    Kd = np.zeros((0, B, Tq, Hk, d)) if l == 0 else _f64(Kd, (l, B, Tq, Hk, d))
    Vd = np.zeros((0, B, Tq, Hk, d)) if l == 0 else _f64(Vd, (l, B, Tq, Hk, d))
    O = np.empty((B, Tq, Hq, d)); LSE = np.empty((B, Hq, Tq))
    for b in range(B):
        for h in range(Hq):
            hk = h // G
            for i in range(Tq):
                n_seq = i + off + 1                                        # keys 0 .. i + off
                keys = np.concatenate([K[b, :n_seq, hk, :], Kd[:, b, i, hk, :]], axis=0)
                vals = np.concatenate([V[b, :n_seq, hk, :], Vd[:, b, i, hk, :]], axis=0)
                s = (keys @ Q[b, i, h]) * float(scale)
                m = s.max()
                p = np.exp(s - m)
                z = p.sum()
                O[b, i, h] = (p / z) @ vals
                LSE[b, h, i] = m + np.log(z)
    return O, LSE


# ---------------------------------------------------------------------------------------
# Lower-precision depth cache (the paper's Discussion names bounded / cheaper depth-KV caching
# as a direction and gives no algorithm).  Reading taken: every depth key row and every depth value
# row (the d features of one slot, position and head) is stored as 8-bit floats of the e4m3 kind
# (1 sign, 4 exponent, 3 mantissa bits, bias 7, no infinities, largest finite value 448) with one
# fp32 scale per row, scale = max|x| / 448; the operator is then the Sec. 2.2 operator on the
# DEQUANTISED depth keys and values.  The decisions that pick an 8-bit code are taken in fp32 (the
# scale, the division x / scale, both rounded to nearest) so that any implementation that follows
# the same steps picks the same codes; the dequantised value code * scale is exact in float64.
# ---------------------------------------------------------------------------------------
E4M3_MAX = 448.0


def e4m3_decode_table():
    """The 256 values of the e4m3 format, from its definition (code 0x7f / 0xff, the NaN patterns, as nan)."""
    vals = np.empty(256)
    for code in range(256):
        sign = -1.0 if code & 0x80 else 1.0
        e, m = (code >> 3) & 0xF, code & 0x7
        if e == 0xF and m == 0x7:
            vals[code] = np.nan
        elif e == 0:
            vals[code] = sign * (m / 8.0) * 2.0 ** -6          # subnormals
        else:
            vals[code] = sign * (1.0 + m / 8.0) * 2.0 ** (e - 7)
    return vals


def e4m3_round(y):
    """Codes (uint8) of float32 values rounded to the nearest e4m3 value, ties to the even mantissa, saturating at
    +-448.  Written from the format: in the binade 2^e the representable values are 2^(e-3) apart, below 2^-6 they
    are 2^-9 apart."""
    y = np.asarray(y, dtype=np.float32)
    a = np.abs(y).astype(np.float64)
    e = np.floor(np.log2(np.maximum(a, 2.0 ** -6)))             # binade of a (subnormals share the step of 2^-6)
    step = 2.0 ** (e - 3)
    q = np.rint(a / step) * step                                # rint: round half to even; a / step is exact (power of two)
    q = np.minimum(q, E4M3_MAX)
    # encode q (now exactly representable)
    qe = np.floor(np.log2(np.maximum(q, 2.0 ** -6)))
    is_sub = q < 2.0 ** -6
    mant = np.where(is_sub, np.rint(q / 2.0 ** -9), np.rint((q / 2.0 ** qe - 1.0) * 8.0)).astype(np.int64)
    expf = np.where(is_sub, 0, qe + 7).astype(np.int64)
    code = (expf << 3) | mant
    code = np.where(np.signbit(y), code | 0x80, code)
    return code.astype(np.uint8)


def quantize_e4m3_rows(X):
    """Per-row e4m3 quantisation of X [..., d]: returns (codes uint8 [..., d], scale float32 [...])."""
    X32 = np.asarray(X, dtype=np.float32)
    amax = np.max(np.abs(X32), axis=-1)
    scale = np.where(amax > 0, amax / np.float32(E4M3_MAX), np.float32(1.0)).astype(np.float32)   # fp32 division
    y = (X32 / scale[..., None]).astype(np.float32)                                                # fp32 division
    return e4m3_round(y), scale


def dequantize_e4m3_rows(codes, scale):
    """float64 values code * scale of what quantize_e4m3_rows stored."""
    return e4m3_decode_table()[np.asarray(codes, dtype=np.uint8)] * np.asarray(scale, dtype=np.float64)[..., None]


# ---------------------------------------------------------------------------------------
# "Write" step with its projection (Sec. 2.1, Q / K / V = X W; Sec. 2.2, the write step: a layer's key-value pair is
# appended to the depth stream, an FFN layer obtains its pair through a KV projection of its input).
# The definition written out with the library's float64 matrix product.  Weights are passed as the transposes of
# the paper's W_K, W_V, i.e. one row per output feature: Wk, Wv [H_k d, D].
# ---------------------------------------------------------------------------------------
def project_kv(X, Wk, Wv, H_k):
    """K, V [B, T, H_k, d] = X [B, T, D] times the key / value projections (float64)."""
    X = np.asarray(X, dtype=np.float64)
    Wk = np.asarray(Wk, dtype=np.float64)
    Wv = np.asarray(Wv, dtype=np.float64)
    B, T, D = X.shape
    n = Wk.shape[0]
    if Wk.shape != (n, D) or Wv.shape != (n, D) or n % H_k:
        raise ValueError("Wk, Wv must be [H_k d, D] matching X [B, T, D]")
    K = np.matmul(X, Wk.T).reshape(B, T, H_k, n // H_k)
    V = np.matmul(X, Wv.T).reshape(B, T, H_k, n // H_k)
    return K, V


# ---------------------------------------------------------------------------------------
# Attention mass on the depth slots (Sec. 2.2: the probabilities of the one softmax over sequence and depth keys;
# the paper's attention analysis looks at how much probability heads give to depth slots, and its discussion of a
# bounded slot buffer keeps the entries of highest utility).  For slot i of query head hq:
#     mass[b, hq, i] = sum_t  exp( scale <q_t, kd_i[t]> - LSE_t )
# i.e. the depth probabilities R_i(t) of the definition, summed over the positions.  LSE is the operator's own
# output (forward / forward_gqa), so the sequence keys enter only through it.  Plain numpy float64.
# ---------------------------------------------------------------------------------------
def depth_slot_mass(Q, Kd, LSE, scale):
    """mass [B, Hq, l] from Q [B, T, Hq, d], depth keys Kd [l, B, T, Hk, d] and LSE [B, Hq, T] (float64)."""
    Q = np.asarray(Q, dtype=np.float64)
    Kd = np.asarray(Kd, dtype=np.float64)
    LSE = np.asarray(LSE, dtype=np.float64)
    B, T, Hq, d = Q.shape
    l = Kd.shape[0]
    Hk = Kd.shape[3] if l else 1
    if l and (Kd.shape != (l, B, T, Hk, d) or Hq % Hk):
        raise ValueError("Kd must be [l, B, T, Hk, d] with Hk dividing Hq")
    if LSE.shape != (B, Hq, T):
        raise ValueError("LSE must be [B, Hq, T]")
    mass = np.zeros((B, Hq, l))
    G = Hq // Hk
    for hq in range(Hq):
        for i in range(l):
            u = scale * np.einsum("btd,btd->bt", Q[:, :, hq, :], Kd[i, :, :, hq // G, :])      # [B, T]
            mass[:, hq, i] = np.exp(u - LSE[:, hq, :]).sum(axis=1)
    return mass
