"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol the
header declares, and rejects bad arguments before touching a device."""
import ctypes
import os
import re

import pytest

import paper_2603_15619_b200 as moda
from paper_2603_15619_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "moda.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(moda_[a-z_0-9]+)\s*\(", text)))


def test_library_loads_and_exports_every_declared_symbol():
    lib = binding.load()
    names = declared_symbols()
    assert set(names) == set(binding.SYMBOLS), (names, binding.SYMBOLS)
    for n in names:
        assert hasattr(lib, n), n
    assert moda.moda_version() >= 100


def test_strerror_covers_all_codes():
    for code in range(0, -14, -1):
        assert binding.strerror(code) != "unknown error code"
    assert binding.strerror(-99) == "unknown error code"


def test_size_queries_are_host_arithmetic():
    # cache[slot][b][h][tile][kv][chunk][row][8] with 128-row tiles, bf16
    assert moda.moda_depth_cache_bytes(1, 256, 2, 64, 4) == 4 * 1 * 2 * 2 * 2 * 128 * 64 * 2
    assert moda.moda_depth_cache_bytes(2, 129, 3, 128, 1) == 2 * 3 * 2 * 2 * 128 * 128 * 2
    assert moda.moda_depth_cache_bytes(1, 256, 2, 96, 4) == 0      # unsupported head width
    assert moda.moda_depth_cache_bytes(1, 256, 2, 64, 257) == 0    # more than 256 slots
    assert moda.moda_depth_cache_bytes(1, 0, 2, 64, 1) == 0
    assert moda.moda_bwd_workspace_bytes(2, 100, 3, 64, 0) >= 2 * 3 * 100 * 4
    assert moda.moda_bwd_workspace_bytes(2, 100, 3, 64, 0) % 16 == 0


def test_argument_validation_rejects_before_any_launch():
    lib = binding.load()
    vp = ctypes.c_void_p
    p = vp(4096)                        # aligned, non-null, never dereferenced: validation fails first
    odd = vp(4100)
    fwd = lambda *a: lib.moda_attn_fwd(*a)
    base = dict(B=1, T=128, H=1, d=64, l=0)

    def call(Q=p, K=p, V=p, dkv=None, O=p, LSE=p, scale=0.125, **kw):
        a = dict(base, **kw)
        return fwd(Q, K, V, dkv, a["B"], a["T"], a["H"], a["d"], a["l"], ctypes.c_float(scale), O, LSE, None)

    assert call(B=0) == -3 and call(T=0) == -3 and call(H=-1) == -3
    assert call(d=96) == -4
    assert call(l=-1) == -5 and call(l=257) == -5
    assert call(Q=None) == -1 and call(O=None) == -1 and call(LSE=None) == -1
    assert call(l=2, dkv=None) == -1
    assert call(K=odd) == -2
    assert lib.moda_depth_cache_append(p, 1, 128, 1, 64, 256, p, p, None) == -6
    assert lib.moda_depth_cache_append(p, 1, 128, 1, 64, -1, p, p, None) == -6
    assert lib.moda_depth_cache_append(None, 1, 128, 1, 64, 0, p, p, None) == -1
    # backward: workspace too small / missing, bad stage mask
    args = [p] * 7 + [1, 128, 1, 64, 0, ctypes.c_float(0.125)] + [p, p, p, None]
    assert lib.moda_attn_bwd(*args, p, ctypes.c_size_t(8), None) == -7
    assert lib.moda_attn_bwd(*args, None, ctypes.c_size_t(1 << 20), None) == -7
    assert lib.moda_attn_bwd_stages(*args, p, ctypes.c_size_t(1 << 20), 0, None) == -3
    assert lib.moda_attn_bwd_stages(*args, p, ctypes.c_size_t(1 << 20), 8, None) == -3      # accumulate bit without a stage
    assert lib.moda_attn_bwd_stages(*args, p, ctypes.c_size_t(1 << 20), 16, None) == -3     # form bit without a stage
    assert lib.moda_attn_bwd_stages(*args, p, ctypes.c_size_t(1 << 20), 32, None) == -3
    assert lib.moda_attn_bwd_stages(*args, p, ctypes.c_size_t(1 << 20), 7 | 32, None) == -3
    # the fused form needs the fp32 dQ accumulator, the reproducible split form only the row terms
    assert lib.moda_attn_bwd_stages(*args, p, ctypes.c_size_t(4096), 7, None) == -7
    assert moda.moda_bwd_workspace_bytes(1, 128, 1, 64, 0) >= 128 * 4 + 128 * 64 * 4
    # grouped-query entry points: H_kv must divide H; 1 to 8, 16 or 32 query heads per group
    gqa = lambda H, Hk: lib.moda_attn_fwd_gqa(p, p, p, None, 1, 128, H, Hk, 64, 0, ctypes.c_float(0.125), p, p, None)
    assert gqa(6, 4) == -12 and gqa(4, 0) == -12 and gqa(12, 1) == -12 and gqa(64, 1) == -12
    gargs = [p] * 7 + [1, 128, 6, 4, 64, 0, ctypes.c_float(0.125)] + [p, p, p, None]
    assert lib.moda_attn_bwd_gqa(*gargs, p, ctypes.c_size_t(1 << 20), None) == -12


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(ImportError):
        binding.load()


def test_decode_entry_point_validates_before_touching_the_device():
    lib = binding.load()
    p = ctypes.c_void_p(4096)
    ws = lib.moda_decode_workspace_bytes(1, 8, 128)
    assert ws >= 8 * 130 * 4 and lib.moda_decode_workspace_bytes(1, 8, 96) == 0

    def call(B=1, T_kv=10, T_cap=16, H=8, Hk=2, d=128, l=2, q=p, depth=p, work=p, wb=None):
        return lib.moda_attn_decode(q, p, p, depth, B, T_kv, T_cap, H, Hk, d, l, ctypes.c_float(0.1), p, p, work,
                                    ctypes.c_size_t(ws if wb is None else wb), None)

    assert call(T_kv=0) == -3 and call(T_kv=17) == -3 and call(B=0) == -3
    assert call(d=96) == -4
    assert call(l=-1) == -5 and call(l=257) == -5
    assert call(H=8, Hk=3) == -12 and call(H=12, Hk=1) == -12 and call(Hk=0) == -12
    assert call(q=None) == -1 and call(depth=None) == -1 and call(l=0, depth=None) != -1
    assert call(q=ctypes.c_void_p(4100)) == -2
    assert call(work=None) == -7 and call(wb=16) == -7


def test_prefill_entry_point_validates_before_touching_the_device():
    lib = binding.load()
    p = ctypes.c_void_p(4096)
    call = lambda Tq, Tkv, H=4, Hk=2, d=64, l=0, Q=p: lib.moda_attn_fwd_prefill(Q, p, p, None, 1, Tq, Tkv, H, Hk, d, l, ctypes.c_float(0.1), p, p, None)
    assert call(128, 64) == -3 and call(0, 64) == -3
    assert call(64, 128, d=96) == -4
    assert call(64, 128, H=6, Hk=4) == -12
    assert call(64, 128, l=2) == -1            # depth cache missing
    assert call(64, 128, Q=None) == -1


def test_paged_decode_entry_point_validates_before_touching_the_device():
    lib = binding.load()
    p = ctypes.c_void_p(4096)
    ws = lib.moda_decode_workspace_bytes(2, 8, 128)

    def call(page=64, pages=10, blocks=4, max_len=200, table=p, lens=p):
        return lib.moda_attn_decode_paged(p, p, p, table, lens, None, 2, max_len, page, pages, blocks, 8, 2, 128, 0,
                                          ctypes.c_float(0.1), p, p, p, ctypes.c_size_t(ws), None)

    assert call(page=48) == -3 and call(page=32) == -3 and call(pages=0) == -3
    assert call(blocks=3, max_len=200) == -3                      # 3 x 64 < 200
    assert call(table=None) == -1 and call(lens=None) == -1
    assert call(lens=ctypes.c_void_p(4098)) == -2
    assert lib.moda_attn_decode_varlen(p, p, p, None, None, 2, 100, 128, 8, 2, 128, 0, ctypes.c_float(0.1), p, p, p,
                                       ctypes.c_size_t(ws), None) == -1


def test_e4m3_cache_entry_points_validate_before_touching_the_device():
    lib = binding.load()
    vp = ctypes.c_void_p
    p, odd = vp(4096), vp(4100)
    sc = ctypes.c_float(0.125)
    # a block is 128 d bytes of codes and 128 fp32 row scales
    assert moda.moda_depth_cache_e4m3_bytes(1, 256, 2, 64, 4) == 4 * 1 * 2 * 2 * 2 * (128 * 64 + 512)
    assert moda.moda_depth_cache_e4m3_bytes(2, 129, 3, 128, 1) == 2 * 3 * 2 * 2 * (128 * 128 + 512)
    assert moda.moda_depth_cache_e4m3_bytes(1, 256, 2, 96, 4) == 0
    assert moda.moda_depth_cache_e4m3_bytes(1, 256, 2, 64, 257) == 0
    assert lib.moda_depth_cache_append_e4m3(p, 1, 128, 1, 64, 256, p, p, None) == -6
    assert lib.moda_depth_cache_append_e4m3(None, 1, 128, 1, 64, 0, p, p, None) == -1
    assert lib.moda_depth_cache_append_e4m3(p, 1, 128, 1, 64, 0, odd, p, None) == -2
    assert lib.moda_depth_cache_append_e4m3(p, 1, 128, 1, 48, 0, p, p, None) == -4
    fwd = lambda dkv=p, H=4, Hk=2, d=64, l=2, Q=p: lib.moda_attn_fwd_e4m3(Q, p, p, dkv, 1, 128, H, Hk, d, l, sc, p, p, None)
    assert fwd(dkv=None) == -1 and fwd(Q=odd) == -2 and fwd(d=32) == -4 and fwd(l=300) == -5
    assert fwd(H=4, Hk=3) == -12
    args = [p] * 7 + [1, 128, 1, 64, 1, sc] + [p, p, p]
    assert lib.moda_attn_bwd_e4m3(*args, None, p, ctypes.c_size_t(1 << 20), None) == -1      # depth slots without a gradient cache
    assert lib.moda_attn_bwd_e4m3(*args, p, p, ctypes.c_size_t(4096), None) == -7
    assert lib.moda_attn_bwd_e4m3(*args, p, None, ctypes.c_size_t(1 << 20), None) == -7


def test_softmax_scale_must_be_usable():
    lib = binding.load()
    p = ctypes.c_void_p(4096)
    for bad in (0.0, 1e-30, -0.09, float("inf"), float("nan")):
        sc = ctypes.c_float(bad)
        assert lib.moda_attn_fwd(p, p, p, None, 1, 128, 1, 64, 0, sc, p, p, None) == -13
        assert lib.moda_attn_fwd_append(p, p, p, None, 1, 128, 1, 1, 64, 0, sc, p, p, p, 0, None) == -13
        args = [p] * 7 + [1, 128, 1, 64, 0, sc] + [p, p, p, None]
        assert lib.moda_attn_bwd(*args, p, ctypes.c_size_t(1 << 20), None) == -13
        assert lib.moda_attn_bwd_static_scratch(*args, None) == -13
        assert lib.moda_attn_decode(p, p, p, None, 1, 128, 128, 2, 1, 64, 0, sc, p, p, p, ctypes.c_size_t(1 << 20), None) == -13
    for ok in (1e-6, 0.09, 3.0):
        # a usable scale passes this check and fails on the next one (no workspace)
        args = [p] * 7 + [1, 128, 1, 64, 0, ctypes.c_float(ok)] + [p, p, p, None]
        assert lib.moda_attn_bwd(*args, None, ctypes.c_size_t(0), None) == -7


def test_kv_projection_entry_point_validates_before_touching_the_device():
    lib = binding.load()
    p, odd = ctypes.c_void_p(4096), ctypes.c_void_p(4100)
    for fn in (lib.moda_kv_project_append, lib.moda_kv_project_append_e4m3):
        call = lambda X=p, Wk=p, Wv=p, B=1, T=128, Dm=256, Hk=2, d=64, K=p, V=p, cache=p, slot=0: \
            fn(X, Wk, Wv, B, T, Dm, Hk, d, K, V, cache, slot, None)
        assert call(Dm=100) == -3 and call(Dm=0) == -3 and call(T=0) == -3
        assert call(d=96) == -4
        assert call(slot=256) == -6 and call(slot=-1) == -6
        assert call(X=None) == -1 and call(Wv=None) == -1
        assert call(K=None) == -1                       # K and V outputs come together
        assert call(K=None, V=None, cache=None) == -1   # nothing to write
        assert call(Wk=odd) == -2 and call(cache=odd) == -2


def test_slot_mass_entry_point_validates_before_touching_the_device():
    lib = binding.load()
    p, odd = ctypes.c_void_p(4096), ctypes.c_void_p(4100)
    need = lib.moda_depth_slot_mass_workspace_bytes(1, 300, 4, 5)
    assert need == 1 * 4 * 3 * 5 * 4 and lib.moda_depth_slot_mass_workspace_bytes(1, 300, 4, 257) == 0
    call = lambda Q=p, cache=p, LSE=p, B=1, T=300, H=4, Hk=2, d=64, l=5, scale=0.1, mass=p, ws=p, wsb=need: \
        lib.moda_depth_slot_mass(Q, cache, LSE, B, T, H, Hk, d, l, ctypes.c_float(scale), mass, ws, ctypes.c_size_t(wsb), None)
    assert call(T=0) == -3 and call(d=96) == -4 and call(l=257) == -5 and call(Hk=3) == -12 and call(scale=0.0) == -13
    assert call(l=0, cache=None, mass=None, ws=None, wsb=0) == 0          # no slots: nothing to do
    assert call(Q=None) == -1 and call(mass=None) == -1 and call(cache=None) == -1
    assert call(LSE=odd) == -2
    assert call(ws=None) == -7 and call(wsb=need - 1) == -7
