"""Pins of the oracle's e4m3 row quantiser (CPU only): the lower-precision depth cache.

The paper names cheaper depth-KV caching only as a direction; the reading taken (per-row scale max|x| / 448, e4m3 codes,
decisions in fp32) is in the oracle's header.  What is fixed independently of the oracle:

  Q1  the library's float32 -> float8_e4m3fn cast picks the same codes (normals, subnormals, ties, saturation)
  Q2  brute force: the code is the nearest of the 256 format values (decode table written from the format definition)
  Q3  values that are representable at the row's scale survive the round trip exactly; the row maximum maps to +-448
  Q4  error bound of the format: relative 2^-4 in the normal range, absolute scale * 2^-10 below it
  Q5  the operator on dequantised depth tensors is the unchanged operator (nothing else moves)
"""
import numpy as np
import pytest
import torch

from oracle import moda_oracle as orc


def test_q1_library_cast_picks_the_same_codes():
    rng = np.random.default_rng(0)
    y = np.concatenate([
        rng.standard_normal(20000) * 100, rng.standard_normal(20000), rng.standard_normal(20000) * 2.0 ** -7,
        np.array([0.0, -0.0, 448.0, -448.0, 460.0, 1000.0, -3e38, 2.0 ** -9, 2.0 ** -10, 3 * 2.0 ** -10, 2.0 ** -6]),
        # exact ties between neighbouring codes in several binades
        np.array([(1 + (2 * k + 1) / 16) * 2.0 ** e for e in range(-6, 8) for k in range(8)]),
        np.array([(2 * k + 1) * 2.0 ** -10 for k in range(8)]),
    ]).astype(np.float32)
    y = y[np.abs(y) <= 464]                                   # the library cast does not saturate beyond the last rounding interval
    got = orc.e4m3_round(y)
    ref = torch.from_numpy(y).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    same = (got == ref) | ((got & 0x7f) == 0) & ((ref & 0x7f) == 0)     # +0 / -0
    assert same.all(), (y[~same][:5], got[~same][:5], ref[~same][:5])


def test_q2_nearest_format_value_by_brute_force():
    table = orc.e4m3_decode_table()
    assert np.isnan(table[0x7f]) and np.isnan(table[0xff]) and table[0x7e] == 448.0 and table[0x01] == 2.0 ** -9
    finite = np.where(np.isnan(table), np.inf, table)
    rng = np.random.default_rng(1)
    y = (rng.standard_normal(5000) * rng.choice([1e-3, 0.1, 1, 30, 200], 5000)).astype(np.float32)
    y = np.clip(y, -448, 448)
    codes = orc.e4m3_round(y)
    dist = np.abs(finite[None, :] - y[:, None].astype(np.float64))
    best = dist.min(axis=1)
    assert np.allclose(np.abs(table[codes] - y), best, rtol=0, atol=0)


def test_q3_representable_rows_round_trip_exactly():
    rng = np.random.default_rng(2)
    table = orc.e4m3_decode_table()
    codes = rng.integers(0, 256, size=(50, 64)).astype(np.uint8)
    codes[(codes & 0x7f) == 0x7f] = 0x10
    codes[:, 0] = 0x7e                                                        # the row maximum: 448
    scale = (2.0 ** rng.integers(-6, 4, size=50)).astype(np.float32)          # power-of-two scales: x is exact in fp32
    X = table[codes] * scale[:, None].astype(np.float64)
    c2, s2 = orc.quantize_e4m3_rows(X)
    assert np.array_equal(s2, scale)
    assert np.array_equal(orc.dequantize_e4m3_rows(c2, s2), X)
    # an all-zero row: scale 1, codes 0
    c0, s0 = orc.quantize_e4m3_rows(np.zeros((1, 8)))
    assert s0[0] == 1.0 and not c0.any()


def test_q4_error_bound_of_the_format():
    rng = np.random.default_rng(3)
    X = torch.from_numpy(rng.standard_normal((200, 128))).to(torch.bfloat16).double().numpy()
    codes, scale = orc.quantize_e4m3_rows(X)
    dq = orc.dequantize_e4m3_rows(codes, scale)
    amax = np.abs(X).max(axis=1)
    # the row maximum maps to +-448 and comes back as 448 * fp32(amax / 448): exact up to the rounding of the scale
    assert np.allclose(np.abs(dq).max(axis=1), amax, rtol=2.0 ** -23, atol=0)
    err = np.abs(dq - X)
    bound = np.maximum(np.abs(X) * 2.0 ** -4, scale[:, None] * 2.0 ** -10) * (1 + 1e-6)
    assert (err <= bound).all()
    assert (err > 0).mean() > 0.5                                              # and it does quantise


def test_q5_operator_on_dequantised_slots_is_the_unchanged_operator():
    rng = np.random.default_rng(4)
    B, T, H, d, l = 1, 9, 2, 16, 3
    Q, K, V = (rng.standard_normal((B, T, H, d)) for _ in range(3))
    Kd, Vd = (rng.standard_normal((l, B, T, H, d)) for _ in range(2))
    Kq = orc.dequantize_e4m3_rows(*orc.quantize_e4m3_rows(Kd))
    Vq = orc.dequantize_e4m3_rows(*orc.quantize_e4m3_rows(Vd))
    O, LSE = orc.forward(Q, K, V, Kq, Vq, 0.25)
    # explicit softmax over the union with the dequantised depth rows, row by row
    for t in (0, 4, 8):
        for h in range(H):
            keys = np.concatenate([K[0, :t + 1, h], Kq[:, 0, t, h]]); vals = np.concatenate([V[0, :t + 1, h], Vq[:, 0, t, h]])
            s = 0.25 * keys @ Q[0, t, h]
            p = np.exp(s - s.max()); p /= p.sum()
            np.testing.assert_allclose(O[0, t, h], p @ vals, rtol=1e-12, atol=1e-12)
