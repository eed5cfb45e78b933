"""P8: the depth FLOP model behind the reported metric, pinned to the paper's printed numbers."""
import os

from paper_2603_15619_b200 import flops

GOLD = os.path.join(os.path.dirname(__file__), "golden", "paper_table3_flops.txt")


def _gold():
    out = {}
    with open(GOLD) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                k, v = line.split()
                out[k] = float(v)
    return out


def test_depth_flops_reproduce_table3_delta():
    g = _gold()
    extra_T = flops.stack_depth_fwd_flops(int(g["T"]), int(g["D"]), int(g["layers"])) / 1e12
    # 8.01 T + model == 8.02 T at the table's two printed decimals
    assert round(g["flops_T_without"] + extra_T, 2) == g["flops_T_with"]
    # "0.12 %" extra: the printed figure is the two-decimal delta over the base (0.01 / 8.01)
    assert abs(100.0 * extra_T / g["flops_T_without"] - g["extra_percent"]) < 0.02
    # a model that forgot one of the two depth products (2 T D l), or counted them twice,
    # misses the percentage; the doubled one also misses the table entry
    for wrong in (extra_T / 2, extra_T * 2):
        assert abs(100.0 * wrong / g["flops_T_without"] - g["extra_percent"]) > 0.05
    assert round(g["flops_T_without"] + 2 * extra_T, 2) != g["flops_T_with"]


def test_depth_flops_match_table1_prefill_formula():
    # Table 1, prefilling FLOPs of depth attention / MoDA: 2 G T L^2 H_k d + 2 G T L H_k d,
    # i.e. 4 T D (L (L + 1) / 2) for layers counted 1..L with D = G H_k d.
    G, Hk, d, T, L = 2, 8, 64, 4096, 36
    D = G * Hk * d
    table1 = 2 * G * T * L * L * Hk * d + 2 * G * T * L * Hk * d
    assert table1 == sum(flops.depth_fwd_flops(1, T, 1, D, i) for i in range(1, L + 1))


def test_flop_and_byte_conventions():
    B, T, H, d, l = 2, 8192, 16, 128, 32
    assert flops.fwd_flops(B, T, H, d, 0) == 2.0 * B * H * d * T * T
    assert flops.bwd_flops(B, T, H, d, l) == 2.5 * flops.fwd_flops(B, T, H, d, l)
    assert flops.fwd_bwd_flops(B, T, H, d, l) == 3.5 * flops.fwd_flops(B, T, H, d, l)
    E = B * T * H * d
    assert flops.depth_bytes_fwd(B, T, H, d, l) == 4 * l * E
    assert flops.fwd_bytes(B, T, H, d, l) == 8 * E + 4 * l * E + 4 * B * H * T
