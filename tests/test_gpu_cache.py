"""Depth-KV cache: layout and append/unpack round trip (GPU)."""
import pytest
import torch

import paper_2603_15619_b200 as moda
from paper_2603_15619_b200 import synthetic

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("B,T,H,d,l", [(1, 256, 2, 64, 4), (2, 129, 3, 128, 2), (1, 1, 1, 64, 1), (1, 300, 2, 128, 3)])
def test_append_layout_and_round_trip(B, T, H, d, l):
    w = synthetic.Workload("t", B, T, H, d, l)
    x = synthetic.make(w, seed=3, device="cuda")
    nt = (T + 127) // 128
    cache = moda.alloc_depth_cache(B, T, H, d, l)
    cache.fill_(7.0)                                   # stale contents must be overwritten, tail rows zeroed
    for i in range(l):
        moda.moda_depth_cache_append(cache, i, x["Kd"][i].contiguous(), x["Vd"][i].contiguous())
    assert moda.moda_depth_cache_bytes(B, T, H, d, l) == l * B * H * nt * 2 * 128 * d * 2
    # documented layout: cache[slot][b][h][tile][kv][chunk][row][8]
    c = cache.view(l, B, H, nt, 2, d // 8, 128, 8)
    for kv, X in ((0, x["Kd"]), (1, x["Vd"])):
        Xp = torch.zeros((l, B, nt * 128, H, d), dtype=torch.bfloat16, device="cuda")
        Xp[:, :, :T] = X
        expect = Xp.view(l, B, nt, 128, H, d // 8, 8).permute(0, 1, 4, 2, 5, 3, 6)   # l,B,H,tile,chunk,row,8
        assert torch.equal(c[:, :, :, :, kv], expect)
    Kd2 = torch.empty_like(x["Kd"])
    Vd2 = torch.empty_like(x["Vd"])
    for i in range(l):
        moda.moda_depth_cache_unpack(cache, i, Kd2[i], Vd2[i])
    assert torch.equal(Kd2, x["Kd"]) and torch.equal(Vd2, x["Vd"])
    assert moda.moda_last_status() == 0
