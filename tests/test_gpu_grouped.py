"""GPU parity for the shared-selection step (snapkv_compress_grouped): one selection per KV head
from the summed votes of the group's query heads, checked against the oracle's compress_grouped
with the acceptance rule of the per-head step; small shapes over every select kernel, the other
input variants, and the 32K GQA workload at full size on sampled KV heads."""
import numpy as np
import pytest
import torch

from oracle import snapkv_oracle as orc
from paper_2404_14469_b200 import binding as sk
from paper_2404_14469_b200 import synth

import parity
from test_gpu_parity import PT, _bits

pytestmark = pytest.mark.gpu


def _check_grouped(dev, W, kernel, ptype, budget, kv_heads=None, lse=None, **kw):
    out_k, out_v, out_idx, ws = sk.snapkv_compress_grouped(dev["q_obs"], dev["k"], dev["v"], kernel,
                                                           PT[ptype], budget, lse_obs=lse, **kw)
    code, detail = sk.snapkv_device_status(ws)
    assert code == sk.OK, (code, detail)
    B, Hq = dev["q_obs"].shape[:2]
    Hkv, L, d = dev["k"].shape[1:]
    ksel = budget - W
    assert out_k.shape == (B, Hkv, budget, d) and out_idx.shape == (B, Hkv, ksel)
    kv_heads = kv_heads or [(b, c) for b in range(B) for c in range(Hkv)]
    q, k, v = _bits(dev["q_obs"]), _bits(dev["k"]), _bits(dev["v"])
    ref = orc.compress_grouped(q, k, v, kernel, PT[ptype], budget, kv_heads=kv_heads,
                               lse=None if lse is None else lse.cpu().numpy().astype(np.float64))
    idx_all = out_idx.cpu().numpy()
    exact = 0
    for (b, c) in kv_heads:
        exact += parity.check_indices(idx_all[b, c], ref["pooled"][b, c], ksel, ref["out_idx"][b, c])
        parity.check_rows(_bits(out_k[b, c]), _bits(out_v[b, c]), k[b, c], v[b, c],
                          idx_all[b, c].astype(np.int64), W)
    return exact, len(kv_heads), (out_k, out_v, out_idx)


@pytest.mark.parametrize("B,Hq,Hkv,L,d,W,kernel,ptype,budget", [
    (2, 8, 2, 1000, 128, 32, 5, "avg", 200),       # g*W = 128: the whole group in one unit
    (1, 8, 1, 2100, 64, 32, 7, "max", 512),        # g*W = 256: two head sub-groups per KV head
    (1, 4, 2, 1500, 128, 64, 13, "max", 300),      # W = 64
    (1, 6, 3, 333, 64, 5, 1, "max", 40),           # no pooling, odd window
    (1, 4, 2, 3000, 64, 16, 17, "avg", 200),       # radius beyond the fast select kernel
    (1, 4, 2, 60000, 64, 32, 7, "max", 1024),      # long rows: many CTAs per row
    (3, 2, 1, 257, 64, 32, 5, "max", 33),          # keeps a single prefix row
])
def test_grouped_compress_small_shapes(B, Hq, Hkv, L, d, W, kernel, ptype, budget):
    w = synth.Workload(70, "t", B, Hq, Hkv, d, L, W, kernel, ptype, (budget,), 1, 2)
    data = synth.make_layer(w, L)
    dev = {x: data[x].cuda() for x in ("q_obs", "k", "v")}
    _check_grouped(dev, W, kernel, ptype, budget)


def test_one_head_per_group_equals_the_per_head_call():
    data = synth.make_random(2, 4, 4, 900, 128, 32, seed=21, q_scale=2.0)
    q, k, v = (data[x].cuda() for x in ("q_obs", "k", "v"))
    a = sk.snapkv_compress_grouped(q, k, v, 7, sk.POOL_MAX, 256)[:3]
    b = sk.snapkv_compress(q, k, v, 7, sk.POOL_MAX, 256)[:3]
    for x, y in zip(a, b):
        assert torch.equal(x.view(torch.int16) if x.dtype == torch.bfloat16 else x,
                           y.view(torch.int16) if y.dtype == torch.bfloat16 else y)


def test_grouped_with_supplied_lse_and_strided_cache():
    B, Hq, Hkv, L, d, W, kernel, budget = 2, 8, 2, 900, 128, 32, 7, 160
    w = synth.Workload(71, "t", B, Hq, Hkv, d, L, W, kernel, "max", (budget,), 1, 2)
    data = synth.make_layer(w, 5)
    dev = {x: data[x].cuda() for x in ("q_obs", "k", "v")}
    lse = torch.from_numpy(orc.lse_obs(_bits(data["q_obs"]), _bits(data["k"])).astype(np.float32)).cuda()
    _, _, dense = _check_grouped(dev, W, kernel, "max", budget, lse=lse)
    blhd = {"q_obs": dev["q_obs"],
            "k": dev["k"].permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3),
            "v": dev["v"].permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)}
    _, _, strided = _check_grouped(blhd, W, kernel, "max", budget, lse=lse)
    for x, y in zip(dense, strided):
        assert torch.equal(x.view(torch.int16) if x.dtype == torch.bfloat16 else x,
                           y.view(torch.int16) if y.dtype == torch.bfloat16 else y)


def test_grouped_identity_keeps_Hkv_heads():
    data = synth.make_random(2, 8, 2, 300, 64, 32, seed=22)
    q, k, v = (data[x].cuda() for x in ("q_obs", "k", "v"))
    ok, ov, oi, _ = sk.snapkv_compress_grouped(q, k, v, 7, sk.POOL_MAX, 300)
    assert torch.equal(ok.view(torch.int16), k.view(torch.int16))
    assert torch.equal(ov.view(torch.int16), v.view(torch.int16))
    assert torch.equal(oi.cpu(), torch.arange(268, dtype=torch.int32).expand(2, 2, 268))


def test_grouped_full_size_gqa_workload_on_sampled_kv_heads():
    w = synth.WORKLOADS[2]
    dev = synth.make_layer(w, 7, device="cuda")
    _check_grouped(dev, w.W, w.pool_kernel, w.pool_type, w.budgets[0], kv_heads=[(0, 3), (2, 0), (3, 7)])
