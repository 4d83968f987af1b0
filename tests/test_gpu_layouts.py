"""GPU parity for caches that are not stored as dense [B, Hkv, L, d] (snapkv_compress_strided):
the same seeded inputs laid out as [B, L, Hkv, d], as one fused K/V buffer, or as a slice of a
longer cache must give the oracle's result and, bit for bit, the dense call's result."""
import numpy as np
import pytest
import torch

from oracle import snapkv_oracle as orc
from paper_2404_14469_b200 import binding as sk
from paper_2404_14469_b200 import synth

from test_gpu_parity import PT, _check_compress

pytestmark = pytest.mark.gpu


def _blhd(t):
    """[B, Hkv, L, d] values stored as [B, L, Hkv, d]; returned as a [B, Hkv, L, d] view."""
    return t.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)


def _fused(k, v):
    """K and V interleaved in one [B, L, 2, Hkv, d] buffer."""
    buf = torch.stack([k.permute(0, 2, 1, 3), v.permute(0, 2, 1, 3)], dim=2).contiguous()
    return buf[:, :, 0].permute(0, 2, 1, 3), buf[:, :, 1].permute(0, 2, 1, 3)


def _padded(t, extra):
    """The first L positions of a cache allocated for L + extra positions."""
    B, H, L, d = t.shape
    big = torch.full((B, H, L + extra, d), float("nan"), dtype=t.dtype, device=t.device)
    big[:, :, :L] = t
    return big[:, :, :L]


def _layouts(k, v):
    fk, fv = _fused(k, v)
    return {
        "blhd": (_blhd(k), _blhd(v)),
        "fused": (fk, fv),
        "padded": (_padded(k, 72), _padded(v, 8)),
        "mixed": (_blhd(k), v),                      # K strided, V dense
    }


SHAPES = [
    # B, Hq, Hkv, L, d, W, kernel, ptype, budget
    (2, 4, 2, 1000, 128, 32, 5, "avg", 200),       # GQA, ragged L
    (1, 8, 1, 2100, 64, 32, 7, "max", 512),        # d = 64, two head sub-groups per KV head
    (3, 6, 3, 700, 128, 16, 13, "max", 100),       # batch 3, W = 16
]


@pytest.mark.parametrize("B,Hq,Hkv,L,d,W,kernel,ptype,budget", SHAPES)
def test_strided_layouts_match_oracle_and_dense_call(B, Hq, Hkv, L, d, W, kernel, ptype, budget):
    w = synth.Workload(60, "t", B, Hq, Hkv, d, L, W, kernel, ptype, (budget,), 1, 2)
    data = synth.make_layer(w, L)
    q, k, v = (data[x].cuda() for x in ("q_obs", "k", "v"))
    dense = sk.snapkv_compress(q, k, v, kernel, PT[ptype], budget)[:3]
    for name, (ks, vs) in _layouts(k, v).items():
        if Hkv > 1 and B > 1:  # (a view over size-1 dimensions counts as contiguous)
            assert not (ks.is_contiguous() and vs.is_contiguous()), name
        assert torch.equal(ks, k) and torch.equal(vs, v)
        # against the oracle, head by head (reads the views themselves)
        _, _, got = _check_compress(None, W, kernel, ptype, budget, dev={"q_obs": q, "k": ks, "v": vs})
        # against the dense call: the arithmetic and its order do not depend on the layout
        for a, b_ in zip(got, dense):
            assert torch.equal(a.view(torch.int16) if a.dtype == torch.bfloat16 else a,
                               b_.view(torch.int16) if b_.dtype == torch.bfloat16 else b_), name


def test_strided_layout_with_supplied_lse():
    B, Hq, Hkv, L, d, W, kernel, budget = 2, 8, 2, 900, 128, 32, 7, 160
    w = synth.Workload(61, "t", B, Hq, Hkv, d, L, W, kernel, "max", (budget,), 1, 2)
    data = synth.make_layer(w, 3)
    q, k, v = (data[x].cuda() for x in ("q_obs", "k", "v"))
    lse = torch.from_numpy(orc.lse_obs(synth.bf16_bits(data["q_obs"]), synth.bf16_bits(data["k"]))
                           .astype(np.float32)).cuda()
    dense = sk.snapkv_compress_lse(q, k, v, lse, kernel, sk.POOL_MAX, budget)[:3]
    got = sk.snapkv_compress(q, _blhd(k), _blhd(v), kernel, sk.POOL_MAX, budget, lse_obs=lse)[:3]
    for a, b_ in zip(got, dense):
        assert torch.equal(a.view(torch.int16) if a.dtype == torch.bfloat16 else a,
                           b_.view(torch.int16) if b_.dtype == torch.bfloat16 else b_)


def test_strided_identity_path_copies_the_cache():
    B, Hq, Hkv, L, d, W = 2, 4, 2, 300, 64, 32
    data = synth.make_random(B, Hq, Hkv, L, d, W, seed=11)
    q, k, v = (data[x].cuda() for x in ("q_obs", "k", "v"))
    ok, ov, oi, _ = sk.snapkv_compress(q, _blhd(k), _padded(v, 40), 7, sk.POOL_MAX, L + 5)
    g = Hq // Hkv
    assert torch.equal(ok.view(torch.int16), k.repeat_interleave(g, dim=1).view(torch.int16))
    assert torch.equal(ov.view(torch.int16), v.repeat_interleave(g, dim=1).view(torch.int16))
    assert torch.equal(oi.cpu(), torch.arange(L - W, dtype=torch.int32).expand(B, Hq, L - W))
