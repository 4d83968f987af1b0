"""GPU parity for the length-sharded step: the shards of a prompt are all held on one GPU and
take the ranks' parts in turn (sharded.compress_sharded_local runs the very protocol code the
multi-GPU path runs; the all-gather is a list).  Checked against the oracle's UNSHARDED step:
merged normalisers, whole vote rows, selected positions, and the assembled cache bit for bit."""
import numpy as np
import pytest
import torch

from oracle import snapkv_oracle as orc
from paper_2404_14469_b200 import binding as sk
from paper_2404_14469_b200 import sharded, synth

import parity
from test_gpu_parity import PT, _bits

pytestmark = pytest.mark.gpu


def _split(data, lens):
    k, v = data["k"].cuda(), data["v"].cuda()
    cuts = np.cumsum([0] + list(lens))
    ks = [k[:, :, a:b].contiguous() for a, b in zip(cuts[:-1], cuts[1:])]
    vs = [v[:, :, a:b].contiguous() for a, b in zip(cuts[:-1], cuts[1:])]
    return ks, vs


@pytest.mark.parametrize("B,Hq,Hkv,d,W,lens,kernel,ptype,budget", [
    (2, 4, 2, 128, 32, [1000, 1200, 800], 7, "max", 256),       # ragged shard edges
    (1, 8, 2, 128, 32, [4096, 4096], 5, "avg", 1024),
    (1, 4, 4, 64, 16, [130, 700, 64, 900], 7, "max", 200),      # a shard shorter than a tile
    (1, 8, 1, 64, 32, [2500, 2500], 13, "max", 512),            # two head sub-groups per KV head
    (1, 2, 2, 128, 64, [3000, 3000, 3000], 7, "max", 2048),     # W = 64
    (2, 2, 2, 128, 32, [300, 300], 7, "max", 1000),             # budget >= L: everything is kept
])
def test_sharded_step_matches_the_unsharded_oracle(B, Hq, Hkv, d, W, lens, kernel, ptype, budget):
    L = sum(lens)
    w = synth.Workload(90, "t", B, Hq, Hkv, d, L, W, kernel, ptype, (budget,), 1, 3)
    data = synth.make_layer(w, L % 97)
    ks, vs = _split(data, lens)
    q = data["q_obs"].cuda()
    results = sharded.compress_sharded_local(q, ks, vs, kernel, PT[ptype], budget)
    qb, kb, vb = (_bits(data[x]) for x in ("q_obs", "k", "v"))
    ref = orc.compress(qb, kb, vb, kernel, PT[ptype], budget)
    lse_ref = orc.lse_obs(qb, kb)
    vote_ref = ref["vote"] if ref["vote"] is not None else orc.votes(qb, kb)   # identity: votes are not needed
    n = L - W
    ksel = min(budget, L) - W
    for r, res in enumerate(results):
        assert torch.equal(res["out_idx"], results[0]["out_idx"])
        assert np.allclose(res["lse_obs"].cpu().numpy(), lse_ref, rtol=0, atol=2e-5)
    votes = results[0]["votes"].cpu().numpy()
    idx = results[0]["out_idx"].cpu().numpy()
    assert votes.shape == (B, Hq, n) and idx.shape == (B, Hq, ksel)
    out_k, out_v = sharded.assemble(results, W)
    g = Hq // Hkv
    for b in range(B):
        for h in range(Hq):
            parity.check_votes(votes[b, h], vote_ref[b, h])
            if budget < L:
                parity.check_indices(idx[b, h], ref["pooled"][b, h], ksel, ref["out_idx"][b, h])
            else:
                assert np.array_equal(idx[b, h], np.arange(n))
            parity.check_rows(_bits(out_k[b, h]), _bits(out_v[b, h]), kb[b, h // g], vb[b, h // g],
                              idx[b, h].astype(np.int64), W)


def test_one_shard_is_the_single_gpu_step():
    data = synth.make_layer(synth.Workload(91, "t", 1, 4, 2, 128, 5000, 32, 7, "max", (512,), 1, 3), 4)
    dev = {x: data[x].cuda() for x in ("q_obs", "k", "v")}
    res = sharded.compress_sharded_local(dev["q_obs"], [dev["k"]], [dev["v"]], 7, sk.POOL_MAX, 512)
    whole = sk.snapkv_compress(dev["q_obs"], dev["k"], dev["v"], 7, sk.POOL_MAX, 512)
    ok, ov = sharded.assemble(res, 32)
    # max pooling, same votes up to the last bit of the normaliser's fold: same positions
    assert torch.equal(res[0]["out_idx"], whole[2])
    assert torch.equal(ok, whole[0]) and torch.equal(ov, whole[1])


def test_shard_steps_reject_bad_arguments():
    L_ = sk.lib()
    FAKE = 0x1000
    assert L_.snapkv_shard_lse(FAKE, FAKE, 1, 4, 2, 16, 64, 32, 0, FAKE, FAKE, 1 << 20, None) == 1   # W > Ls
    assert L_.snapkv_shard_votes(FAKE, FAKE, FAKE, 1, 4, 2, 100, 64, 32, 101, FAKE, FAKE, 1 << 20, None) == 1
    assert L_.snapkv_shard_votes(FAKE, FAKE, None, 1, 4, 2, 100, 64, 32, 50, FAKE, FAKE, 1 << 20, None) == 1
    assert L_.snapkv_lse_merge(FAKE, 0, 10, FAKE, None) == 1
    assert L_.snapkv_gather_range(FAKE, FAKE, FAKE, 1, 4, 2, 100, 64, 0, 10, 0, FAKE, FAKE, 5, FAKE, None) == 1
    assert L_.snapkv_gather_range(FAKE, FAKE, FAKE, 1, 4, 2, 100, 64, 0, 10, 200, FAKE, FAKE, 500, FAKE, None) == 1
