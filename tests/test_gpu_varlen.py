"""GPU parity for batches of prompts of different lengths (snapkv_compress_varlen): every
sequence must come out as the oracle's single-sequence step on that sequence alone, for a padded
[B, Hkv, Lmax, d] cache and for a packed [total_tokens, Hkv, d] cache."""
import numpy as np
import pytest
import torch

from oracle import snapkv_oracle as orc
from paper_2404_14469_b200 import binding as sk
from paper_2404_14469_b200 import synth

import parity
from test_gpu_parity import PT, _bits

pytestmark = pytest.mark.gpu


def _sequences(lens, Hq, Hkv, d, W, kernel, ptype, budget, seed):
    """One seeded single-sequence layer per length (clusters planted as in the workloads)."""
    out = []
    for i, L in enumerate(lens):
        w = synth.Workload(80 + seed, "t", 1, Hq, Hkv, d, L, W, kernel, ptype, (budget,), 1, 2)
        out.append(synth.make_layer(w, 100 * seed + i))
    return out


def _check_sequence(b, seq, L, W, kernel, ptype, budget, out_k, out_v, out_idx, lse=None):
    q, k, v = (_bits(seq[x]) for x in ("q_obs", "k", "v"))
    ref = orc.compress(q, k, v, kernel, PT[ptype], budget, lse=lse)
    Hq, Hkv = q.shape[1], k.shape[1]
    g = Hq // Hkv
    rows = min(budget, L)
    ksel = rows - W
    idx = out_idx[b].cpu().numpy()
    ok, ov = _bits(out_k[b]), _bits(out_v[b])
    for h in range(Hq):
        if budget >= L:   # copied through; nothing beyond its rows is touched
            assert np.array_equal(idx[h, :ksel], np.arange(ksel)) and np.all(idx[h, ksel:] == -1)
            assert not ok[h, rows:].any() and not ov[h, rows:].any()
        else:
            parity.check_indices(idx[h], ref["pooled"][0, h], ksel, ref["out_idx"][0, h])
        parity.check_rows(ok[h, :rows], ov[h, :rows], k[0, h // g], v[0, h // g],
                          idx[h, :ksel].astype(np.int64), W)


@pytest.mark.parametrize("lens,Hq,Hkv,d,W,kernel,ptype,budget", [
    ([1000, 333, 2048, 129], 4, 2, 128, 32, 5, "avg", 200),     # 129 < budget: copied through
    ([700, 64, 1500], 8, 1, 64, 32, 7, "max", 256),             # 64 = 2 W, shorter than a tile
    ([900, 50000], 2, 2, 64, 16, 7, "max", 512),                # a long row next to a short one
])
def test_padded_batch_matches_per_sequence_oracle(lens, Hq, Hkv, d, W, kernel, ptype, budget):
    seqs = _sequences(lens, Hq, Hkv, d, W, kernel, ptype, budget, seed=1)
    B, Lmax = len(lens), max(lens)
    k = torch.full((B, Hkv, Lmax, d), float("nan"), dtype=torch.bfloat16)   # padding must not be read
    v = torch.full((B, Hkv, Lmax, d), float("nan"), dtype=torch.bfloat16)
    for b, s in enumerate(seqs):
        k[b, :, :lens[b]] = s["k"][0]
        v[b, :, :lens[b]] = s["v"][0]
    q = torch.cat([s["q_obs"] for s in seqs])
    out_k, out_v, out_idx, ws = sk.snapkv_compress_varlen(q.cuda(), k.cuda(), v.cuda(), lens, kernel,
                                                          PT[ptype], budget)
    code, detail = sk.snapkv_device_status(ws)
    assert code == sk.OK, (code, detail)
    for b, s in enumerate(seqs):
        _check_sequence(b, s, lens[b], W, kernel, ptype, budget, out_k, out_v, out_idx)


def test_packed_cache_with_supplied_lse_matches_per_sequence_oracle():
    lens, Hq, Hkv, d, W, kernel, budget = [640, 1111, 200], 8, 2, 128, 32, 7, 300
    seqs = _sequences(lens, Hq, Hkv, d, W, kernel, "max", budget, seed=2)
    cu = [0, 640, 640 + 1111]
    k = torch.cat([s["k"][0].permute(1, 0, 2) for s in seqs]).contiguous()      # [T, Hkv, d]
    v = torch.cat([s["v"][0].permute(1, 0, 2) for s in seqs]).contiguous()
    q = torch.cat([s["q_obs"] for s in seqs])
    lses = [orc.lse_obs(_bits(s["q_obs"]), _bits(s["k"])).astype(np.float32) for s in seqs]
    lse = torch.from_numpy(np.concatenate(lses)).cuda()
    for use_lse in (False, True):
        out_k, out_v, out_idx, ws = sk.snapkv_compress_varlen(
            q.cuda(), k.cuda(), v.cuda(), lens, kernel, sk.POOL_MAX, budget, cu_seqlens=cu,
            lse_obs=lse if use_lse else None)
        code, detail = sk.snapkv_device_status(ws)
        assert code == sk.OK, (code, detail)
        for b, s in enumerate(seqs):
            _check_sequence(b, s, lens[b], W, kernel, "max", budget, out_k, out_v, out_idx,
                            lse=lses[b].astype(np.float64) if use_lse else None)


@pytest.mark.parametrize("use_lse", [False, True])
def test_status_block_is_clean_whichever_path_the_first_sequence_takes(use_lse):
    # first sequence shorter than the budget (copied through), second one compressed; the
    # workspace arrives full of 0xFF, as memory that was never cleared may
    lens, Hq, Hkv, d, W, kernel, budget = [129, 1000], 4, 2, 128, 32, 5, 200
    seqs = _sequences(lens, Hq, Hkv, d, W, kernel, "avg", budget, seed=3)
    B, Lmax = len(lens), max(lens)
    k = torch.zeros(B, Hkv, Lmax, d, dtype=torch.bfloat16)
    v = torch.zeros(B, Hkv, Lmax, d, dtype=torch.bfloat16)
    for b, s in enumerate(seqs):
        k[b, :, :lens[b]] = s["k"][0]
        v[b, :, :lens[b]] = s["v"][0]
    q = torch.cat([s["q_obs"] for s in seqs])
    lses = [orc.lse_obs(_bits(s["q_obs"]), _bits(s["k"])).astype(np.float32) for s in seqs]
    lse = torch.from_numpy(np.concatenate(lses)).cuda() if use_lse else None
    need = sk.snapkv_workspace_size(1, Hq, Hkv, Lmax, d, W, kernel, sk.POOL_AVG, budget)
    ws = torch.full((need,), 0xFF, dtype=torch.uint8, device="cuda")
    out_k, out_v, out_idx, ws2 = sk.snapkv_compress_varlen(q.cuda(), k.cuda(), v.cuda(), lens, kernel,
                                                           sk.POOL_AVG, budget, lse_obs=lse, workspace=ws)
    assert ws2 is ws
    assert sk.snapkv_device_status(ws) == (sk.OK, 0)
    for b, s in enumerate(seqs):
        _check_sequence(b, s, lens[b], W, kernel, "avg", budget, out_k, out_v, out_idx,
                        lse=lses[b].astype(np.float64) if use_lse else None)
    # the same for a plain call that only copies the cache through
    ws.fill_(0xFF)
    dev = {x: seqs[0][x].cuda() for x in ("q_obs", "k", "v")}
    sk.snapkv_compress(dev["q_obs"], dev["k"], dev["v"], kernel, sk.POOL_AVG, budget, workspace=ws)
    assert sk.snapkv_device_status(ws) == (sk.OK, 0)
