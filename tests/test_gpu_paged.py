"""GPU parity for the paged cache (snapkv_compress_paged): every sequence against the oracle,
which reads K and V through the block table one row at a time, and bit for bit against the
library's own result on a dense copy.  Pages arrive in a random order; what lies behind a
sequence's end and in pages nobody uses is NaN and must never reach a result."""
import numpy as np
import pytest
import torch

from oracle import snapkv_oracle as orc
from paper_2404_14469_b200 import binding as sk
from paper_2404_14469_b200 import synth

import parity
from test_gpu_parity import PT, _bits
from test_oracle_paged import _paged_copy

pytestmark = pytest.mark.gpu


def _pools(data, page_size, seed, layout):
    k, v = _bits(data["k"]), _bits(data["v"])
    k_pool, v_pool, table = _paged_copy(k, v, page_size, np.random.default_rng(seed))
    tk = torch.from_numpy(k_pool.view(np.int16)).view(torch.bfloat16).cuda()
    tv = torch.from_numpy(v_pool.view(np.int16)).view(torch.bfloat16).cuda()
    if layout == "page-pos-head":      # stored [page, row, head, d], addressed as [page, head, row, d]
        tk = tk.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
        tv = tv.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    return k_pool, v_pool, table, tk, tv


@pytest.mark.parametrize("B,Hq,Hkv,L,d,W,page,kernel,ptype,budget,layout", [
    (2, 4, 2, 1000, 128, 32, 128, 5, "avg", 200, "page-head-pos"),
    (1, 8, 2, 3000, 128, 32, 256, 7, "max", 512, "page-pos-head"),
    (2, 4, 4, 2100, 64, 16, 384, 7, "max", 300, "page-head-pos"),
    (1, 8, 1, 5000, 64, 32, 1024, 13, "max", 1024, "page-pos-head"),   # two head sub-groups per KV head
    (2, 2, 2, 300, 128, 32, 128, 7, "max", 300, "page-head-pos"),      # budget >= L: copied through
    (1, 4, 2, 20000, 128, 32, 128, 5, "avg", 2048, "page-head-pos"),   # many pages, cluster select
])
def test_paged_cache_matches_oracle_and_the_dense_call(B, Hq, Hkv, L, d, W, page, kernel, ptype, budget, layout):
    data = synth.make_random(B, Hq, Hkv, L, d, W, seed=L + page, q_scale=1.5)
    k_pool, v_pool, table, tk, tv = _pools(data, page, L, layout)
    q = data["q_obs"].cuda()
    out_k, out_v, out_idx, ws = sk.snapkv_compress_paged(q, tk, tv, torch.from_numpy(table).cuda(), L,
                                                         kernel, PT[ptype], budget)
    assert sk.snapkv_device_status(ws) == (sk.OK, 0)
    ref = orc.compress_paged(_bits(data["q_obs"]), k_pool, v_pool, table, page, [L] * B, kernel, PT[ptype], budget)
    rows = min(budget, L)
    g = Hq // Hkv
    kb, vb = _bits(data["k"]), _bits(data["v"])
    idx = out_idx.cpu().numpy()
    for b in range(B):
        for h in range(Hq):
            if budget < L:
                parity.check_indices(idx[b, h], ref[b]["pooled"][0, h], rows - W, ref[b]["out_idx"][0, h])
            else:
                assert np.array_equal(idx[b, h], np.arange(L - W))
            parity.check_rows(_bits(out_k[b, h]), _bits(out_v[b, h]), kb[b, h // g], vb[b, h // g],
                              idx[b, h].astype(np.int64), W)
    # the same tiles reach the same arithmetic in the same order: identical to the dense call
    dense = sk.snapkv_compress(q, data["k"].cuda(), data["v"].cuda(), kernel, PT[ptype], budget)
    assert torch.equal(out_idx, dense[2]) and torch.equal(out_k, dense[0]) and torch.equal(out_v, dense[1])


def test_paged_batch_with_its_own_lengths_and_supplied_lse():
    lens, Hq, Hkv, d, W, page, kernel, budget = [700, 129, 2048, 1500], 4, 2, 128, 32, 256, 7, 256
    B, Lmax = len(lens), max(lens)
    seqs = [synth.make_random(1, Hq, Hkv, x, d, W, seed=40 + i, q_scale=1.5) for i, x in enumerate(lens)]
    # one pool for all sequences: pad every sequence to Lmax positions for the scatter helper,
    # then hand the true lengths to the call (the padding is NaN: it must not be read)
    k = np.full((B, Hkv, Lmax, d), 0x7FC0, dtype=np.uint16)
    v = np.full_like(k, 0x7FC0)
    for b, s in enumerate(seqs):
        k[b, :, : lens[b]], v[b, :, : lens[b]] = _bits(s["k"])[0], _bits(s["v"])[0]
    k_pool, v_pool, table = _paged_copy(k, v, page, np.random.default_rng(7))
    tk = torch.from_numpy(k_pool.view(np.int16)).view(torch.bfloat16).cuda()
    tv = torch.from_numpy(v_pool.view(np.int16)).view(torch.bfloat16).cuda()
    q = torch.cat([s["q_obs"] for s in seqs])
    lses = [orc.lse_obs(_bits(s["q_obs"]), _bits(s["k"])).astype(np.float32) for s in seqs]
    lse = torch.from_numpy(np.concatenate(lses)).cuda()
    for use_lse in (False, True):
        out_k, out_v, out_idx, ws = sk.snapkv_compress_paged(
            q.cuda(), tk, tv, torch.from_numpy(table).cuda(), Lmax, kernel, sk.POOL_MAX, budget,
            seq_lens=lens, lse_obs=lse if use_lse else None)
        assert sk.snapkv_device_status(ws) == (sk.OK, 0)
        for b, s in enumerate(seqs):
            qb, kb, vb = (_bits(s[x]) for x in ("q_obs", "k", "v"))
            ref = orc.compress(qb, kb, vb, kernel, orc.POOL_MAX, budget,
                               lse=lses[b].astype(np.float64) if use_lse else None)
            rows = min(budget, lens[b])
            ksel = rows - W
            idx = out_idx[b].cpu().numpy()
            for h in range(Hq):
                if budget < lens[b]:
                    parity.check_indices(idx[h], ref["pooled"][0, h], ksel, ref["out_idx"][0, h])
                else:
                    assert np.array_equal(idx[h, :ksel], np.arange(ksel)) and np.all(idx[h, ksel:] == -1)
                parity.check_rows(_bits(out_k[b, h])[:rows], _bits(out_v[b, h])[:rows], kb[0, h // 2], vb[0, h // 2],
                                  idx[h, :ksel].astype(np.int64), W)


def test_paged_arguments_are_checked_on_the_host():
    L_ = sk.lib()
    import ctypes
    st = (ctypes.c_int64 * 3)(2 * 128 * 64, 128 * 64, 64)
    FAKE = 0x1000
    def call(page_size=128, pages_per_seq=8, num_pages=16, L=1000, table=FAKE, strides=st):
        return L_.snapkv_compress_paged(FAKE, FAKE, FAKE, strides, strides, table, pages_per_seq, page_size,
                                        num_pages, None, None, 1, 2, 2, L, 64, 32, 7, 0, 256, FAKE, FAKE, FAKE,
                                        None, 0, None)
    assert call(page_size=100) == 1            # not a multiple of 128
    assert call(page_size=64) == 1
    assert call(pages_per_seq=7) == 1          # 7 * 128 < 1000
    assert call(num_pages=0) == 1
    assert call(table=None) == 1
    assert call(strides=(ctypes.c_int64 * 3)(2 * 128 * 64, 128 * 64, 60)) == 1
    assert call() == 3                         # everything fine but no workspace
