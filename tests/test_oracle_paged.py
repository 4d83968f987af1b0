"""Pins for the oracle's paged-cache reader.  Paging only changes where a row of K or V lives
(Listing 1 takes dense key_states / value_states), so everything is fixed by one statement:
the step on a paged cache equals the step on the dense sequence the table describes."""
import numpy as np
import pytest

from oracle import snapkv_oracle as orc
from paper_2404_14469_b200 import synth


def _paged_copy(k, v, page_size, rng, extra_pages=3, fill=0x7FC0):
    """Scatter dense [B, Hkv, L, d] bit patterns into a pool in a random page order; what a
    page holds behind a sequence's end, and the pages nobody uses, are filled with NaN."""
    B, Hkv, L, d = k.shape
    pps = -(-L // page_size)
    num_pages = B * pps + extra_pages
    order = rng.permutation(num_pages)
    k_pool = np.full((num_pages, Hkv, page_size, d), fill, dtype=np.uint16)
    v_pool = np.full_like(k_pool, fill)
    table = np.zeros((B, pps), dtype=np.int32)
    for b in range(B):
        for s in range(pps):
            page = int(order[b * pps + s])
            table[b, s] = page
            lo, hi = s * page_size, min(L, (s + 1) * page_size)
            k_pool[page, :, : hi - lo] = k[b, :, lo:hi]
            v_pool[page, :, : hi - lo] = v[b, :, lo:hi]
    return k_pool, v_pool, table


@pytest.mark.parametrize("L,page_size", [(300, 128), (512, 256), (1000, 384)])
def test_paged_step_equals_the_dense_step(L, page_size):
    w = synth.make_random(2, 4, 2, L, 32, 16, seed=L)
    q, k, v = (synth.bf16_bits(w[x]) for x in ("q_obs", "k", "v"))
    k_pool, v_pool, table = _paged_copy(k, v, page_size, np.random.default_rng(L))
    dense = orc.compress(q, k, v, 5, orc.POOL_AVG, 64)
    paged = orc.compress_paged(q, k_pool, v_pool, table, page_size, [L, L], 5, orc.POOL_AVG, 64)
    for b in range(2):
        for name in ("out_k", "out_v", "out_idx"):
            assert np.array_equal(paged[b][name][0], dense[name][b])
        assert np.array_equal(paged[b]["vote"][0], dense["vote"][b])


def test_reader_follows_the_table_row_by_row():
    rng = np.random.default_rng(1)
    pool = rng.integers(0, 2 ** 16, size=(7, 2, 128, 4), dtype=np.uint16)
    row = [5, 0, 3]
    got = orc.read_paged(pool, row, 128, 300)
    assert got.shape == (2, 300, 4)
    for p in (0, 1, 127, 128, 255, 256, 299):
        assert np.array_equal(got[:, p], pool[row[p // 128], :, p % 128])
    # an entry outside the pool reads as zeros
    got = orc.read_paged(pool, [5, 99, -1], 128, 300)
    assert not got[:, 128:].any() and np.array_equal(got[:, :128], pool[5, :, :128])


def test_sequences_may_share_pages_and_differ_in_length():
    # two prompts with a common 256-token prefix held once in the pool
    a = synth.make_random(1, 2, 2, 600, 32, 16, seed=3)
    b = synth.make_random(1, 2, 2, 400, 32, 16, seed=4)
    ka, va, kb, vb = (synth.bf16_bits(x) for x in (a["k"], a["v"], b["k"], b["v"]))
    kb[:, :, :256], vb[:, :, :256] = ka[:, :, :256], va[:, :, :256]
    page = 128
    k_pool = np.zeros((8, 2, page, 32), dtype=np.uint16)
    v_pool = np.zeros_like(k_pool)
    table = np.array([[0, 1, 2, 3, 4], [0, 1, 5, 6, 0]], dtype=np.int32)   # pages 0, 1 shared
    for s, pg in enumerate(table[0]):
        lo, hi = s * page, min(600, (s + 1) * page)
        k_pool[pg, :, : hi - lo], v_pool[pg, :, : hi - lo] = ka[0, :, lo:hi], va[0, :, lo:hi]
    for s, pg in enumerate(table[1][:4]):
        lo, hi = s * page, min(400, (s + 1) * page)
        k_pool[pg, :, : hi - lo], v_pool[pg, :, : hi - lo] = kb[0, :, lo:hi], vb[0, :, lo:hi]
    q = np.concatenate([synth.bf16_bits(a["q_obs"]), synth.bf16_bits(b["q_obs"])])
    res = orc.compress_paged(q, k_pool, v_pool, table, page, [600, 400], 7, orc.POOL_MAX, 100)
    ref_a = orc.compress(q[:1], ka, va, 7, orc.POOL_MAX, 100)
    ref_b = orc.compress(q[1:], kb, vb, 7, orc.POOL_MAX, 100)
    assert np.array_equal(res[0]["out_idx"], ref_a["out_idx"]) and np.array_equal(res[0]["out_k"], ref_a["out_k"])
    assert np.array_equal(res[1]["out_idx"], ref_b["out_idx"]) and np.array_equal(res[1]["out_v"], ref_b["out_v"])


def test_a_reader_that_ignores_the_table_is_caught():
    # planted mistake: pages read in pool order instead of table order
    w = synth.make_random(1, 2, 2, 512, 32, 16, seed=9)
    q, k, v = (synth.bf16_bits(w[x]) for x in ("q_obs", "k", "v"))
    k_pool, v_pool, table = _paged_copy(k, v, 128, np.random.default_rng(2), fill=0)
    assert not np.array_equal(table[0], np.arange(table.shape[1]))
    good = orc.compress_paged(q, k_pool, v_pool, table, 128, [512], 5, orc.POOL_MAX, 64)[0]
    wrong_table = np.arange(table.shape[1], dtype=np.int32)[None]
    bad = orc.compress_paged(q, k_pool, v_pool, wrong_table, 128, [512], 5, orc.POOL_MAX, 64)[0]
    dense = orc.compress(q, k, v, 5, orc.POOL_MAX, 64)
    assert np.array_equal(good["out_k"], dense["out_k"])
    assert not np.array_equal(bad["out_k"], dense["out_k"])
