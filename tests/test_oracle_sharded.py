"""Pins for the oracle's per-shard functions (a prompt sharded along its length).  Eq. 1's
normaliser is a sum over keys and so splits over key ranges; what fixes the shard functions is
therefore the unsharded definition itself: merged shares equal the whole normaliser, and the
shards' votes, side by side, are the whole vote row."""
import numpy as np
import pytest

from oracle import snapkv_oracle as orc
from paper_2404_14469_b200 import synth


def _head(L, d, W, seed):
    w = synth.make_random(1, 1, 1, L, d, W, seed=seed, q_scale=2.0)
    q = orc.bf16_bits_to_f64(synth.bf16_bits(w["q_obs"])[0, 0])
    k = orc.bf16_bits_to_f64(synth.bf16_bits(w["k"])[0, 0])
    return q, k


@pytest.mark.parametrize("cuts", [[0, 300, 1000], [0, 100, 500, 1000], [0, 990, 1000], [0, 975, 985, 1000]])
def test_shares_merge_to_the_whole_normaliser_and_votes_concatenate(cuts):
    L, d, W = 1000, 32, 16
    n = L - W
    q, k = _head(L, d, W, seed=len(cuts))
    whole_lse = orc.window_lse(orc.window_logits(q, k))
    parts = np.stack([orc.shard_lse(q, k[a:b], a, n) for a, b in zip(cuts[:-1], cuts[1:])])
    merged = orc.merge_lse(parts)
    assert np.allclose(merged, whole_lse, rtol=1e-13, atol=1e-13)
    votes = np.concatenate([orc.shard_votes(q, k[a:b], merged, max(0, min(b - a, n - a)))
                            for a, b in zip(cuts[:-1], cuts[1:])])
    assert votes.shape == (n,)
    assert np.allclose(votes, orc.window_votes(q, k), rtol=1e-12)


def test_a_shard_behind_a_rows_horizon_contributes_nothing():
    # shard [992, 1000) of a prompt with n = 984, W = 16: row 0 sees keys <= 984, nothing here
    q, k = _head(1000, 32, 16, seed=5)
    part = orc.shard_lse(q, k[992:], 992, 984)
    assert np.all(np.isneginf(part[:8])) and np.all(np.isfinite(part[8:]))
    # and the merge ignores such shares
    other = orc.shard_lse(q, k[:992], 0, 984)
    assert np.allclose(orc.merge_lse(np.stack([other, part])), orc.window_lse(orc.window_logits(q, k)), rtol=1e-13)


def test_merge_is_a_plain_log_sum_exp():
    rng = np.random.default_rng(0)
    parts = rng.normal(size=(5, 7)) * 30
    assert np.allclose(orc.merge_lse(parts), np.log(np.exp(parts - parts.max()).sum(axis=0)) + parts.max())


def test_a_mask_that_ignores_the_shards_offset_is_caught():
    # planted mistake: the shard's mask taken in local coordinates (pos0 forgotten)
    q, k = _head(600, 32, 16, seed=6)
    n = 600 - 16
    good = orc.merge_lse(np.stack([orc.shard_lse(q, k[:300], 0, n), orc.shard_lse(q, k[300:], 300, n)]))
    bad = orc.merge_lse(np.stack([orc.shard_lse(q, k[:300], 0, n), orc.shard_lse(q, k[300:], 0, n)]))
    whole = orc.window_lse(orc.window_logits(q, k))
    assert np.allclose(good, whole, rtol=1e-13) and not np.allclose(bad, whole, rtol=1e-6)
