"""Pins for the oracle's shared-selection variant (group_votes, compress_grouped): a library
softmax restatement with the head map written out, a closed form, the reduction to the per-head
step, a replication law, structural invariants, and planted mistakes these pins must catch.
CPU only."""
import math

import numpy as np
import pytest
import torch

from oracle import snapkv_oracle as orc
from paper_2404_14469_b200 import synth


def _bits(B, Hq, Hkv, L, d, W, seed, q_scale=2.0):
    data = synth.make_random(B, Hq, Hkv, L, d, W, seed=seed, q_scale=q_scale)
    return tuple(synth.bf16_bits(data[x]) for x in ("q_obs", "k", "v"))


def _library_group_vote(q, k, b, c, g):
    """Group vote of KV head c from framework ops: masked softmax per query head, summed over the
    window rows and over heads c*g .. c*g+g-1."""
    W, d = q.shape[2], q.shape[3]
    L = k.shape[2]
    n = L - W
    kf = torch.from_numpy(orc.bf16_bits_to_f64(k[b, c]))
    total = torch.zeros(n, dtype=torch.float64)
    for h in range(c * g, c * g + g):
        qf = torch.from_numpy(orc.bf16_bits_to_f64(q[b, h]))
        s = qf @ kf.T / math.sqrt(d)
        mask = torch.arange(L)[None, :] > (n + torch.arange(W))[:, None]
        p = torch.softmax(s.masked_fill(mask, float("-inf")), dim=-1)
        total += p[:, :n].sum(dim=0)
    return total.numpy()


def test_group_vote_matches_library_softmax_with_the_head_map_written_out():
    B, Hq, Hkv, L, d, W = 2, 6, 2, 90, 16, 8
    q, k, v = _bits(B, Hq, Hkv, L, d, W, seed=1)
    ref = orc.compress_grouped(q, k, v, 5, orc.POOL_MAX, 30)
    for b in range(B):
        for c in range(Hkv):
            lib = _library_group_vote(q, k, b, c, Hq // Hkv)
            assert np.allclose(ref["vote"][b, c], lib, rtol=1e-12, atol=0)


def test_uniform_attention_gives_g_times_the_harmonic_difference():
    B, Hq, Hkv, L, d, W = 1, 4, 2, 57, 8, 6
    q, k, v = _bits(B, Hq, Hkv, L, d, W, seed=2)
    q[:] = 0  # bf16 zero: every visible key gets the same probability
    ref = orc.compress_grouped(q, k, v, 1, orc.POOL_MAX, 20)
    n = L - W
    closed = 2 * sum(1.0 / (n + i + 1) for i in range(W))
    assert np.allclose(ref["vote"], closed, rtol=1e-13, atol=0)


def test_one_head_per_group_is_the_per_head_step():
    q, k, v = _bits(2, 3, 3, 120, 16, 8, seed=3)
    a = orc.compress_grouped(q, k, v, 7, orc.POOL_AVG, 40)
    b = orc.compress(q, k, v, 7, orc.POOL_AVG, 40)
    for key in ("out_k", "out_v", "out_idx", "vote", "pooled"):
        assert np.array_equal(a[key], b[key]), key


def test_replicated_heads_select_what_the_single_head_selects():
    # g copies of the same query head: the group vote is g times the head's vote, and scaling
    # by a power of two changes neither the pooled order nor the ties
    B, Hkv, L, d, W, g = 1, 2, 150, 16, 8, 4
    q1, k, v = _bits(B, Hkv, Hkv, L, d, W, seed=4)
    q = np.repeat(q1, g, axis=1)
    grouped = orc.compress_grouped(q, k, v, 5, orc.POOL_MAX, 48)
    single = orc.compress(q1, k, v, 5, orc.POOL_MAX, 48)
    assert np.array_equal(grouped["vote"], 4.0 * single["vote"])
    assert np.array_equal(grouped["out_idx"], single["out_idx"])
    assert np.array_equal(grouped["out_k"], single["out_k"])


def test_structure_of_the_grouped_cache():
    B, Hq, Hkv, L, d, W, budget = 2, 8, 2, 200, 16, 8, 50
    q, k, v = _bits(B, Hq, Hkv, L, d, W, seed=5)
    ref = orc.compress_grouped(q, k, v, 7, orc.POOL_MAX, budget)
    n, ksel = L - W, budget - W
    assert ref["out_k"].shape == (B, Hkv, budget, d) and ref["out_idx"].shape == (B, Hkv, ksel)
    for b in range(B):
        for c in range(Hkv):
            idx = ref["out_idx"][b, c]
            assert np.all(np.diff(idx) > 0) and idx[0] >= 0 and idx[-1] < n
            assert np.array_equal(ref["out_k"][b, c, :ksel], k[b, c, idx])
            assert np.array_equal(ref["out_v"][b, c, :ksel], v[b, c, idx])
            assert np.array_equal(ref["out_k"][b, c, ksel:], k[b, c, n:])
            assert np.array_equal(ref["out_v"][b, c, ksel:], v[b, c, n:])
            # the chosen set has the largest pooled mass among all sets of its size
            order = np.sort(ref["pooled"][b, c])[::-1]
            assert math.isclose(ref["pooled"][b, c, idx].sum(), order[:ksel].sum(), rel_tol=1e-12)
    # group votes are at most g window sums: every window row spends at most 1
    assert np.all(ref["vote"].sum(axis=-1) <= (Hq // Hkv) * W + 1e-9)


def test_budget_at_least_L_keeps_the_cache_at_Hkv_heads():
    q, k, v = _bits(1, 4, 2, 60, 16, 8, seed=6)
    ref = orc.compress_grouped(q, k, v, 7, orc.POOL_MAX, 60)
    assert np.array_equal(ref["out_k"], k) and np.array_equal(ref["out_v"], v)
    assert np.array_equal(ref["out_idx"][0, 1], np.arange(52))


def test_supplied_lse_gives_the_recomputed_group_votes():
    q, k, v = _bits(1, 4, 2, 100, 16, 8, seed=7)
    a = orc.compress_grouped(q, k, v, 5, orc.POOL_AVG, 30)
    b = orc.compress_grouped(q, k, v, 5, orc.POOL_AVG, 30, lse=orc.lse_obs(q, k))
    assert np.allclose(a["vote"], b["vote"], rtol=1e-12, atol=0)
    assert np.array_equal(a["out_idx"], b["out_idx"])


# ---- planted mistakes: each must be caught by one of the pins above
_REAL_GROUP_VOTES = orc.group_votes


def _drops_last_head(vote_heads):
    return _REAL_GROUP_VOTES(vote_heads[:-1] if vote_heads.shape[0] > 1 else vote_heads)


def _takes_the_maximum(vote_heads):
    return vote_heads.max(axis=0)


def _averages(vote_heads):
    return _REAL_GROUP_VOTES(vote_heads) / 3.0   # a wrong constant, not a power of two


@pytest.mark.parametrize("wrong,pin", [
    (_drops_last_head, test_group_vote_matches_library_softmax_with_the_head_map_written_out),
    (_takes_the_maximum, test_uniform_attention_gives_g_times_the_harmonic_difference),
    (_averages, test_replicated_heads_select_what_the_single_head_selects),
])
def test_planted_mistakes_in_the_group_vote_are_caught(monkeypatch, wrong, pin):
    monkeypatch.setattr(orc, "group_votes", wrong)
    with pytest.raises(AssertionError):
        pin()


def test_a_wrong_head_map_is_caught(monkeypatch):
    # heads c, c + Hkv, ... instead of c*g .. c*g + g - 1
    real = orc.compress_grouped

    def interleaved(q, k, v, *a, **kw):
        B, Hq = q.shape[:2]
        Hkv = k.shape[1]
        g = Hq // Hkv
        perm = [c + j * Hkv for c in range(Hkv) for j in range(g)]
        return real(q[:, perm], k, v, *a, **kw)

    monkeypatch.setattr(orc, "compress_grouped", interleaved)
    with pytest.raises(AssertionError):
        test_group_vote_matches_library_softmax_with_the_head_map_written_out()
