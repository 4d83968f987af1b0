"""Pins for the oracle's supplied-normaliser variant (window_lse, votes_given_lse, lse_obs):
library log-sum-exp, a closed form, the identity with the recomputing path, a shift law, and
planted mistakes that these pins must catch.  CPU only."""
import math

import numpy as np
import pytest
import torch

from oracle import snapkv_oracle as orc
from paper_2404_14469_b200 import synth


def _logits(W=8, L=40, d=16, seed=0):
    rng = np.random.default_rng(seed)
    return orc.window_logits(rng.standard_normal((W, d)) * 2.0, rng.standard_normal((L, d)) * 2.0)


def test_lse_matches_library_logsumexp_on_visible_keys():
    s = _logits()
    W, L = s.shape
    n = L - W
    lse = orc.window_lse(s)
    for i in range(W):
        ref = torch.logsumexp(torch.from_numpy(s[i, : n + i + 1]), dim=0).item()
        assert abs(lse[i] - ref) < 1e-12
    # the mask is part of the definition: a huge logit at a key the row cannot see changes nothing
    # for that row, and dominates the next row, which does see it
    t = s.copy()
    t[:, n + 3] = 50.0
    lse2 = orc.window_lse(t)
    assert np.array_equal(lse2[:3], lse[:3])
    assert np.all(lse2[3:] > 49.9)


def test_lse_of_constant_logits_is_log_of_visible_count():
    W, L = 5, 23
    s = np.full((W, L), 0.75)
    lse = orc.window_lse(s)
    for i in range(W):
        assert abs(lse[i] - (0.75 + math.log(L - W + i + 1))) < 1e-13


def test_votes_with_own_lse_equal_recomputed_votes():
    s = _logits(seed=3)
    a = orc.votes_given_lse(s, orc.window_lse(s))
    b = orc.vote_from_probs(orc.window_softmax(s))
    assert np.allclose(a, b, rtol=1e-12, atol=0)


def test_shifted_lse_scales_that_rows_contribution():
    s = _logits(seed=4)
    lse = orc.window_lse(s)
    base = orc.votes_given_lse(s, lse)
    W, L = s.shape
    n = L - W
    bumped = lse.copy()
    bumped[2] += math.log(2.0)          # row 2 now counts half
    row2 = np.exp(s[2, :n] - lse[2])
    assert np.allclose(orc.votes_given_lse(s, bumped), base - 0.5 * row2, rtol=1e-12, atol=1e-300)


def test_uniform_attention_gives_harmonic_votes_through_lse():
    # q = 0: every visible key gets 1 / (n + i + 1); vote_j = H_L - H_n exactly
    W, L, d = 4, 30, 8
    n = L - W
    s = orc.window_logits(np.zeros((W, d)), np.random.default_rng(1).standard_normal((L, d)))
    v = orc.votes_given_lse(s, orc.window_lse(s))
    expect = sum(1.0 / t for t in range(n + 1, L + 1))
    assert np.allclose(v, expect, rtol=1e-13)


def test_lse_obs_and_compress_variant_follow_the_kv_head_map():
    data = synth.make_random(2, 4, 2, 96, 16, 8, seed=9)
    q, k, v = (synth.bf16_bits(data[x]) for x in ("q_obs", "k", "v"))
    lse = orc.lse_obs(q, k)
    assert lse.shape == (2, 4, 8)
    kf = orc.bf16_bits_to_f64(k[1, 1])
    s = orc.window_logits(orc.bf16_bits_to_f64(q[1, 3]), kf)   # head 3 reads KV head 1
    assert np.allclose(lse[1, 3], orc.window_lse(s), rtol=0, atol=0)
    full = orc.compress(q, k, v, 5, orc.POOL_MAX, 40)
    var = orc.compress(q, k, v, 5, orc.POOL_MAX, 40, lse=lse)
    assert np.allclose(var["vote"], full["vote"], rtol=1e-12)
    assert np.array_equal(var["out_idx"], full["out_idx"])
    assert np.array_equal(var["out_k"], full["out_k"]) and np.array_equal(var["out_v"], full["out_v"])


@pytest.mark.parametrize("mistake", ["plus_lse", "prefix_only_lse", "unmasked_lse", "lse_of_wrong_row"])
def test_planted_mistakes_are_caught(monkeypatch, mistake):
    s = _logits(seed=7)
    W, L = s.shape
    n = L - W

    def wrong_lse(x):
        if mistake == "prefix_only_lse":
            return np.array([torch.logsumexp(torch.from_numpy(x[i, :n]), 0).item() for i in range(W)])
        if mistake == "unmasked_lse":
            return np.array([torch.logsumexp(torch.from_numpy(x[i]), 0).item() for i in range(W)])
        return orc.window_lse(x)

    def wrong_votes(x, lse):
        if mistake == "plus_lse":
            return np.exp(x[:, :n] + lse[:, None]).sum(axis=0)
        if mistake == "lse_of_wrong_row":
            return np.exp(x[:, :n] - np.roll(lse, 1)[:, None]).sum(axis=0)
        return np.exp(x[:, :n] - lse[:, None]).sum(axis=0)

    good = orc.vote_from_probs(orc.window_softmax(s))
    bad = wrong_votes(s, wrong_lse(s))
    assert not np.allclose(bad, good, rtol=1e-9)
