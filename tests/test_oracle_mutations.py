"""The pins must be sharp: plant one plausible mistake at a time in the oracle (on
the CPU, by patching its functions) and check that some pin then fails."""
import math

import numpy as np
import pytest

from oracle import snapkv_oracle as orc
import test_oracle_pins as pins


def _softmax_mask_off_by_one(s):
    W, L = s.shape
    n = L - W
    vis = np.arange(L)[None, :] < (n + np.arange(W)[:, None])   # drops the diagonal
    m = np.where(vis, s, -np.inf).max(axis=1, keepdims=True)
    e = np.where(vis, np.exp(s - m), 0.0)
    return e / e.sum(axis=1, keepdims=True)


def _softmax_no_mask(s):
    e = np.exp(s - s.max(axis=1, keepdims=True))
    return e / e.sum(axis=1, keepdims=True)


def _softmax_prefix_only_normaliser(s):
    W, L = s.shape
    n = L - W
    out = np.zeros_like(s)
    e = np.exp(s[:, :n] - s[:, :n].max(axis=1, keepdims=True))
    out[:, :n] = e / e.sum(axis=1, keepdims=True)
    return out


def _logits_no_scale(q, k):
    return q @ k.T


def _logits_wrong_scale(q, k):
    return (q @ k.T) / q.shape[-1]


def _vote_mean(p):
    W, L = p.shape
    return p[:, : L - W].mean(axis=0)


def _vote_drop_last_row(p):
    W, L = p.shape
    return p[:-1, : L - W].sum(axis=0)


def _pool_avg_valid_count(vote, kernel, pool_type):
    n, r = vote.shape[0], kernel // 2
    out = np.empty(n)
    for j in range(n):
        w = vote[max(0, j - r): min(n, j + r + 1)]
        out[j] = w.max() if pool_type == orc.POOL_MAX else w.mean()
    return out


def _pool_one_sided(vote, kernel, pool_type):
    n = vote.shape[0]
    out = np.empty(n)
    for j in range(n):
        w = vote[j: min(n, j + kernel)]
        out[j] = w.max() if pool_type == orc.POOL_MAX else w.sum() / kernel
    return out


def _topk_smallest(pooled, k):
    return np.sort(np.argsort(pooled, kind="stable")[:k])


def _topk_ties_high(pooled, k):
    n = pooled.shape[0]
    order = sorted(range(n), key=lambda j: (-pooled[j], -j))
    return np.sort(np.array(order[:k], dtype=np.int64))


MUTANTS = [
    ("window_softmax", _softmax_mask_off_by_one,
     [lambda: pins.test_uniform_attention_gives_harmonic_votes(64, 16),
      pins.test_softmax_matches_library_softmax_with_causal_mask]),
    ("window_softmax", _softmax_no_mask,
     [pins.test_softmax_rows_sum_to_one_and_mask_is_causal,
      pins.test_window_key_change_does_not_reach_earlier_rows]),
    ("window_softmax", _softmax_prefix_only_normaliser,
     [pins.test_logit_scale_and_orientation_two_level_closed_form,
      lambda: pins.test_uniform_attention_gives_harmonic_votes(9, 3)]),
    ("window_logits", _logits_no_scale, [pins.test_logit_scale_and_orientation_two_level_closed_form,
                                         pins.test_single_row_window_is_a_plain_softmax]),
    ("window_logits", _logits_wrong_scale, [pins.test_logit_scale_and_orientation_two_level_closed_form]),
    ("vote_from_probs", _vote_mean, [lambda: pins.test_uniform_attention_gives_harmonic_votes(9, 3)]),
    ("vote_from_probs", _vote_drop_last_row, [pins.test_vote_mass_identity]),
    ("pool1d", _pool_avg_valid_count, [lambda: pins.test_pool_of_a_delta(5, 0),
                                       lambda: pins.test_pool_matches_library_pooling(7)]),
    ("pool1d", _pool_one_sided, [lambda: pins.test_pool_of_a_delta(5, 10)]),
    ("topk_positions", _topk_smallest, [pins.test_topk_brute_force_maximises_the_kept_mass]),
    ("topk_positions", _topk_ties_high, [pins.test_topk_ties_go_to_lower_positions_and_output_is_ascending]),
]


@pytest.mark.parametrize("name,mutant,catchers", MUTANTS, ids=[m[1].__name__ for m in MUTANTS])
def test_planted_mistake_is_caught(monkeypatch, name, mutant, catchers):
    monkeypatch.setattr(orc, name, mutant)
    for check in catchers:
        with pytest.raises(AssertionError):
            check()
