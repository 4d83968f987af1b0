"""Pins for the oracle's hit-rate measure (Sec. 3, Eq. 3-7): brute force, closed forms, bounds,
and planted mistakes.  CPU only."""
import numpy as np
import pytest

from oracle import snapkv_oracle as orc


def _case(N=3, n=50, k=12, seed=0):
    rng = np.random.default_rng(seed)
    a = rng.random((N, n)).astype(np.float32)
    idx = np.stack([np.sort(rng.choice(n, size=k, replace=False)) for _ in range(N)])
    return a, idx


def test_brute_force_on_small_inputs():
    a, idx = _case()
    theta = np.float32(0.6)
    c = orc.hit_counts(a, idx, theta)
    for h in range(a.shape[0]):
        important = [j for j in range(a.shape[1]) if a[h, j] > theta]
        hits = [j for j in important if j in set(idx[h].tolist())]
        assert c[h, 0] == len(hits) and c[h, 1] == len(important)
    tot_hits = sum(1 for h in range(3) for j in idx[h] if a[h, j] > theta)
    tot_imp = int((a > theta).sum())
    assert orc.hit_rate(a, idx, theta) == tot_hits / tot_imp


def test_threshold_below_everything_gives_k_over_n():
    a, idx = _case(N=4, n=40, k=10, seed=1)
    assert orc.hit_rate(a, idx, -1.0) == 10 / 40
    assert np.array_equal(orc.hit_counts(a, idx, -1.0), np.tile([10, 40], (4, 1)))


def test_selecting_everything_hits_everything_and_a_disjoint_selection_nothing():
    a, _ = _case(N=2, n=30, seed=2)
    everything = np.tile(np.arange(30), (2, 1))
    assert orc.hit_rate(a, everything, 0.5) == 1.0
    # select exactly the unimportant positions of each head (same count per head needed: pad)
    a2 = np.zeros((2, 8), dtype=np.float32)
    a2[:, :4] = 1.0
    assert orc.hit_rate(a2, np.tile(np.arange(4, 8), (2, 1)), 0.5) == 0.0
    assert np.isnan(orc.hit_rate(a2, np.tile(np.arange(4), (2, 1)), 2.0))


def test_the_comparison_is_strict_and_per_head():
    a = np.array([[0.5, 0.5, 0.7, 0.2], [0.9, 0.1, 0.5, 0.6]], dtype=np.float32)
    idx = np.array([[0, 2], [1, 2]])
    # theta = 0.5: 0.5 itself is not important (Eq. 5 uses >)
    assert np.array_equal(orc.hit_counts(a, idx, 0.5), [[1, 1], [0, 2]])
    assert orc.hit_rate(a, idx, 0.5) == 1 / 3
    # bounds: hits <= min(k, important)
    c = orc.hit_counts(*_case(seed=5), 0.3)
    assert np.all(c[:, 0] <= np.minimum(12, c[:, 1]))


# ---- planted mistakes
def _geq(a_cur, idx, theta):
    a = np.asarray(a_cur, dtype=np.float32)
    m_vote = np.zeros(a.shape, dtype=bool)
    for h in range(a.shape[0]):
        m_vote[h, idx[h]] = True
    m_thr = a >= np.float32(theta)
    return np.stack([(m_thr & m_vote).sum(axis=1), m_thr.sum(axis=1)], axis=1).astype(np.int64)


def _shared_mask(a_cur, idx, theta):
    a = np.asarray(a_cur, dtype=np.float32)
    m_vote = np.zeros(a.shape, dtype=bool)
    m_vote[:, idx[0]] = True            # head 0's selection used for every head
    m_thr = a > np.float32(theta)
    return np.stack([(m_thr & m_vote).sum(axis=1), m_thr.sum(axis=1)], axis=1).astype(np.int64)


@pytest.mark.parametrize("wrong", [_geq, _shared_mask])
def test_planted_mistakes_are_caught(monkeypatch, wrong):
    monkeypatch.setattr(orc, "hit_counts", wrong)
    with pytest.raises(AssertionError):
        test_the_comparison_is_strict_and_per_head()
