"""Acceptance rule shared by the GPU parity tests (helpers only, no CUDA, no oracle maths).

With P the oracle's pooled votes of one head, t its ksel-th largest value and eps = 1e-3:
  votes    |vote_gpu - vote_orc| <= eps * vote_orc (+1e-30 for exp flushed to zero)
  indices  exactly ksel, strictly ascending, all in [0, n);
           {j : P_j > t (1 + eps)}  is a subset of idx  is a subset of  {j : P_j >= t (1 - eps)}
  rows     out_k / out_v rows bit-equal to k / v at out_idx, window rows last.
fp32 accumulation of bf16 products and exp2 with ~2^-22 relative error put the vote
error near 1e-5, two orders inside eps.
"""
import numpy as np

EPS = 1e-3


def check_votes(vote_gpu: np.ndarray, vote_orc: np.ndarray):
    err = np.abs(vote_gpu.astype(np.float64) - vote_orc)
    bound = EPS * np.abs(vote_orc) + 1e-30
    bad = err > bound
    assert not bad.any(), (
        f"{int(bad.sum())} votes off; worst rel err "
        f"{float((err / np.maximum(np.abs(vote_orc), 1e-300)).max()):.3e}")
    return float((err / np.maximum(np.abs(vote_orc), 1e-300)).max())


def check_indices(idx_gpu: np.ndarray, pooled_orc: np.ndarray, ksel: int, idx_orc=None):
    """One head.  Returns True when the set equals the oracle's exactly."""
    n = pooled_orc.shape[0]
    idx = idx_gpu.astype(np.int64)
    assert idx.shape == (ksel,)
    assert idx.min() >= 0 and idx.max() < n
    assert np.all(np.diff(idx) > 0), "indices must be strictly ascending"
    t = np.sort(pooled_orc)[::-1][ksel - 1]
    must = np.nonzero(pooled_orc > t * (1 + EPS))[0]
    may = pooled_orc >= t * (1 - EPS)
    chosen = np.zeros(n, dtype=bool)
    chosen[idx] = True
    assert chosen[must].all(), "a clearly-above-threshold position was dropped"
    assert may[idx].all(), "a clearly-below-threshold position was kept"
    if idx_orc is not None:
        return bool(np.array_equal(idx, idx_orc))
    return True


def check_rows(out_k, out_v, k_head, v_head, idx, W):
    """One head, uint16 bit patterns: gathered rows then the window rows."""
    L = k_head.shape[0]
    n = L - W
    ksel = idx.shape[0]
    assert out_k.shape[0] == ksel + W
    assert np.array_equal(out_k[:ksel], k_head[idx])
    assert np.array_equal(out_v[:ksel], v_head[idx])
    assert np.array_equal(out_k[ksel:], k_head[n:])
    assert np.array_equal(out_v[ksel:], v_head[n:])
