"""Pins for the CPU oracle: every check here is fixed by the paper's definitions
or by mathematics, not by the oracle's own formulas (closed forms, invariants,
library routines, brute force on tiny inputs, planted-structure behaviour)."""
import itertools
import math
from fractions import Fraction

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import snapkv_oracle as orc
from paper_2404_14469_b200 import synth


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    t = torch.from_numpy(np.asarray(x, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16)


def harmonic(a: int) -> Fraction:
    return sum((Fraction(1, t) for t in range(1, a + 1)), Fraction(0))


# ---------------------------------------------------------------- widening
def test_bf16_widening_is_exact():
    vals = np.array([0.0, 1.0, -2.5, 3.140625, 2.0 ** -120, -(2.0 ** 100), 0.00390625], dtype=np.float32)
    bits = f32_to_bf16_bits(vals)
    assert np.array_equal(orc.bf16_bits_to_f64(bits), vals.astype(np.float64))
    # all finite bf16 patterns agree with torch's own widening
    allbits = np.arange(0, 1 << 16, dtype=np.uint32).astype(np.uint16)
    ref = torch.from_numpy(allbits.view(np.int16)).view(torch.bfloat16).to(torch.float64).numpy()
    got = orc.bf16_bits_to_f64(allbits)
    fin = np.isfinite(ref)
    assert np.array_equal(got[fin], ref[fin])


# ---------------------------------------------------------------- softmax / mask
def test_softmax_rows_sum_to_one_and_mask_is_causal():
    rng = np.random.default_rng(1)
    W, L = 5, 23
    s = rng.normal(size=(W, L)) * 3
    p = orc.window_softmax(s)
    n = L - W
    assert np.allclose(p.sum(axis=1), 1.0, atol=1e-14)
    for i in range(W):
        assert np.all(p[i, n + i + 1:] == 0.0)
        assert np.all(p[i, : n + i + 1] > 0.0)


def test_softmax_matches_library_softmax_with_causal_mask():
    rng = np.random.default_rng(2)
    W, L = 7, 40
    s = rng.normal(size=(W, L)) * 2
    n = L - W
    full_mask = torch.full((L, L), float("-inf"), dtype=torch.float64).triu(1)  # textbook causal mask
    st = torch.from_numpy(s) + full_mask[n:, :]
    ref = torch.softmax(st, dim=-1).numpy()
    assert np.allclose(orc.window_softmax(s), ref, rtol=1e-13, atol=0)


def test_window_key_change_does_not_reach_earlier_rows():
    rng = np.random.default_rng(3)
    W, L, d = 4, 12, 8
    q = rng.normal(size=(W, d))
    k = rng.normal(size=(L, d))
    base = orc.window_softmax(orc.window_logits(q, k))
    n = L - W
    k2 = k.copy()
    k2[n + 2] += 5.0  # window key i' = 2
    pert = orc.window_softmax(orc.window_logits(q, k2))
    assert np.array_equal(base[:2], pert[:2])          # rows 0, 1 cannot see it
    assert not np.allclose(base[2:], pert[2:])         # rows 2, 3 do


def test_single_row_window_is_a_plain_softmax():
    rng = np.random.default_rng(4)
    L, d = 17, 16
    q = rng.normal(size=(1, d))
    k = rng.normal(size=(L, d))
    s = (k @ q[0]) / math.sqrt(d)
    e = np.exp(s - s.max())
    ref = e / e.sum()
    vt = orc.window_votes(q, k)
    assert vt.shape == (L - 1,)
    assert np.allclose(vt, ref[:-1], rtol=1e-13)


def test_logit_scale_and_orientation_two_level_closed_form():
    # d = 4 so sqrt(d) = 2; q = (2,0,0,0); keys (x,0,0,0) with x in {0,1}: logit = x.
    # Row i sees n + i + 1 keys; p = e^x / (#zeros + e * #ones) among the visible ones.
    L, W, d = 12, 3, 4
    n = L - W
    x = np.array([0, 1, 0, 0, 1, 1, 0, 0, 0, 1, 0, 1], dtype=np.float64)
    k = np.zeros((L, d))
    k[:, 0] = x
    q = np.zeros((W, d))
    q[:, 0] = 2.0
    q[:, 1] = 7.0  # multiplies key zeros: must not matter (catches a transposed operand)
    expect = np.zeros(n)
    for i in range(W):
        vis = x[: n + i + 1]
        denom = (vis == 0).sum() + math.e * (vis == 1).sum()
        expect += np.exp(x[:n]) / denom
    got = orc.window_votes(q, k)
    assert np.allclose(got, expect, rtol=1e-13)


# ---------------------------------------------------------------- vote closed forms
@pytest.mark.parametrize("L,W", [(9, 3), (64, 16), (1024, 32)])
def test_uniform_attention_gives_harmonic_votes(L, W):
    # q = 0 -> every visible key gets 1/(n+i+1); vote_j = H_L - H_n for every prefix j.
    d = 8
    n = L - W
    rng = np.random.default_rng(5)
    k = rng.normal(size=(L, d))
    q = np.zeros((W, d))
    expect = float(harmonic(L) - harmonic(n))
    got = orc.window_votes(q, k)
    assert got.shape == (n,)
    assert np.allclose(got, expect, rtol=1e-13)


def test_vote_mass_identity():
    # sum_j vote_j + (probability mass the window rows put on window keys) = W
    rng = np.random.default_rng(6)
    W, L, d = 6, 50, 16
    q = rng.normal(size=(W, d))
    k = rng.normal(size=(L, d))
    p = orc.window_softmax(orc.window_logits(q, k))
    vt = orc.vote_from_probs(p)
    n = L - W
    assert math.isclose(vt.sum() + p[:, n:].sum(), W, rel_tol=1e-13)
    assert np.all(vt > 0)
    assert np.all(vt < W)


def test_vote_invariant_to_row_constant():
    rng = np.random.default_rng(7)
    W, L = 4, 30
    s = rng.normal(size=(W, L))
    shift = rng.normal(size=(W, 1)) * 10
    a = orc.vote_from_probs(orc.window_softmax(s))
    b = orc.vote_from_probs(orc.window_softmax(s + shift))
    assert np.allclose(a, b, rtol=1e-12)


def test_votes_wrapper_uses_shared_kv_head():
    w = synth.make_random(2, 4, 2, 40, 16, 5, seed=8)
    q, k = synth.bf16_bits(w["q_obs"]), synth.bf16_bits(w["k"])
    got = orc.votes(q, k)
    for b in range(2):
        for h in range(4):
            ref = orc.window_votes(orc.bf16_bits_to_f64(q[b, h]), orc.bf16_bits_to_f64(k[b, h // 2]))
            assert np.array_equal(got[b, h], ref)
    assert np.array_equal(orc.votes(q, k, workers=3), got)


# ---------------------------------------------------------------- pooling
@pytest.mark.parametrize("kernel", [1, 3, 5, 7, 13])
@pytest.mark.parametrize("p", [0, 1, 10, 28, 29])
def test_pool_of_a_delta(kernel, p):
    n = 30
    r = kernel // 2
    vote = np.zeros(n)
    vote[p] = 1.0
    lo, hi = max(0, p - r), min(n, p + r + 1)
    mx = orc.pool1d(vote, kernel, orc.POOL_MAX)
    av = orc.pool1d(vote, kernel, orc.POOL_AVG)
    expect = np.zeros(n)
    expect[lo:hi] = 1.0
    assert np.array_equal(mx, expect)
    assert np.allclose(av, expect / kernel, rtol=1e-15)


def test_pool_kernel_one_is_identity_and_even_is_rejected():
    rng = np.random.default_rng(9)
    v = rng.random(20)
    assert np.array_equal(orc.pool1d(v, 1, orc.POOL_MAX), v)
    assert np.array_equal(orc.pool1d(v, 1, orc.POOL_AVG), v)
    with pytest.raises(ValueError):
        orc.pool1d(v, 4, orc.POOL_MAX)


@pytest.mark.parametrize("kernel", [3, 5, 7, 13])
def test_pool_matches_library_pooling(kernel):
    rng = np.random.default_rng(10)
    v = rng.random(101)
    t = torch.from_numpy(v)[None, None, :]
    ref_max = F.max_pool1d(t, kernel_size=kernel, padding=kernel // 2, stride=1)[0, 0].numpy()
    ref_avg = F.avg_pool1d(t, kernel_size=kernel, padding=kernel // 2, stride=1,
                           count_include_pad=True)[0, 0].numpy()
    assert np.array_equal(orc.pool1d(v, kernel, orc.POOL_MAX), ref_max)
    assert np.allclose(orc.pool1d(v, kernel, orc.POOL_AVG), ref_avg, rtol=1e-14)


# ---------------------------------------------------------------- top-k
def test_topk_brute_force_maximises_the_kept_mass():
    rng = np.random.default_rng(11)
    for n, k in [(8, 3), (12, 5), (10, 10), (9, 0), (11, 1)]:
        pooled = rng.random(n)
        best = max(itertools.combinations(range(n), k), key=lambda S: sum(pooled[list(S)]))
        assert list(orc.topk_positions(pooled, k)) == sorted(best)


def test_topk_ties_go_to_lower_positions_and_output_is_ascending():
    pooled = np.array([0.5, 0.9, 0.5, 0.9, 0.5, 0.1, 0.5])
    assert list(orc.topk_positions(pooled, 2)) == [1, 3]
    assert list(orc.topk_positions(pooled, 3)) == [0, 1, 3]
    assert list(orc.topk_positions(pooled, 4)) == [0, 1, 2, 3]
    assert list(orc.topk_positions(pooled, 5)) == [0, 1, 2, 3, 4]
    assert list(orc.topk_positions(np.ones(6), 3)) == [0, 1, 2]


def test_topk_matches_textbook_sort():
    rng = np.random.default_rng(12)
    pooled = rng.random(200)
    k = 37
    ref = sorted(sorted(range(200), key=lambda j: (-pooled[j], j))[:k])
    assert list(orc.topk_positions(pooled, k)) == ref


def test_topk_nesting_across_budgets():
    rng = np.random.default_rng(13)
    pooled = orc.pool1d(rng.random(500), 7, orc.POOL_MAX)  # plateaus -> real ties
    prev = set()
    for k in (10, 50, 200, 500):
        cur = set(orc.topk_positions(pooled, k).tolist())
        assert len(cur) == k and prev <= cur
        prev = cur


# ---------------------------------------------------------------- whole step
def _step_head_by_head(q_bits, k_bits, v_bits, W, budget, kernel, pool_type):
    """Second, independent statement of the whole step (Sec. 4, Eq. 1-2), MHA, fp64, one head
    at a time: each window row is an ordinary attention row over the keys it may see
    (library log-sum-exp), Eq. 1 adds the rows, a sliding-window view does the pooling, a
    sort of (value, position) pairs ranks the positions, and the kept rows are picked by
    plain indexing."""
    tq = orc.bf16_bits_to_f64(q_bits)
    tk = orc.bf16_bits_to_f64(k_bits)
    B, H, L, d = tk.shape
    n, r, ksel = L - W, kernel // 2, budget - W
    vote = np.zeros((B, H, n))
    pooled = np.zeros((B, H, n))
    idx = np.zeros((B, H, ksel), dtype=np.int64)
    ck = np.zeros((B, H, budget, d), dtype=np.uint16)
    cv = np.zeros((B, H, budget, d), dtype=np.uint16)
    for b, h in itertools.product(range(B), range(H)):
        for i in range(W):
            seen = n + i + 1                                    # the prefix and the window up to row i
            row = torch.from_numpy(tk[b, h, :seen] @ tq[b, h, i]) / math.sqrt(d)
            vote[b, h] += torch.exp(row - torch.logsumexp(row, dim=0)).numpy()[:n]
        padded = np.concatenate([np.zeros(r), vote[b, h], np.zeros(r)])   # votes are >= 0
        windows = np.lib.stride_tricks.sliding_window_view(padded, kernel)
        pooled[b, h] = windows.max(axis=1) if pool_type == orc.POOL_MAX else windows.sum(axis=1) / kernel
        ranked = sorted(range(n), key=lambda j: pooled[b, h, j], reverse=True)
        idx[b, h] = np.array(ranked[:ksel])
        keep = np.sort(idx[b, h])
        ck[b, h] = np.concatenate([k_bits[b, h, keep], k_bits[b, h, n:]])
        cv[b, h] = np.concatenate([v_bits[b, h, keep], v_bits[b, h, n:]])
    return vote, pooled, idx, ck, cv


@pytest.mark.parametrize("pool_type,kernel", [(orc.POOL_MAX, 7), (orc.POOL_AVG, 5), (orc.POOL_MAX, 1)])
def test_whole_step_against_library_ops(pool_type, kernel):
    W, budget = 8, 40
    w = synth.make_random(2, 3, 3, 150, 32, W, seed=14, q_scale=2.0)
    q, k, v = (synth.bf16_bits(w[x]) for x in ("q_obs", "k", "v"))
    res = orc.compress(q, k, v, kernel, pool_type, budget)
    vote, pooled, idx, ck, cv = _step_head_by_head(q, k, v, W, budget, kernel, pool_type)
    assert np.allclose(res["vote"], vote, rtol=1e-12)
    assert np.allclose(res["pooled"], pooled, rtol=1e-12)
    ksel = budget - W
    for b in range(2):
        for h in range(3):
            mine = res["out_idx"][b, h]
            theirs = np.sort(idx[b, h])
            # identical unless an exact tie straddles the k-th boundary (max pooling
            # makes exact ties; the library's tie order is unspecified)
            if not np.array_equal(mine, theirs):
                P = res["pooled"][b, h]
                t = np.sort(P)[::-1][ksel - 1]
                diff = set(mine.tolist()) ^ set(theirs.tolist())
                assert all(P[j] == t for j in diff)
            rows_k = {bytes(r) for r in res["out_k"][b, h, :ksel]}
            assert res["out_k"].shape == (2, 3, budget, 32)
            # window rows bit-exact and last
            assert np.array_equal(res["out_k"][b, h, ksel:], ck[b, h, ksel:].astype(np.uint16))
            assert np.array_equal(res["out_v"][b, h, ksel:], cv[b, h, ksel:].astype(np.uint16))
            if np.array_equal(mine, theirs):
                assert rows_k == {bytes(r) for r in ck[b, h, :ksel].astype(np.uint16)}


def test_output_structure_and_bit_exact_gather():
    W, budget, kernel = 4, 24, 3
    w = synth.make_random(1, 4, 2, 90, 16, W, seed=15)
    q, k, v = (synth.bf16_bits(w[x]) for x in ("q_obs", "k", "v"))
    res = orc.compress(q, k, v, kernel, orc.POOL_MAX, budget)
    n = 90 - W
    assert res["out_k"].shape == (1, 4, budget, 16) and res["out_idx"].shape == (1, 4, budget - W)
    for h in range(4):
        idx = res["out_idx"][0, h]
        assert np.all(np.diff(idx) > 0) and idx.min() >= 0 and idx.max() < n
        c = h // 2
        assert np.array_equal(res["out_k"][0, h, : budget - W], k[0, c, idx])
        assert np.array_equal(res["out_v"][0, h, : budget - W], v[0, c, idx])
        assert np.array_equal(res["out_k"][0, h, budget - W:], k[0, c, n:])
        assert np.array_equal(res["out_v"][0, h, budget - W:], v[0, c, n:])


@pytest.mark.parametrize("budget", [90, 91, 500])
def test_budget_at_least_L_is_identity(budget):
    W = 4
    w = synth.make_random(2, 4, 2, 90, 16, W, seed=16)
    q, k, v = (synth.bf16_bits(w[x]) for x in ("q_obs", "k", "v"))
    res = orc.compress(q, k, v, 7, orc.POOL_MAX, budget)
    assert res["out_k"].shape == (2, 4, 90, 16)
    for h in range(4):
        assert np.array_equal(res["out_k"][:, h], k[:, h // 2])
        assert np.array_equal(res["out_v"][:, h], v[:, h // 2])
        assert np.array_equal(res["out_idx"][0, h], np.arange(90 - W))


def test_gqa_equals_mha_on_repeated_kv():
    W = 6
    w = synth.make_random(1, 6, 2, 120, 32, W, seed=17, q_scale=2.0)
    q, k, v = (synth.bf16_bits(w[x]) for x in ("q_obs", "k", "v"))
    a = orc.compress(q, k, v, 5, orc.POOL_AVG, 30)
    krep, vrep = np.repeat(k, 3, axis=1), np.repeat(v, 3, axis=1)
    b = orc.compress(q, krep, vrep, 5, orc.POOL_AVG, 30)
    for key in ("out_k", "out_v", "out_idx", "vote", "pooled"):
        assert np.array_equal(a[key], b[key])


def test_heads_subset_and_workers_agree_with_full_run():
    W = 4
    w = synth.make_random(2, 4, 2, 80, 16, W, seed=18)
    q, k, v = (synth.bf16_bits(w[x]) for x in ("q_obs", "k", "v"))
    full = orc.compress(q, k, v, 3, orc.POOL_MAX, 20)
    part = orc.compress(q, k, v, 3, orc.POOL_MAX, 20, heads=[(1, 3)], workers=2)
    assert np.array_equal(full["out_idx"][1, 3], part["out_idx"][1, 3])
    assert np.array_equal(full["out_k"][1, 3], part["out_k"][1, 3])
    assert not part["out_idx"][0, 0].any()


def test_invalid_arguments_raise():
    w = synth.make_random(1, 2, 2, 30, 16, 4, seed=19)
    q, k, v = (synth.bf16_bits(w[x]) for x in ("q_obs", "k", "v"))
    with pytest.raises(ValueError):
        orc.compress(q, k, v, 3, orc.POOL_MAX, 4)       # budget <= W
    with pytest.raises(ValueError):
        orc.compress(q, k, v, 2, orc.POOL_MAX, 10)      # even kernel
    with pytest.raises(ValueError):
        orc.compress(q[:, :1].repeat(3, axis=1), k, v, 3, orc.POOL_MAX, 10)  # Hq % Hkv != 0


# ---------------------------------------------------------------- behaviour (Sec. 4.3, 5.1.1)
def test_planted_clusters_are_retrieved_on_the_tiny_workload():
    w = synth.WORKLOADS[0]
    data = synth.make_layer(w, 0)
    q, k, v = (synth.bf16_bits(data[x]) for x in ("q_obs", "k", "v"))
    res = orc.compress(q, k, v, w.pool_kernel, orc.POOL_MAX, w.budgets[0])
    starts = data["starts"][0].tolist()
    assert len(starts) == 3
    for h in range(w.Hq):
        kept = set(res["out_idx"][0, h].tolist())
        for s in starts:
            assert set(range(s, s + synth.CLUSTER_LEN)) <= kept
        # pooling keeps the neighbours of a peak with it: every position within r of
        # a cluster's strongest key shares that key's pooled value
        r = w.pool_kernel // 2
        for s in starts:
            peak = s + int(np.argmax(res["vote"][0, h, s:s + synth.CLUSTER_LEN]))
            assert set(range(max(0, peak - r), min(w.n, peak + r + 1))) <= kept


def test_needle_is_retrieved_at_any_depth():
    # a scaled-down stand-in for the single-needle workload: one planted run, budget ~1%
    base = synth.Workload(9, "needle-small", 1, 2, 2, 64, 4096, 32, 7, "max", (96,), 1, 1)
    for layer in range(4):  # different seeds -> different depths
        data = synth.make_layer(base, layer)
        q, k, v = (synth.bf16_bits(data[x]) for x in ("q_obs", "k", "v"))
        res = orc.compress(q, k, v, 7, orc.POOL_MAX, 96)
        s = int(data["starts"][0][0])
        for h in range(2):
            kept = set(res["out_idx"][0, h].tolist())
            assert kept & set(range(s, s + synth.CLUSTER_LEN))
