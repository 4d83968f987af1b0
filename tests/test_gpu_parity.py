"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle, element by
element on the same seeded inputs.  Small cases span several 128-key tiles and a ragged
tail; the full-size workloads are checked on sampled heads."""
import numpy as np
import pytest
import torch

from oracle import snapkv_oracle as orc
from paper_2404_14469_b200 import binding as sk
from paper_2404_14469_b200 import synth

import parity

pytestmark = pytest.mark.gpu

PT = {"max": sk.POOL_MAX, "avg": sk.POOL_AVG}


def _to_dev(data):
    return {x: data[x].cuda() for x in ("q_obs", "k", "v")}


def _bits(t):
    return synth.bf16_bits(t)


def _oracle_head(q_bits, k_bits, b, h, g):
    return orc.window_votes(orc.bf16_bits_to_f64(q_bits[b, h]), orc.bf16_bits_to_f64(k_bits[b, h // g]))


# ------------------------------------------------------------------ scoring
SCORE_SHAPES = [
    # B, Hq, Hkv, L, d, W
    (1, 4, 4, 1024, 64, 32),      # tiny workload shape
    (2, 4, 2, 1000, 128, 32),     # GQA, ragged L (not a tile multiple)
    (1, 8, 2, 777, 128, 32),      # g*W = 128: one unit per KV head
    (1, 8, 1, 900, 64, 32),       # g*W = 256: two head sub-groups per KV head
    (1, 2, 2, 600, 128, 16),      # W = 16 (paper's needle setting)
    (1, 4, 2, 1500, 128, 64),     # W = 64 (Command-R setting)
    (1, 3, 3, 300, 64, 5),        # odd window, generic column path
    (1, 6, 2, 410, 128, 24),      # W not a multiple of 16, GQA
    (1, 2, 2, 129, 128, 1),       # one-row window
    (1, 1, 1, 40, 64, 32),        # L shorter than one tile
    (1, 2, 1, 5000, 128, 128),    # W = 128
    (3, 2, 2, 257, 64, 32),       # batch > 1, prefix of 225 keys
]


@pytest.mark.parametrize("B,Hq,Hkv,L,d,W", SCORE_SHAPES)
def test_window_scores_match_oracle(B, Hq, Hkv, L, d, W):
    data = synth.make_random(B, Hq, Hkv, L, d, W, seed=L + W, q_scale=1.5)
    dev = _to_dev(data)
    vote, ws = sk.snapkv_window_scores(dev["q_obs"], dev["k"])
    code, detail = sk.snapkv_device_status(ws)
    assert code == sk.OK, (code, detail)
    got = vote.cpu().numpy()
    ref = orc.votes(_bits(data["q_obs"]), _bits(data["k"]))
    assert got.shape == ref.shape == (B, Hq, L - W)
    parity.check_votes(got, ref)


def test_window_scores_with_large_logits():
    # All window rows of a head point the same way, scaled so that the logits spread over
    # about +-50: the running maximum must keep exp2 in range, and the smallest votes fall
    # far below the largest ones (a vote is small only if every row's probability is).
    B, Hq, Hkv, L, d, W = 1, 4, 2, 2000, 128, 32
    data = synth.make_random(B, Hq, Hkv, L, d, W, seed=3)
    g = torch.Generator().manual_seed(33)
    u = torch.randn(B, Hq, 1, d, generator=g)
    u = u / u.norm(dim=-1, keepdim=True)
    data["q_obs"] = (170.0 * u + torch.randn(B, Hq, W, d, generator=g)).to(torch.bfloat16)
    dev = _to_dev(data)
    vote, _ = sk.snapkv_window_scores(dev["q_obs"], dev["k"])
    ref = orc.votes(_bits(data["q_obs"]), _bits(data["k"]))
    got = vote.cpu().numpy()
    assert np.isfinite(got).all()
    # The acceptance rule as it stands, floor of 1e-30 included: a vote is a sum of
    # exp2(x - lse) with x - lse accurate to a few ulp of ~100 (1e-5 relative in the result),
    # and fp32 only flushes results below 1.2e-38 to zero, far under the floor.
    assert ref.min() < 1e-30 and np.any((ref > 1e-29) & (ref < 1e-20)) and ref.max() > 1e-2
    parity.check_votes(got, ref)


def test_uniform_attention_closed_form_on_gpu():
    # q = 0: every prefix key gets vote H_L - H_n (the oracle's closed-form pin, on the GPU)
    B, Hq, Hkv, L, d, W = 1, 2, 2, 1000, 128, 32
    data = synth.make_random(B, Hq, Hkv, L, d, W, seed=1)
    q0 = torch.zeros_like(data["q_obs"]).cuda()
    vote, _ = sk.snapkv_window_scores(q0, data["k"].cuda())
    expect = sum(1.0 / t for t in range(L - W + 1, L + 1))
    assert np.allclose(vote.cpu().numpy(), expect, rtol=1e-5)


# ------------------------------------------------------------------ pool + top-k
@pytest.mark.parametrize("rows,n,kernel,ptype,ksel", [
    (4, 992, 7, "max", 224),
    (3, 1000, 5, "avg", 100),
    (2, 4097, 1, "max", 1),
    (2, 33, 13, "max", 33),
    (5, 20000, 7, "max", 2016),
    (2, 60000, 7, "max", 4064),     # longer than the on-chip key buffer: scratch path
    (2, 60001, 5, "avg", 1000),
    (1, 7, 7, "avg", 3),
    (2, 3000, 63, "max", 1500),
    (2, 40960, 5, "avg", 4064),     # longest row of the vectorised one-CTA kernel (40 keys a thread)
    (2, 40961, 7, "max", 4064),     # one more: generic one-CTA kernel, keys still on chip
    (1, 49152, 13, "max", 8128),
    (3, 32736, 13, "avg", 4064),    # radius 6 with its own instantiation
    (2, 16352, 3, "max", 992),      # radius 1: run-time radius path
    # one cluster of CTAs per row: 4096 to 131072 positions, pooling radius up to 7
    (3, 4095, 7, "max", 500),       # just below: one CTA per row
    (3, 4096, 7, "max", 500),       # two CTAs of 8 keys a thread
    (2, 4100, 5, "avg", 4099),
    (2, 16384, 15, "avg", 2016),    # radius 7, run-time radius
    (2, 16385, 7, "max", 2016),     # 16 keys a thread, last CTA nearly empty
    (4, 32736, 5, "avg", 4064),     # the 32K workload's rows: 8 CTAs of 16 keys a thread
    (2, 65536, 7, "max", 8128),     # 8 CTAs of 32 keys a thread, full
    (2, 65537, 7, "max", 8128),     # 16 CTAs
    (2, 131008, 7, "max", 8128),    # the 128K workload's rows
    (1, 131072, 5, "avg", 2016),
    (1, 131073, 7, "max", 2016),    # one more: many-CTA path with global scratch
    (2, 140000, 7, "max", 4064),
    (1, 150001, 5, "avg", 1000),
    (50, 20000, 7, "max", 2016),    # more rows than the cluster kernel takes on: one CTA per row
    (49, 32736, 5, "avg", 4064),
    (64, 40960, 13, "max", 31000),
    (2, 20000, 17, "max", 2016),    # radius 8: beyond the cluster kernel, one CTA per row
    (1, 70000, 17, "avg", 2016),    # radius 8, long row: many-CTA path
])
def test_pool_topk_matches_oracle(rows, n, kernel, ptype, ksel):
    g = torch.Generator().manual_seed(n + kernel)
    vote = torch.rand(rows, n, generator=g, dtype=torch.float32) ** 4
    idx = sk.snapkv_pool_topk(vote.cuda(), kernel, PT[ptype], ksel).cpu().numpy()
    for r in range(rows):
        pooled = orc.pool1d(vote[r].numpy().astype(np.float64), kernel, PT[ptype])
        ref = orc.topk_positions(pooled, ksel)
        same = parity.check_indices(idx[r], pooled, ksel, ref)
        if ptype == "max":  # max of fp32 values is exact: ties included, the sets must be equal
            assert same


@pytest.mark.parametrize("rows,n,kernel,ptype,ksel", [
    (2, 40960, 7, "max", 32767),    # one below / at the point where a 16-bit count reaches bit 15
    (2, 40960, 7, "max", 32768),
    (2, 40000, 5, "avg", 39000),
    (1, 40960, 1, "max", 40960),    # everything is kept
    (49, 40960, 7, "max", 32767),   # enough rows for the one-CTA kernel: the same two points there
    (49, 40960, 7, "max", 32768),
    (49, 40000, 5, "avg", 39000),
    (2, 49000, 17, "max", 48000),   # radius 8: generic one-CTA kernel
    (1, 70000, 5, "avg", 69000),    # many-CTA path
])
def test_pool_topk_with_very_large_ksel_stays_inside_its_rows(rows, n, kernel, ptype, ksel):
    g = torch.Generator().manual_seed(n + ksel)
    vote = torch.rand(rows, n, generator=g, dtype=torch.float32) ** 4
    # the index rows sit inside a poisoned buffer: anything written before or behind them shows
    guard = 4096
    POISON = -0x5A5A5A5B
    buf = torch.full((guard + rows * ksel + guard,), POISON, dtype=torch.int32, device="cuda")
    out = buf[guard:guard + rows * ksel].view(rows, ksel)
    sk.snapkv_pool_topk(vote.cuda(), kernel, PT[ptype], ksel, out_idx=out)
    torch.cuda.synchronize()
    assert bool((buf[:guard] == POISON).all()) and bool((buf[guard + rows * ksel:] == POISON).all())
    idx = out.cpu().numpy()
    for r in range(rows):
        pooled = orc.pool1d(vote[r].numpy().astype(np.float64), kernel, PT[ptype])
        ref = orc.topk_positions(pooled, ksel)
        same = parity.check_indices(idx[r], pooled, ksel, ref)
        if ptype == "max":
            assert same


def test_compress_that_keeps_all_but_one_row_of_a_long_prompt():
    # budget = L - 1 at L = 40000: ksel = 39967 goes through the one-CTA select kernel
    B, Hq, Hkv, L, d, W, budget = 1, 2, 1, 40000, 128, 32, 39999
    w = synth.Workload(52, "t", B, Hq, Hkv, d, L, W, 5, "avg", (budget,), 1, 4)
    data = synth.make_layer(w, 3)
    _check_compress(data, W, 5, "avg", budget)


@pytest.mark.parametrize("n,ksel", [(3000, 700), (5000, 700), (40000, 9000), (100000, 30000), (200000, 1234)])
def test_pool_topk_exact_ties_take_lower_positions(n, ksel):
    vote = torch.zeros(3, n)
    vote[0, :] = 0.25                         # all equal: the first ksel positions win
    vote[1, 100::10] = 1.0                    # plateaus of width 7 around every tenth position
    vote[2, :] = 0.0                          # all zero: again the first ksel positions
    idx = sk.snapkv_pool_topk(vote.cuda(), 7, sk.POOL_MAX, ksel).cpu().numpy()
    assert np.array_equal(idx[0], np.arange(ksel))
    assert np.array_equal(idx[2], np.arange(ksel))
    pooled = orc.pool1d(vote[1].numpy().astype(np.float64), 7, orc.POOL_MAX)
    assert np.array_equal(idx[1], orc.topk_positions(pooled, ksel))


@pytest.mark.parametrize("rows,n,kernel,ptype,ksel", [
    (128, 32736, 5, "avg", 4064),    # the one-CTA kernel, the benchmarked shape
    (8, 16352, 7, "max", 992),       # the cluster kernel
    (2, 200000, 7, "max", 2048),     # the many-launch path
])
def test_pool_topk_leaves_the_callers_votes_alone(rows, n, kernel, ptype, ksel):
    # the whole-step calls let the select kernel drop their scratch votes from L2 once read;
    # votes that the caller hands to the staged call are the caller's and must come back intact,
    # also after a second call on the same tensor
    g = torch.Generator().manual_seed(11)
    vote = (torch.rand(rows, n, generator=g) ** 4).cuda()
    before = vote.clone()
    first = sk.snapkv_pool_topk(vote, kernel, PT[ptype], ksel)
    torch.cuda.synchronize()
    assert torch.equal(vote, before)
    again = sk.snapkv_pool_topk(vote, kernel, PT[ptype], ksel)
    assert torch.equal(first, again)
    assert torch.equal(vote, before)


# ------------------------------------------------------------------ gather
@pytest.mark.parametrize("B,Hq,Hkv,L,d,W,ksel", [
    (1, 4, 4, 1024, 64, 32, 224),
    (2, 8, 2, 777, 128, 16, 301),
    (1, 2, 1, 130, 128, 64, 1),
    (1, 3, 3, 50, 64, 7, 43),
])
def test_gather_is_bit_exact(B, Hq, Hkv, L, d, W, ksel):
    data = synth.make_random(B, Hq, Hkv, L, d, W, seed=5)
    n = L - W
    g = torch.Generator().manual_seed(1)
    idx = torch.stack([torch.stack([torch.sort(torch.randperm(n, generator=g)[:ksel]).values
                                    for _ in range(Hq)]) for _ in range(B)]).to(torch.int32)
    ok, ov = sk.snapkv_gather(data["k"].cuda(), data["v"].cuda(), idx.cuda(), W)
    okb, ovb, kb, vb = _bits(ok), _bits(ov), _bits(data["k"]), _bits(data["v"])
    for b in range(B):
        for h in range(Hq):
            c = h // (Hq // Hkv)
            parity.check_rows(okb[b, h], ovb[b, h], kb[b, c], vb[b, c], idx[b, h].numpy().astype(np.int64), W)


# ------------------------------------------------------------------ whole step
def _check_compress(data, w_W, kernel, ptype, budget, heads=None, dev=None):
    dev = dev or _to_dev(data)
    out_k, out_v, out_idx, ws = sk.snapkv_compress(dev["q_obs"], dev["k"], dev["v"], kernel, PT[ptype], budget)
    code, detail = sk.snapkv_device_status(ws)
    assert code == sk.OK, (code, detail)
    B, Hq = dev["q_obs"].shape[:2]
    Hkv = dev["k"].shape[1]
    g = Hq // Hkv
    L = dev["k"].shape[2]
    ksel = budget - w_W
    assert out_k.shape == (B, Hq, budget, dev["k"].shape[3]) and out_idx.shape == (B, Hq, ksel)
    heads = heads or [(b, h) for b in range(B) for h in range(Hq)]
    idx_all = out_idx.cpu().numpy()
    exact = 0
    for (b, h) in heads:
        c = h // g
        qb = _bits(dev["q_obs"][b, h])
        kb = _bits(dev["k"][b, c])
        vb = _bits(dev["v"][b, c])
        vt = orc.window_votes(orc.bf16_bits_to_f64(qb), orc.bf16_bits_to_f64(kb))
        pooled = orc.pool1d(vt, kernel, PT[ptype])
        ref = orc.topk_positions(pooled, ksel)
        exact += parity.check_indices(idx_all[b, h], pooled, ksel, ref)
        parity.check_rows(_bits(out_k[b, h]), _bits(out_v[b, h]), kb, vb, idx_all[b, h].astype(np.int64), w_W)
    return exact, len(heads), (out_k, out_v, out_idx)


def test_compress_tiny_workload_matches_golden_and_oracle():
    from test_oracle_golden import load_golden
    w = synth.WORKLOADS[0]
    data = synth.make_layer(w, 0)                      # CPU-drawn: the golden file's inputs
    exact, total, (ok, ov, oi) = _check_compress(data, w.W, w.pool_kernel, w.pool_type, w.budgets[0])
    starts, idx_golden, _ = load_golden()
    got = oi.cpu().numpy()
    for h in range(w.Hq):
        kept = set(got[0, h].tolist())
        for s in starts:
            assert set(range(s, s + synth.CLUSTER_LEN)) <= kept
    assert exact >= total - 1  # sets equal to the golden ones unless a near-tie straddles the cut
    if exact == total:
        for h in range(w.Hq):
            assert np.array_equal(got[0, h], idx_golden[h])


@pytest.mark.parametrize("B,Hq,Hkv,L,d,W,kernel,ptype,budget", [
    (2, 4, 2, 1000, 128, 32, 5, "avg", 200),
    (1, 8, 1, 2100, 64, 32, 7, "max", 512),
    (1, 4, 4, 3000, 128, 16, 5, "max", 116),
    (1, 4, 2, 1500, 128, 64, 13, "max", 300),
    (1, 2, 2, 333, 64, 5, 1, "max", 40),
    (1, 2, 2, 1000, 128, 32, 7, "max", 999),      # keeps all but one prefix row
    (1, 2, 2, 1000, 128, 32, 7, "max", 33),       # keeps a single prefix row
])
def test_compress_small_shapes(B, Hq, Hkv, L, d, W, kernel, ptype, budget):
    w = synth.Workload(50, "t", B, Hq, Hkv, d, L, W, kernel, ptype, (budget,), 1, 2)
    data = synth.make_layer(w, L)
    _check_compress(data, W, kernel, ptype, budget)


@pytest.mark.parametrize("budget", [1000, 1001, 4096])
def test_budget_at_least_L_copies_the_cache(budget):
    B, Hq, Hkv, L, d, W = 2, 4, 2, 1000, 128, 32
    data = synth.make_random(B, Hq, Hkv, L, d, W, seed=11)
    dev = _to_dev(data)
    ok, ov, oi, _ = sk.snapkv_compress(dev["q_obs"], dev["k"], dev["v"], 7, sk.POOL_MAX, budget)
    assert ok.shape == (B, Hq, L, d) and oi.shape == (B, Hq, L - W)
    assert torch.equal(ok, dev["k"].repeat_interleave(2, dim=1))
    assert torch.equal(ov, dev["v"].repeat_interleave(2, dim=1))
    assert torch.equal(oi, torch.arange(L - W, dtype=torch.int32, device="cuda").expand(B, Hq, -1))


def test_identity_with_budget_rows_leaves_the_tail_untouched():
    # raw ABI: budget > L addresses outputs with `budget` rows per head, rows >= L untouched
    B, Hq, Hkv, L, d, W, budget = 1, 2, 2, 100, 64, 8, 128
    data = synth.make_random(B, Hq, Hkv, L, d, W, seed=12)
    dev = _to_dev(data)
    ok = torch.full((B, Hq, budget, d), 7.0, dtype=torch.bfloat16, device="cuda")
    ov = torch.full_like(ok, 7.0)
    oi = torch.full((B, Hq, budget - W), -5, dtype=torch.int32, device="cuda")
    code = sk.lib().snapkv_compress(dev["q_obs"].data_ptr(), dev["k"].data_ptr(), dev["v"].data_ptr(),
                                    B, Hq, Hkv, L, d, W, 7, 0, budget, ok.data_ptr(), ov.data_ptr(),
                                    oi.data_ptr(), None, 0, None)
    assert code == sk.OK
    torch.cuda.synchronize()
    assert torch.equal(ok[:, :, :L], dev["k"]) and torch.all(ok[:, :, L:] == 7.0)
    assert torch.equal(oi[:, :, : L - W], torch.arange(L - W, dtype=torch.int32, device="cuda").expand(B, Hq, -1))
    assert torch.all(oi[:, :, L - W:] == -5)


def test_gqa_equals_mha_on_repeated_kv():
    B, Hq, Hkv, L, d, W = 1, 8, 2, 1200, 128, 32
    data = synth.make_layer(synth.Workload(51, "t", B, Hq, Hkv, d, L, W, 7, "max", (256,), 1, 3), 0)
    dev = _to_dev(data)
    a = sk.snapkv_compress(dev["q_obs"], dev["k"], dev["v"], 7, sk.POOL_MAX, 256)
    krep = dev["k"].repeat_interleave(4, dim=1).contiguous()
    vrep = dev["v"].repeat_interleave(4, dim=1).contiguous()
    b = sk.snapkv_compress(dev["q_obs"], krep, vrep, 7, sk.POOL_MAX, 256)
    # same keys, same queries: the logits are bit-identical whichever way the heads are
    # grouped into MMA tiles, so the outputs are too
    assert torch.equal(a[2], b[2]) and torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])


def test_runs_are_bit_identical():
    w = synth.WORKLOADS[0]
    dev = _to_dev(synth.make_layer(w, 0))
    first = sk.snapkv_compress(dev["q_obs"], dev["k"], dev["v"], 7, sk.POOL_MAX, 256)
    for _ in range(5):
        again = sk.snapkv_compress(dev["q_obs"], dev["k"], dev["v"], 7, sk.POOL_MAX, 256)
        assert all(torch.equal(first[i], again[i]) for i in range(3))


def test_compress_from_host_buffers():
    w = synth.WORKLOADS[0]
    data = synth.make_layer(w, 0)
    budget = w.budgets[0]
    q, k, v = (data[x].pin_memory() for x in ("q_obs", "k", "v"))
    ok = torch.empty(w.B, w.Hq, budget, w.d, dtype=torch.bfloat16).pin_memory()
    ov = torch.empty_like(ok).pin_memory()
    oi = torch.empty(w.B, w.Hq, budget - w.W, dtype=torch.int32).pin_memory()
    need = sk.snapkv_host_staging_size(w.B, w.Hq, w.Hkv, w.L, w.d, w.W, 7, 0, budget)
    staging = torch.empty(need, dtype=torch.uint8, device="cuda")
    sk.snapkv_compress_host(q, k, v, 7, sk.POOL_MAX, budget, ok, ov, oi, staging)
    torch.cuda.synchronize()
    dev = _to_dev(data)
    ref = sk.snapkv_compress(dev["q_obs"], dev["k"], dev["v"], 7, sk.POOL_MAX, budget)
    assert torch.equal(ok, ref[0].cpu()) and torch.equal(ov, ref[1].cpu()) and torch.equal(oi, ref[2].cpu())


@pytest.mark.parametrize("B,Hq,Hkv,L,d,W,kernel,budget", [
    (3, 8, 2, 700, 128, 16, 5, 128),     # 6 (batch, KV head) pairs, one per part
    (1, 22, 11, 900, 64, 32, 7, 300),    # 11 pairs: five parts of two and one of one
    (2, 4, 4, 300, 128, 32, 7, 300),     # budget >= L: identity, expanded to Hq heads
    (1, 2, 1, 4000, 128, 64, 13, 1000),  # one pair: a single part
])
def test_compress_from_host_buffers_in_parts(B, Hq, Hkv, L, d, W, kernel, budget):
    data = synth.make_random(B, Hq, Hkv, L, d, W, seed=21)
    rows = min(budget, L)
    q, k, v = (data[x].pin_memory() for x in ("q_obs", "k", "v"))
    dev = _to_dev(data)
    ref = sk.snapkv_compress(dev["q_obs"], dev["k"], dev["v"], kernel, sk.POOL_MAX, budget)
    need = sk.snapkv_host_staging_size(B, Hq, Hkv, L, d, W, kernel, 0, rows)
    staging = torch.empty(need, dtype=torch.uint8, device="cuda")
    for _ in range(2):  # the second call reuses the library's side stream and events
        ok = torch.zeros(B, Hq, rows, d, dtype=torch.bfloat16).pin_memory()
        ov = torch.zeros_like(ok).pin_memory()
        oi = torch.zeros(B, Hq, rows - W, dtype=torch.int32).pin_memory()
        sk.snapkv_compress_host(q, k, v, kernel, sk.POOL_MAX, budget, ok, ov, oi, staging)
        torch.cuda.current_stream().synchronize()  # the caller's stream alone covers the copies back
        assert torch.equal(ok, ref[0].cpu()) and torch.equal(ov, ref[1].cpu())
        assert torch.equal(oi, ref[2].cpu())


# ------------------------------------------------------------------ full-size workloads, sampled heads
def _sample_heads(B, Hq, count, seed):
    g = torch.Generator().manual_seed(seed)
    flat = torch.randperm(B * Hq, generator=g)[:count].tolist()
    return [(f // Hq, f % Hq) for f in flat]


@pytest.mark.parametrize("wid,layer,budget,nheads", [
    (1, 0, 1024, 4), (1, 31, 4096, 3),
    (2, 0, 4096, 6), (2, 15, 4096, 3),
    (3, 0, 2048, 2), (3, 1, 8192, 2),
])
def test_full_size_workloads_on_sampled_heads(wid, layer, budget, nheads):
    w = synth.WORKLOADS[wid]
    dev = synth.make_layer(w, layer, device="cuda")
    heads = _sample_heads(w.B, w.Hq, nheads, wid * 100 + layer)
    _check_compress(None, w.W, w.pool_kernel, w.pool_type, budget, heads=heads, dev=dev)


@pytest.mark.parametrize("wid,layer,heads", [
    # workload 2 (the benchmarked shape): heads in different batches, i.e. in different waves
    # of the scoring schedule, and all four heads of one KV group once
    (2, 0, [(0, 0), (0, 31), (1, 9), (2, 18), (3, 4), (3, 5), (3, 6), (3, 7)]),
    (2, 17, [(0, 12), (1, 30), (2, 1), (3, 23)]),
    # workload 3: W = 64, two head sub-groups per KV head (column-split epilogue)
    (3, 0, [(0, 0), (0, 2), (0, 15), (0, 29)]),
])
def test_full_size_votes_of_the_recomputing_path(wid, layer, heads):
    """Eq. 1 element by element at full size: every vote of the sampled heads, from the
    two-sweep scoring call in the configuration the benchmark times."""
    w = synth.WORKLOADS[wid]
    dev = synth.make_layer(w, layer, device="cuda", want_v=False)
    vote, ws = sk.snapkv_window_scores(dev["q_obs"], dev["k"])
    code, detail = sk.snapkv_device_status(ws)
    assert code == sk.OK, (code, detail)
    qb, kb = _bits(dev["q_obs"]), _bits(dev["k"])
    worst = 0.0
    for b, h in heads:
        ref = _oracle_head(qb, kb, b, h, w.Hq // w.Hkv)
        worst = max(worst, parity.check_votes(vote[b, h].cpu().numpy(), ref))
    assert worst < 1e-4  # fp32 accumulation and exp2.approx leave about 1e-6


def test_fused_call_leaves_the_same_votes_as_the_staged_call():
    # the whole-step entry point scores into its workspace; what it selects from must be the
    # votes the staged scoring call returns, bit for bit (same kernel, same schedule)
    w = synth.WORKLOADS[2]
    dev = synth.make_layer(w, 5, device="cuda")
    budget = w.budgets[-1]
    ok, ov, oi, ws = sk.snapkv_compress(dev["q_obs"], dev["k"], dev["v"], w.pool_kernel, PT[w.pool_type], budget)
    staged, _ = sk.snapkv_window_scores(dev["q_obs"], dev["k"])
    idx = sk.snapkv_pool_topk(staged.view(w.B * w.Hq, w.n), w.pool_kernel, PT[w.pool_type], budget - w.W)
    assert torch.equal(idx.view_as(oi), oi)


def test_extreme_prompt_keeps_the_needle():
    w = synth.WORKLOADS[4]
    dev = synth.make_layer(w, 0, device="cuda")
    budget = w.budgets[0]
    heads = _sample_heads(w.B, w.Hq, 2, 4)
    _, _, (ok, ov, oi) = _check_compress(None, w.W, w.pool_kernel, w.pool_type, budget, heads=heads, dev=dev)
    s = int(dev["starts"][0][0])
    needle = torch.arange(s, s + synth.CLUSTER_LEN, device="cuda", dtype=torch.int32)
    hits = (oi[0][:, :, None] == needle[None, None, :]).any(dim=1).sum(dim=1)  # per head
    # every head keeps part of the needle (the oracle does too, by parity on the sampled heads)
    assert int((hits > 0).sum()) == w.Hq
    # votes of one head over the whole 380K prompt
    vote, _ = sk.snapkv_window_scores(dev["q_obs"][:, :2].contiguous(), dev["k"][:, :2].contiguous())
    ref = _oracle_head(_bits(dev["q_obs"][:, :2]), _bits(dev["k"][:, :2]), 0, 1, 1)
    parity.check_votes(vote[0, 1].cpu().numpy(), ref)
