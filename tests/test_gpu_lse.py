"""GPU parity of the supplied-normaliser variant (snapkv_window_scores_lse,
snapkv_compress_lse) against the oracle's votes_given_lse / compress(lse=...)."""
import numpy as np
import pytest
import torch

from oracle import snapkv_oracle as orc
from paper_2404_14469_b200 import binding as sk
from paper_2404_14469_b200 import synth

import parity
from test_gpu_parity import SCORE_SHAPES, _bits, _to_dev

pytestmark = pytest.mark.gpu


def _oracle_votes_lse(q_bits, k_bits, lse):
    B, Hq = q_bits.shape[:2]
    g = Hq // k_bits.shape[1]
    out = []
    for b in range(B):
        for h in range(Hq):
            s = orc.window_logits(orc.bf16_bits_to_f64(q_bits[b, h]), orc.bf16_bits_to_f64(k_bits[b, h // g]))
            out.append(orc.votes_given_lse(s, lse[b, h]))
    return np.stack(out).reshape(B, Hq, -1)


@pytest.mark.parametrize("B,Hq,Hkv,L,d,W", SCORE_SHAPES)
def test_votes_with_supplied_lse_match_oracle(B, Hq, Hkv, L, d, W):
    data = synth.make_random(B, Hq, Hkv, L, d, W, seed=L + 2 * W, q_scale=1.5)
    qb, kb = _bits(data["q_obs"]), _bits(data["k"])
    lse = orc.lse_obs(qb, kb)
    lse32 = torch.from_numpy(lse.astype(np.float32)).cuda()
    dev = _to_dev(data)
    vote, ws = sk.snapkv_window_scores_lse(dev["q_obs"], dev["k"], lse32)
    code, detail = sk.snapkv_device_status(ws)
    assert code == sk.OK, (code, detail)
    # the oracle takes the very fp32 values the GPU was given
    ref = _oracle_votes_lse(qb, kb, lse32.cpu().numpy().astype(np.float64))
    parity.check_votes(vote.cpu().numpy(), ref)
    # and with the rows' true log-sum-exp that is the two-sweep result
    two, _ = sk.snapkv_window_scores(dev["q_obs"], dev["k"])
    assert torch.allclose(vote, two, rtol=2e-4, atol=1e-30)


def test_a_shifted_lse_row_scales_that_row_on_the_gpu():
    B, Hq, Hkv, L, d, W = 1, 2, 1, 700, 128, 32
    data = synth.make_random(B, Hq, Hkv, L, d, W, seed=8)
    qb, kb = _bits(data["q_obs"]), _bits(data["k"])
    lse = orc.lse_obs(qb, kb)
    lse[0, 1, 5] += np.log(4.0)
    lse32 = torch.from_numpy(lse.astype(np.float32)).cuda()
    dev = _to_dev(data)
    vote, _ = sk.snapkv_window_scores_lse(dev["q_obs"], dev["k"], lse32)
    ref = _oracle_votes_lse(qb, kb, lse32.cpu().numpy().astype(np.float64))
    parity.check_votes(vote.cpu().numpy(), ref)


@pytest.mark.parametrize("B,Hq,Hkv,L,d,W,kernel,ptype,budget", [
    (1, 4, 4, 1024, 64, 32, 7, "max", 256),
    (2, 8, 2, 1500, 128, 32, 5, "avg", 300),
    (1, 4, 1, 2100, 128, 64, 13, "max", 512),
    (2, 3, 3, 400, 64, 16, 5, "max", 400),      # budget >= L: identity, lse unused
])
def test_compress_with_supplied_lse_matches_oracle(B, Hq, Hkv, L, d, W, kernel, ptype, budget):
    data = synth.make_random(B, Hq, Hkv, L, d, W, seed=31)
    qb, kb, vb = _bits(data["q_obs"]), _bits(data["k"]), _bits(data["v"])
    lse32 = torch.from_numpy(orc.lse_obs(qb, kb).astype(np.float32)).cuda()
    dev = _to_dev(data)
    pt = sk.POOL_MAX if ptype == "max" else sk.POOL_AVG
    ok, ov, oi, ws = sk.snapkv_compress_lse(dev["q_obs"], dev["k"], dev["v"], lse32, kernel, pt, budget)
    torch.cuda.synchronize()
    ref = orc.compress(qb, kb, vb, kernel, pt, budget, lse=lse32.cpu().numpy().astype(np.float64))
    g = Hq // Hkv
    rows = min(budget, L)
    okb, ovb, idx = _bits(ok), _bits(ov), oi.cpu().numpy()
    for b in range(B):
        for h in range(Hq):
            if budget < L:
                parity.check_indices(idx[b, h], ref["pooled"][b, h], rows - W, ref["out_idx"][b, h])
            else:
                assert np.array_equal(idx[b, h], ref["out_idx"][b, h])
            parity.check_rows(okb[b, h], ovb[b, h], kb[b, h // g], vb[b, h // g], idx[b, h].astype(np.int64), W)


def test_full_size_workload_2_with_supplied_lse_on_sampled_heads():
    w = synth.WORKLOADS[2]
    dev = synth.make_layer(w, 3, device="cuda")
    qb, kb = _bits(dev["q_obs"]), _bits(dev["k"])
    heads = [(0, 1), (1, 13), (3, 31), (2, 20)]
    g = w.Hq // w.Hkv
    lse = np.zeros((w.B, w.Hq, w.W))
    # the kernel needs every row's normaliser: the oracle computes all of them (fp64)
    for b in range(w.B):
        for c in range(w.Hkv):
            kf = orc.bf16_bits_to_f64(kb[b, c])
            for h in range(c * g, (c + 1) * g):
                lse[b, h] = orc.window_lse(orc.window_logits(orc.bf16_bits_to_f64(qb[b, h]), kf))
    lse32 = torch.from_numpy(lse.astype(np.float32)).cuda()
    vote, ws = sk.snapkv_window_scores_lse(dev["q_obs"], dev["k"], lse32)
    code, detail = sk.snapkv_device_status(ws)
    assert code == sk.OK, (code, detail)
    got = vote.cpu().numpy()
    lse_used = lse32.cpu().numpy().astype(np.float64)
    for b, h in heads:
        s = orc.window_logits(orc.bf16_bits_to_f64(qb[b, h]), orc.bf16_bits_to_f64(kb[b, h // g]))
        parity.check_votes(got[b, h], orc.votes_given_lse(s, lse_used[b, h]))
