"""Pins for the oracle's decode attention over the compressed cache: the framework's attention
routine, closed forms, invariance to the order of cache rows, agreement between attending to
the compressed cache and attending to the selected rows of the full cache, planted mistakes.
CPU only."""
import math

import numpy as np
import pytest
import torch

from oracle import snapkv_oracle as orc
from paper_2404_14469_b200 import synth


def _case(B=2, Hq=4, Hc=2, R=37, d=16, seed=0, q_scale=2.0):
    g = torch.Generator().manual_seed(seed)
    q = (q_scale * torch.randn(B, Hq, d, generator=g)).to(torch.bfloat16)
    k = torch.randn(B, Hc, R, d, generator=g).to(torch.bfloat16)
    v = torch.randn(B, Hc, R, d, generator=g).to(torch.bfloat16)
    return q, k, v


def _run(q, k, v):
    return orc.decode_attention(synth.bf16_bits(q), synth.bf16_bits(k), synth.bf16_bits(v))


def test_matches_the_frameworks_attention_routine():
    q, k, v = _case()
    out, lse, _ = _run(q, k, v)
    g = q.shape[1] // k.shape[1]
    kk = k.double().repeat_interleave(g, dim=1)
    vv = v.double().repeat_interleave(g, dim=1)
    ref = torch.nn.functional.scaled_dot_product_attention(q.double()[:, :, None, :], kk, vv)[:, :, 0]
    assert np.allclose(out, ref.numpy(), rtol=1e-12, atol=1e-14)
    ref_lse = torch.logsumexp(torch.einsum("bhd,bhjd->bhj", q.double(), kk) / math.sqrt(q.shape[2]), dim=-1)
    assert np.allclose(lse, ref_lse.numpy(), rtol=1e-12, atol=0)


def test_zero_query_averages_the_values_and_a_dominant_key_returns_its_value():
    q, k, v = _case(B=1, Hq=2, Hc=2, R=9, seed=1)
    out, lse, scale = _run(torch.zeros_like(q), k, v)
    assert np.allclose(out, v.double().mean(dim=2).numpy(), rtol=1e-13, atol=1e-15)
    assert np.allclose(lse, math.log(9), rtol=1e-13)
    assert np.allclose(scale, v.double().abs().mean(dim=2).numpy(), rtol=1e-13, atol=1e-15)
    k2 = torch.zeros_like(k)
    k2[:, :, 4] = 64.0 * q[0, :, :].sign()[None]          # logit of row 4 dwarfs the others
    out, _, _ = _run(q, k2, v)
    assert np.allclose(out, v.double()[:, :, 4].numpy(), rtol=0, atol=1e-12)


def test_order_of_cache_rows_does_not_matter():
    q, k, v = _case(seed=2)
    perm = torch.randperm(k.shape[2], generator=torch.Generator().manual_seed(3))
    a = _run(q, k, v)
    b = _run(q, k[:, :, perm], v[:, :, perm])
    for x, y in zip(a, b):
        assert np.allclose(x, y, rtol=1e-12, atol=1e-14)


def test_attending_to_the_compressed_cache_is_attending_to_the_selected_rows():
    data = synth.make_random(1, 4, 2, 120, 16, 8, seed=4, q_scale=2.0)
    qb, kb, vb = (synth.bf16_bits(data[x]) for x in ("q_obs", "k", "v"))
    comp = orc.compress(qb, kb, vb, 5, orc.POOL_MAX, 40)
    q_cur = qb[:, :, -1]                                   # any query will do
    out, lse, _ = orc.decode_attention(q_cur, comp["out_k"], comp["out_v"])
    for h in range(4):
        rows = np.concatenate([comp["out_idx"][0, h], np.arange(112, 120)])
        kf = orc.bf16_bits_to_f64(kb[0, h // 2][rows])
        vf = orc.bf16_bits_to_f64(vb[0, h // 2][rows])
        p = torch.softmax(torch.from_numpy(kf @ orc.bf16_bits_to_f64(q_cur[0, h]) / 4.0), dim=0).numpy()
        assert np.allclose(out[0, h], p @ vf, rtol=1e-12, atol=1e-14)


def test_planted_mistakes_are_caught(monkeypatch):
    real = orc.decode_attention

    def swapped(q, k, v):           # keys and values exchanged
        return real(q, v, k)

    def wrong_head_map(q, k, v):    # h % Hc instead of h // g
        Hq, Hc = q.shape[1], k.shape[1]
        perm = [c + j * Hc for c in range(Hc) for j in range(Hq // Hc)]
        out, lse, scale = real(q[:, perm], k, v)
        return out, lse, scale

    for wrong in (swapped, wrong_head_map):
        monkeypatch.setattr(orc, "decode_attention", wrong)
        with pytest.raises(AssertionError):
            test_matches_the_frameworks_attention_routine()
        monkeypatch.setattr(orc, "decode_attention", real)
