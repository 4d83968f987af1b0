"""GPU parity for snapkv_decode_attention (one generation step over the compressed cache):
element by element against the oracle, |error| <= 1e-3 * sum_j p_j |v_j| (the magnitude of the
terms that are summed; fp32 accumulation of bf16 products sits two to three orders inside)."""
import numpy as np
import pytest
import torch

from oracle import snapkv_oracle as orc
from paper_2404_14469_b200 import binding as sk
from paper_2404_14469_b200 import synth

pytestmark = pytest.mark.gpu

EPS = 1e-3


def _check(q, ck, cv):
    out, lse, _ = sk.snapkv_decode_attention(q.cuda(), ck.cuda(), cv.cuda())
    ref, ref_lse, scale = orc.decode_attention(synth.bf16_bits(q), synth.bf16_bits(ck), synth.bf16_bits(cv))
    err = np.abs(out.cpu().numpy().astype(np.float64) - ref)
    assert np.all(err <= EPS * scale + 1e-30), float((err / np.maximum(scale, 1e-300)).max())
    assert np.allclose(lse.cpu().numpy(), ref_lse, rtol=0, atol=EPS)
    return float((err / np.maximum(scale, 1e-300)).max())


@pytest.mark.parametrize("B,Hq,Hc,rows,d,q_scale", [
    (1, 4, 4, 256, 64, 1.0),        # tiny workload's cache
    (2, 8, 2, 1000, 128, 2.0),      # cache kept at Hkv heads, ragged split
    (1, 2, 2, 1, 128, 1.0),         # a single row: the output is that row's value
    (3, 2, 1, 63, 64, 4.0),         # fewer rows than one split
    (1, 32, 32, 4096, 128, 3.0),    # MHA workload's budget
    (1, 1, 1, 70000, 128, 1.0),     # one head, many splits
])
def test_decode_matches_oracle(B, Hq, Hc, rows, d, q_scale):
    g = torch.Generator().manual_seed(rows + Hq)
    q = (q_scale * torch.randn(B, Hq, d, generator=g)).to(torch.bfloat16)
    ck = torch.randn(B, Hc, rows, d, generator=g).to(torch.bfloat16)
    cv = torch.randn(B, Hc, rows, d, generator=g).to(torch.bfloat16)
    _check(q, ck, cv)


def test_large_logits_and_a_dominant_row():
    g = torch.Generator().manual_seed(5)
    q = (8.0 * torch.randn(1, 4, 128, generator=g)).to(torch.bfloat16)
    ck = torch.randn(1, 4, 777, 128, generator=g).to(torch.bfloat16)
    cv = torch.randn(1, 4, 777, 128, generator=g).to(torch.bfloat16)
    ck[0, :, 500] = q[0] * 4.0          # logits in the hundreds for one row
    out, _, _ = sk.snapkv_decode_attention(q.cuda(), ck.cuda(), cv.cuda())
    _check(q, ck, cv)
    assert torch.allclose(out[0].cpu(), cv[0, :, 500].float(), atol=1e-6)


def test_decode_over_the_steps_own_output_and_runs_are_bit_identical():
    w = synth.WORKLOADS[0]
    data = synth.make_layer(w, 0)
    q, k, v = (data[x].cuda() for x in ("q_obs", "k", "v"))
    ok, ov, _, _ = sk.snapkv_compress(q, k, v, w.pool_kernel, sk.POOL_MAX, w.budgets[0])
    q_cur = q[:, :, -1].contiguous()
    _check(q_cur.cpu(), ok.cpu(), ov.cpu())
    a = sk.snapkv_decode_attention(q_cur, ok, ov)
    b = sk.snapkv_decode_attention(q_cur, ok, ov)
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])
