"""The time-out path of the scoring kernel, exercised on the GPU in the only safe form: a
wait on a flag that nothing ever sets, with a short limit.  Every wait in the kernel is
bounded; when one runs out the block records the wait's code, lets its copies and
tensor-core operations finish, frees its tensor memory and returns, and the host reads
SNAPKV_ERR_TIMEOUT from the workspace.  Nothing here faults or hangs the device."""
import time

import pytest
import torch

from oracle import snapkv_oracle as orc
from paper_2404_14469_b200 import binding as sk
from paper_2404_14469_b200 import synth

import parity

pytestmark = pytest.mark.gpu

TIMEOUT, WAIT_UNIT_STATS = 5, 7


@pytest.mark.parametrize("B,Hq,Hkv,L,d,W", [
    (1, 4, 2, 3000, 128, 32),       # a few blocks have work
    (2, 32, 8, 16384, 128, 32),     # every block of the grid has work and runs into the limit
])
def test_a_wait_that_nothing_satisfies_runs_out_and_the_context_survives(B, Hq, Hkv, L, d, W):
    data = synth.make_random(B, Hq, Hkv, L, d, W, seed=77)
    q, k = data["q_obs"].cuda(), data["k"].cuda()
    vote = torch.full((B, Hq, L - W), -1.0, dtype=torch.float32, device="cuda")
    prev = sk.snapkv_set_wait_limit_ns(20_000_000)          # 20 ms; waits on other blocks: 10 ms
    try:
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        _, ws = sk.snapkv_selftest_stalled_scores(q, k, vote)
        code, detail = sk.snapkv_device_status(ws)           # synchronises the stream
        took = time.perf_counter() - t0
    finally:
        sk.snapkv_set_wait_limit_ns(prev)
    assert (code, detail) == (TIMEOUT, WAIT_UNIT_STATS)
    assert sk.status_string(code) == "SNAPKV_ERR_TIMEOUT"
    assert 0.005 < took < 2.0                                # it did wait, and it did return
    assert bool((vote == -1.0).all())                        # no vote was written
    # the context is intact: the ordinary call on the same buffers is correct and clean
    vote2, ws2 = sk.snapkv_window_scores(q, k, vote, ws)
    assert sk.snapkv_device_status(ws2) == (sk.OK, 0)
    heads = [(0, 0), (B - 1, Hq - 1)]
    qb, kb = synth.bf16_bits(data["q_obs"]), synth.bf16_bits(data["k"])
    g = Hq // Hkv
    for b, h in heads:
        ref = orc.window_votes(orc.bf16_bits_to_f64(qb[b, h]), orc.bf16_bits_to_f64(kb[b, h // g]))
        parity.check_votes(vote2[b, h].cpu().numpy(), ref)
