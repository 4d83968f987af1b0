"""The stored oracle output of the tiny workload still is what the oracle computes
(guards the oracle and the seeded CPU input generator against silent drift)."""
import os

import numpy as np

from oracle import snapkv_oracle as orc
from paper_2404_14469_b200 import synth

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "workload0_oracle.txt")


def load_golden():
    idx, votes, starts = {}, {}, None
    with open(GOLDEN) as f:
        for line in f:
            t = line.split()
            if t[0] == "#" and len(t) > 1 and t[1] == "starts":
                starts = [int(x) for x in t[2:]]
            elif t[0] == "idx":
                idx[int(t[1])] = np.array([int(x) for x in t[2:]], dtype=np.int64)
            elif t[0] == "vote":
                votes[(int(t[1]), int(t[2]))] = float.fromhex(t[3])
    return starts, idx, votes


def test_golden_matches_oracle():
    w = synth.WORKLOADS[0]
    data = synth.make_layer(w, 0)
    q, k, v = (synth.bf16_bits(data[x]) for x in ("q_obs", "k", "v"))
    res = orc.compress(q, k, v, w.pool_kernel, orc.POOL_MAX, w.budgets[0])
    starts, idx, votes = load_golden()
    assert starts == [int(s) for s in data["starts"][0]]
    assert len(idx) == w.Hq
    for h in range(w.Hq):
        assert np.array_equal(idx[h], res["out_idx"][0, h])
    for (h, j), val in votes.items():
        assert abs(res["vote"][0, h, j] - val) <= 1e-12 * abs(val)
