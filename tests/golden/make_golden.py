"""Writes tests/golden/workload0_oracle.txt from the CPU oracle alone.

Run from the repository root:  python tests/golden/make_golden.py
The file stores, for the tiny workload (B=1, Hq=Hkv=4, d=64, L=1024, W=32, max pool 7,
budget 256; inputs drawn by the seeded CPU generator), the selected positions per head
and a few votes.  No value in it comes from the CUDA path.  There is no worked numeric
example of the compression step in the paper (Sec. 4, Listing 1) to store instead.
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import snapkv_oracle as orc          # noqa: E402
from paper_2404_14469_b200 import synth           # noqa: E402


def main():
    w = synth.WORKLOADS[0]
    data = synth.make_layer(w, 0)
    q, k, v = (synth.bf16_bits(data[x]) for x in ("q_obs", "k", "v"))
    res = orc.compress(q, k, v, w.pool_kernel, orc.POOL_MAX, w.budgets[0])
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "workload0_oracle.txt")
    with open(path, "w") as f:
        f.write("# written by tests/golden/make_golden.py from oracle/snapkv_oracle.py only\n")
        f.write("# starts " + " ".join(str(int(s)) for s in data["starts"][0]) + "\n")
        for h in range(w.Hq):
            f.write(f"idx {h} " + " ".join(str(int(j)) for j in res["out_idx"][0, h]) + "\n")
        for h in range(w.Hq):
            for j in (0, 1, 500, w.n - 1):
                f.write(f"vote {h} {j} {float(res['vote'][0, h, j]).hex()}\n")
    print("wrote", path)


if __name__ == "__main__":
    main()
