"""snapkv_pool_topk_static: the pool + top-k entry point for hosts that cannot allocate
device memory when they call (frozen memory pools, code between the launches of a decode
loop, plug-ins without an allocator).  Its scratch is an array inside the library, shared
by all calls, so the checks below run two calls back to back and compare each with the
ordinary entry point on the same votes.  This file is collected last on purpose."""
import numpy as np
import pytest
import torch

from oracle import snapkv_oracle as orc
from paper_2404_14469_b200 import binding as sk

import parity

FAKE = 0x1000


def test_static_variant_rejects_what_does_not_fit_before_touching_the_device():
    L = sk.lib()
    too_many = sk.STATIC_MAX_KEYS // 1000 + 1
    assert L.snapkv_pool_topk_static(FAKE, too_many, 1000, 7, 0, 10, FAKE, None) == 3  # WORKSPACE
    assert L.snapkv_pool_topk_static(FAKE, 2, 100, 8, 0, 10, FAKE, None) == 1
    assert L.snapkv_pool_topk_static(FAKE, 2, 100, 7, 0, 101, FAKE, None) == 1
    assert L.snapkv_pool_topk_static(None, 2, 100, 7, 0, 10, FAKE, None) == 1


@pytest.mark.gpu
def test_static_variant_matches_the_ordinary_entry_point_on_two_calls_in_a_row():
    g = torch.Generator().manual_seed(2024)
    # first call: long rows (the ordinary entry point needs a workspace for these)
    vote_a = (torch.rand(3, 60001, generator=g) ** 4).cuda()
    # second call: shorter rows, other pooling; it finds the first call's keys in the array
    vote_b = (torch.rand(5, 20000, generator=g) ** 4).cuda()
    cases = [(vote_a, 5, sk.POOL_AVG, 1000), (vote_b, 7, sk.POOL_MAX, 2016)]
    for rounds in range(2):          # and once more in the opposite order of sizes
        for vote, kernel, ptype, ksel in (cases if rounds == 0 else cases[::-1]):
            out = torch.full((vote.shape[0], ksel), -1, dtype=torch.int32, device="cuda")
            sk.snapkv_pool_topk_static(vote, kernel, ptype, ksel, out)
            ref = sk.snapkv_pool_topk(vote, kernel, ptype, ksel)
            torch.cuda.synchronize()
            if ptype == sk.POOL_MAX:
                # max pooling is exact whatever the kernel: the index lists must be identical
                assert torch.equal(out, ref)
            else:
                # Average pooling: the two entry points run different kernels (a cluster of
                # CTAs per row that ranks by the fp32 window sum there, one CTA per row on the
                # built-in array that ranks by sum / kernel here), so their lists may differ
                # where two pooled votes are within an fp32 rounding of each other.  Both
                # must satisfy the acceptance rule against the oracle's pooled votes.
                for r_ in range(vote.shape[0]):
                    pooled = orc.pool1d(vote[r_].cpu().numpy().astype(np.float64), kernel, orc.POOL_AVG)
                    for got in (out, ref):
                        parity.check_indices(got[r_].cpu().numpy(), pooled, ksel)
            assert bool((out[:, 1:] > out[:, :-1]).all()) and int(out.min()) >= 0
            assert int(out.max()) < vote.shape[1]
