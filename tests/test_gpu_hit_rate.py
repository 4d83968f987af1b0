"""GPU parity for snapkv_hit_counts (Sec. 3, Eq. 3-7): exact integer counts against the oracle,
on random features, on features equal to the threshold, and on the selection the compression
step itself makes for the tiny workload."""
import numpy as np
import pytest
import torch

from oracle import snapkv_oracle as orc
from paper_2404_14469_b200 import binding as sk
from paper_2404_14469_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("rows,n,k,theta", [
    (4, 992, 224, 0.002),
    (32, 16352, 4064, 1e-4),
    (3, 5000, 5000, 0.5),        # everything selected
    (2, 100000, 7, 1e-5),        # several chunks per row, tiny selection
    (1, 1, 1, 0.0),
])
def test_counts_match_oracle_exactly(rows, n, k, theta):
    g = torch.Generator().manual_seed(rows * 7 + k)
    a = torch.rand(rows, n, generator=g) ** 8            # most mass near zero, a few large values
    a = a / a.sum(dim=1, keepdim=True) if n > 1 else a
    idx = torch.stack([torch.sort(torch.randperm(n, generator=g)[:k]).values for _ in range(rows)]).to(torch.int32)
    got = sk.snapkv_hit_counts(a.cuda(), idx.cuda(), theta).cpu().numpy()
    ref = orc.hit_counts(a.numpy(), idx.numpy(), theta)
    assert np.array_equal(got.astype(np.int64), ref)


def test_features_equal_to_the_threshold_are_not_important():
    a = torch.tensor([[0.25, 0.25, 0.5, 0.125]] * 3)
    idx = torch.tensor([[0, 2], [1, 3], [2, 3]], dtype=torch.int32)
    got = sk.snapkv_hit_counts(a.cuda(), idx.cuda(), 0.25).cpu().numpy()
    assert np.array_equal(got, orc.hit_counts(a.numpy(), idx.numpy(), 0.25))
    assert np.array_equal(got, [[1, 1], [0, 1], [1, 1]])


def test_hit_rate_of_the_steps_own_selection_on_the_tiny_workload():
    # a generated query pointing along the planted direction: its attention over the prefix is
    # concentrated on the planted clusters, which the window's vote selected
    w = synth.WORKLOADS[0]
    data = synth.make_layer(w, 0)
    q, k, v = (data[x].cuda() for x in ("q_obs", "k", "v"))
    _, _, out_idx, _ = sk.snapkv_compress(q, k, v, w.pool_kernel, sk.POOL_MAX, w.budgets[0])
    n = w.L - w.W
    q_cur = q[0, :, -1].float()                                        # [Hq, d]
    a_cur = torch.softmax(torch.einsum("hd,hjd->hj", q_cur, k[0, :, :n].float()) / w.d ** 0.5, dim=-1)
    a_cur = a_cur.contiguous()
    theta = 5.0 / n
    got = sk.snapkv_hit_counts(a_cur, out_idx[0].contiguous(), theta).cpu().numpy()
    ref = orc.hit_counts(a_cur.cpu().numpy(), out_idx[0].cpu().numpy(), theta)
    assert np.array_equal(got.astype(np.int64), ref)
    assert ref[:, 1].sum() > 0 and ref[:, 0].sum() / ref[:, 1].sum() > 0.5
