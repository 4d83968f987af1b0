"""The exchange of the length-sharded step (paper_2404_14469_b200/sharded.py) on CPU ranks: two
and three gloo processes run the real protocol code with the per-shard steps supplied by the
oracle, and the assembled result must be the oracle's unsharded step.  This checks the
host-side logic - who sends what, offsets, the order of the merge, the tie rule across shard
edges - without several GPUs; the kernels behind the per-shard steps are checked against the
same oracle in tests/test_gpu_sharded.py."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


class OracleOps:
    """Per-shard steps on CPU tensors, straight from the oracle (fp64 votes)."""
    vote_dtype = torch.float64

    def __init__(self):
        sys.path.insert(0, ROOT)
        from oracle import snapkv_oracle as orc
        from paper_2404_14469_b200 import synth
        self.orc, self.synth = orc, synth

    def _f64(self, t):
        return self.orc.bf16_bits_to_f64(self.synth.bf16_bits(t))

    def shard_lse(self, q_obs, k_shard, mask_n):
        q, k = self._f64(q_obs), self._f64(k_shard)
        B, Hq, W, _ = q.shape
        g = Hq // k.shape[1]
        out = np.empty((B, Hq, W))
        for b in range(B):
            for h in range(Hq):
                out[b, h] = self.orc.shard_lse(q[b, h], k[b, h // g], 0, mask_n)
        return torch.from_numpy(out)

    def lse_merge(self, parts):
        return torch.from_numpy(self.orc.merge_lse(parts.numpy()))

    def shard_votes(self, q_obs, k_shard, lse, n_vote):
        q, k = self._f64(q_obs), self._f64(k_shard)
        B, Hq, W, _ = q.shape
        g = Hq // k.shape[1]
        out = np.empty((B, Hq, n_vote))
        for b in range(B):
            for h in range(Hq):
                out[b, h] = self.orc.shard_votes(q[b, h], k[b, h // g], lse[b, h].numpy(), n_vote)
        return torch.from_numpy(out)

    def pool_topk(self, vote_rows, pool_kernel, pool_type, ksel):
        rows = [self.orc.topk_positions(self.orc.pool1d(v.numpy(), pool_kernel, pool_type), ksel) for v in vote_rows]
        return torch.from_numpy(np.stack(rows).astype(np.int32))

    def gather_range(self, k_shard, v_shard, idx, pos0, append):
        B, Hkv, Ls, d = k_shard.shape
        _, Hq, ksel = idx.shape
        g = Hq // Hkv
        rows = min(ksel, Ls) + append
        out_k = torch.zeros(B, Hq, rows, d, dtype=k_shard.dtype)
        out_v = torch.zeros_like(out_k)
        seg = torch.zeros(B, Hq, 2, dtype=torch.int32)
        for b in range(B):
            for h in range(Hq):
                sel = idx[b, h].numpy()
                lo, hi = int(np.searchsorted(sel, pos0)), int(np.searchsorted(sel, pos0 + Ls))
                local = torch.from_numpy(sel[lo:hi].astype(np.int64) - pos0)
                out_k[b, h, : hi - lo] = k_shard[b, h // g][local]
                out_v[b, h, : hi - lo] = v_shard[b, h // g][local]
                if append:
                    out_k[b, h, hi - lo: hi - lo + append] = k_shard[b, h // g, Ls - append:]
                    out_v[b, h, hi - lo: hi - lo + append] = v_shard[b, h // g, Ls - append:]
                seg[b, h, 0], seg[b, h, 1] = lo, hi - lo
        return out_k, out_v, seg


def _case(name):
    sys.path.insert(0, ROOT)
    from paper_2404_14469_b200 import synth
    if name == "plain":
        data = synth.make_layer(synth.Workload(70, "t", 2, 4, 2, 32, 900, 16, 7, "max", (96,), 1, 3), 1)
        return data, 7, 0, 96
    if name == "avg":
        data = synth.make_layer(synth.Workload(71, "t", 1, 4, 4, 32, 700, 16, 5, "avg", (200,), 1, 2), 2)
        return data, 5, 1, 200
    if name == "plateau":
        # one dominant key just before a shard edge (position 299 with cuts at 300): under max
        # pooling of width 7 its plateau covers 296..302 on both sides of the edge, and with five
        # rows to keep the cut falls inside the plateau: the lower positions must win
        data = synth.make_random(1, 2, 2, 600, 32, 16, seed=8)
        u = data["q_obs"][0, :, :, :].float().mean(dim=1)
        data["k"][0, :, 299, :] = (6.0 * u / u.norm(dim=-1, keepdim=True) * 4).to(torch.bfloat16)
        return data, 7, 0, 16 + 5
    if name == "identity":
        data = synth.make_random(1, 2, 1, 500, 32, 16, seed=9)
        return data, 7, 0, 600
    raise KeyError(name)


def _worker(rank, world, port, lens, name, out):
    sys.path.insert(0, ROOT)
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    import torch.distributed as dist
    from paper_2404_14469_b200 import sharded
    dist.init_process_group("gloo")
    data, kernel, ptype, budget = _case(name)
    lo = sum(lens[:rank])
    k = data["k"][:, :, lo:lo + lens[rank]].contiguous()
    v = data["v"][:, :, lo:lo + lens[rank]].contiguous()
    res = sharded.compress_sharded(data["q_obs"], k, v, lens, kernel, ptype, budget, ops=OracleOps())
    out.put((rank, {x: res[x].numpy() if res[x].dtype != torch.bfloat16 else res[x].view(torch.int16).numpy()
                    for x in ("out_idx", "out_k", "out_v", "seg")}))
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("lens,name", [
    ([300, 600], "plain"), ([100, 500, 300], "plain"), ([884, 16], "plain"),
    ([350, 350], "avg"), ([300, 300], "plateau"), ([200, 100, 300], "plateau"), ([250, 250], "identity"),
])
def test_sharded_protocol_on_gloo_ranks_equals_the_unsharded_oracle(lens, name):
    sys.path.insert(0, ROOT)
    from oracle import snapkv_oracle as orc
    from paper_2404_14469_b200 import synth
    world = len(lens)
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, lens, name, out)) for r in range(world)]
    for p in procs:
        p.start()
    got = dict(out.get(timeout=300) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    data, kernel, ptype, budget = _case(name)
    q, k, v = (synth.bf16_bits(data[x]) for x in ("q_obs", "k", "v"))
    ref = orc.compress(q, k, v, kernel, ptype, budget)
    B, Hq = q.shape[:2]
    W = q.shape[2]
    ksel = ref["out_idx"].shape[2]
    for r in range(world):
        assert np.array_equal(got[r]["out_idx"], got[0]["out_idx"])        # the same list on every rank
    assert np.array_equal(got[0]["out_idx"], ref["out_idx"])
    if name == "plateau":
        assert np.array_equal(got[0]["out_idx"][0, 0], np.arange(296, 301))  # the plateau's lowest five
    for b in range(B):
        for h in range(Hq):
            at, rows_k, rows_v = 0, [], []
            for r in range(world):
                first, cnt = got[r]["seg"][b, h]
                assert first == at
                extra = W if r == world - 1 else 0
                rows_k.append(got[r]["out_k"][b, h, : cnt + extra])
                rows_v.append(got[r]["out_v"][b, h, : cnt + extra])
                at += cnt
            assert at == ksel
            assert np.array_equal(np.concatenate(rows_k).view(np.uint16), ref["out_k"][b, h])
            assert np.array_equal(np.concatenate(rows_v).view(np.uint16), ref["out_v"][b, h])
