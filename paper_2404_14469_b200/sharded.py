"""Compression of a prompt that is sharded along its length over the ranks of a process group.

The paper runs on one GPU and stops at what its memory holds (Sec. 5.1.1); Eq. 1-2 split over
ranges of keys, so R ranks that each hold the K/V of a contiguous range of positions can do the
step with two small exchanges and no movement of K or V:

  1. every rank computes its share of each window row's softmax normaliser
     (snapkv_shard_lse), the shares are all-gathered ([R, B, Hq, W] floats) and merged in
     rank order (snapkv_lse_merge): every rank holds the same lse_obs;
  2. every rank computes the votes of its own prefix keys (snapkv_shard_votes); the vote
     shards are all-gathered (4 bytes per key and head: what the single-GPU path keeps in its
     workspace), and every rank runs pooling + top-k on the whole rows (snapkv_pool_topk): no
     halo exchange, identical index lists everywhere, ties included;
  3. every rank copies the selected rows that live in its shard (snapkv_gather_range); the
     rank that holds the window appends the window rows.  The compressed cache stays sharded:
     a head's rows are the ranks' segments in rank order.

The collectives go through torch.distributed (NCCL on GPUs: the gathered data lands in local
memory before any kernel reads it).  `ops` carries the per-shard steps; the default is the
CUDA library.  The tests run the same protocol on CPU ranks (gloo) with a stand-in built on
the oracle, which is how the exchange logic is checked without several GPUs.
"""
from __future__ import annotations

import torch


class LibraryOps:
    """The per-shard steps as the CUDA library does them."""

    def __init__(self):
        from . import binding as sk

        self.sk = sk
        self.ws = None

    def shard_lse(self, q_obs, k_shard, mask_n):
        out, self.ws = self.sk.snapkv_shard_lse(q_obs, k_shard, mask_n, self.ws)
        return out

    def lse_merge(self, parts):
        return self.sk.snapkv_lse_merge(parts)

    def shard_votes(self, q_obs, k_shard, lse, n_vote):
        out, self.ws = self.sk.snapkv_shard_votes(q_obs, k_shard, lse, n_vote, self.ws)
        return out

    def pool_topk(self, vote_rows, pool_kernel, pool_type, ksel):
        return self.sk.snapkv_pool_topk(vote_rows, pool_kernel, pool_type, ksel)

    def gather_range(self, k_shard, v_shard, idx, pos0, append):
        return self.sk.snapkv_gather_range(k_shard, v_shard, idx, pos0, append)


def _group_info(group):
    import torch.distributed as dist

    if dist.is_available() and dist.is_initialized():
        return dist.get_rank(group), dist.get_world_size(group)
    return 0, 1


def _all_gather(t, group, world):
    if world == 1:
        return [t]
    import torch.distributed as dist

    out = [torch.empty_like(t) for _ in range(world)]
    dist.all_gather(out, t.contiguous(), group=group)
    return out


def _protocol(rank, world, q_obs, k_shard, v_shard, shard_lens, pool_kernel, pool_type, budget, ops):
    """One rank's side of the exchange, as a generator: it yields the tensor it contributes to an
    all-gather and is sent back the list of all ranks' tensors, twice; its return value is the
    rank's result."""
    lens = [int(x) for x in shard_lens]
    if len(lens) != world:
        raise ValueError("one shard length per rank is needed")
    B, Hq, W, d = q_obs.shape
    Ls = lens[rank]
    if k_shard.shape[2] != Ls or tuple(v_shard.shape) != tuple(k_shard.shape):
        raise ValueError("k_shard / v_shard do not have this rank's shard length")
    if min(lens) < W:
        raise ValueError("every shard must hold at least W positions (the last one holds the window)")
    L = sum(lens)
    n = L - W
    pos0 = sum(lens[:rank])
    ksel = min(budget, L) - W

    # 1. normalisers
    part = ops.shard_lse(q_obs, k_shard, n - pos0)
    parts = yield part
    lse = ops.lse_merge(torch.stack(list(parts)).contiguous())

    # 2. votes of this rank's prefix keys, then the whole rows everywhere
    n_votes = [max(0, min(lens[r], n - sum(lens[:r]))) for r in range(world)]
    width = max(n_votes)
    mine = torch.zeros(B, Hq, width, dtype=getattr(ops, "vote_dtype", torch.float32), device=k_shard.device)
    if n_votes[rank] > 0:
        mine[:, :, : n_votes[rank]] = ops.shard_votes(q_obs, k_shard, lse, n_votes[rank])
    gathered = yield mine
    votes = torch.cat([g[:, :, : n_votes[r]] for r, g in enumerate(gathered)], dim=2).contiguous()

    # 3. selection on whole rows (budget >= L keeps everything: Listing 1's early return)
    if budget >= L:
        idx = torch.arange(n, dtype=torch.int32, device=k_shard.device).expand(B, Hq, n).contiguous()
    else:
        idx = ops.pool_topk(votes.view(B * Hq, n), pool_kernel, pool_type, ksel).view(B, Hq, ksel)

    # 4. this rank's rows
    out_k, out_v, seg = ops.gather_range(k_shard, v_shard, idx, pos0, W if rank == world - 1 else 0)
    return {"out_idx": idx, "out_k": out_k, "out_v": out_v, "seg": seg, "lse_obs": lse, "votes": votes}


def compress_sharded(q_obs, k_shard, v_shard, shard_lens, pool_kernel: int, pool_type: int, budget: int,
                     group=None, ops=None):
    """q_obs [B, Hq, W, d] (the same on every rank); k_shard, v_shard [B, Hkv, shard_lens[rank], d]:
    this rank's positions; shard_lens: the R shard lengths in rank order.

    Returns a dict: out_idx int32 [B, Hq, ksel] (global positions, the same on every rank),
    out_k / out_v [B, Hq, rows, d] with this rank's segment of every head's compressed rows
    first (then, on the last rank, the window rows), seg int32 [B, Hq, 2] = (first entry of the
    segment in out_idx, entries), lse_obs fp32 [B, Hq, W], votes fp32 [B, Hq, n]."""
    rank, world = _group_info(group)
    gen = _protocol(rank, world, q_obs, k_shard, v_shard, shard_lens, pool_kernel, pool_type, budget,
                    ops or LibraryOps())
    x = next(gen)
    while True:
        try:
            x = gen.send(_all_gather(x, group, world))
        except StopIteration as done:
            return done.value


def compress_sharded_local(q_obs, k_shards, v_shards, pool_kernel: int, pool_type: int, budget: int, ops=None):
    """The same protocol with every shard in this process (a prompt held as several chunks on
    one GPU, or a dry run of the multi-GPU exchange): the shards take the ranks' parts in turn
    and the "all-gather" is a list.  Returns one result dict per shard."""
    ops = ops or LibraryOps()
    world = len(k_shards)
    lens = [int(k.shape[2]) for k in k_shards]
    gens = [_protocol(r, world, q_obs, k_shards[r], v_shards[r], lens, pool_kernel, pool_type, budget, ops)
            for r in range(world)]
    xs = [next(g) for g in gens]
    results = [None] * world
    while any(r is None for r in results):
        nxt = []
        for r, g in enumerate(gens):
            try:
                nxt.append(g.send(xs))
            except StopIteration as done:
                results[r] = done.value
        xs = nxt
    return results


def assemble(results, W):
    """Concatenate the shards' segments (in shard order) and the window rows into the dense
    compressed cache [B, Hq, ksel + W, d] that the single-GPU step returns (for checking, or
    for a consumer that wants the whole cache in one place)."""
    idx = results[0]["out_idx"]
    B, Hq, ksel = idx.shape
    d = results[0]["out_k"].shape[-1]
    out_k = torch.empty(B, Hq, ksel + W, d, dtype=results[0]["out_k"].dtype, device=idx.device)
    out_v = torch.empty_like(out_k)
    segs = [r["seg"].cpu() for r in results]
    for b in range(B):
        for h in range(Hq):
            at = 0
            for r, res in enumerate(results):
                first, cnt = int(segs[r][b, h, 0]), int(segs[r][b, h, 1])
                assert first == at, "segments must tile the index list in shard order"
                extra = W if r == len(results) - 1 else 0
                out_k[b, h, at:at + cnt + extra] = res["out_k"][b, h, : cnt + extra]
                out_v[b, h, at:at + cnt + extra] = res["out_v"][b, h, : cnt + extra]
                at += cnt
            assert at == ksel
    return out_k, out_v
