"""Plain CPU oracle for the SnapKV prompt KV-cache compression step.

TEST INFRASTRUCTURE ONLY.  This module is the slow, obviously-correct statement of
what the compression step computes, written from the paper (Sec. 4, Eq. 1-2 and
Listing 1) in fp64.  It shares no code with the CUDA path and must never be
imported by the product package; only the tests, the smoke check and the
benchmark's CPU-baseline leg call it.

Notation (paper, Sec. 4): L = L_prompt, W = L_obs (observation window), n = L - W =
L_prefix, k = budget - W selected prefix rows, r = pool_kernel // 2.

Inputs are bf16 tensors passed as numpy uint16 bit patterns so that no precision
is lost or invented on the way in and the gathered rows can be compared bit for
bit.  Shapes follow Listing 1: q_obs [B, Hq, W, d] (the last W prompt queries),
k and v [B, Hkv, L, d].  With grouped-query attention query head h reads KV head
h // (Hq // Hkv).

Readings of points the paper leaves open (all listed again in the design notes):
  * logits are q.k / sqrt(d), the mask is purely causal: window row i sees keys
    j <= n + i;
  * the softmax normaliser runs over every visible key (prefix and window), the
    slice to the prefix happens after normalisation (Listing 1 slices after
    compute_attn);
  * Eq. 1's sum runs over the W window rows (Listing 1's .sum over the window axis);
  * k = budget - W (Listing 1), not floor(p * L_prefix);
  * average pooling divides by pool_kernel everywhere (zero padding counted);
    max pooling ignores positions outside [0, n);
  * ties in the top-k go to the lower position; indices are emitted ascending;
  * budget >= L is the identity.

A variant outside the paper's listing is stated too: votes_given_lse / window_lse /
lse_obs / compress(lse=...) take the window rows' log-sum-exp as an input (the prompt
phase's attention kernel holds it) instead of recomputing the softmax.

A second one, for grouped-query attention: group_votes / compress_grouped let the query
heads of a group select TOGETHER on the KV head they share (Eq. 1's sum runs over the
window rows of all the group's heads), which keeps the compressed cache at Hkv heads.

read_paged / compress_paged read K and V through a block table (a paged cache: position p of
sequence b is row p % page_size of page table[b][p // page_size] of a pool), one element row
at a time, and then run the very same step: paging changes where a row lives, not what the
method computes.

shard_lse / merge_lse / shard_votes split Eq. 1 over ranges of keys (a prompt sharded along
its length): a row's normaliser is the sum of the shards' shares, and a key's vote needs only
its own logits and the merged normalisers.

hit_counts / hit_rate state the paper's hit-rate measure of a selection (Sec. 3, Eq. 3-7);
decode_attention is the generation step's attention over the compressed cache (Sec. 5.1.2).

Every function here is pinned by tests that do not go through this file's own
formulas (closed forms, invariants, library routines, brute force): see
tests/test_oracle_*.py.  Nothing is "parity unpinned".
"""
from __future__ import annotations

import math
from concurrent.futures import ThreadPoolExecutor

import numpy as np

POOL_MAX = 0
POOL_AVG = 1


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns (uint16) to fp64 exactly.

    A bf16 number is the upper half of an IEEE fp32 number, so placing the 16 bits
    in the high half of a 32-bit word and reading it as fp32 is exact.
    """
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    with np.errstate(invalid="ignore"):  # signalling-NaN patterns are quieted by the cast
        return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def window_logits(q_head: np.ndarray, k_head: np.ndarray) -> np.ndarray:
    """s[i, j] = q_i . k_j / sqrt(d) for one head (Listing 1, compute_attn).

    q_head: [W, d] fp64, k_head: [L, d] fp64 -> [W, L] fp64.
    """
    d = q_head.shape[-1]
    return (q_head @ k_head.T) / math.sqrt(d)


def window_softmax(s: np.ndarray) -> np.ndarray:
    """Causally masked, softmax-normalised attention of the window rows (Sec. 4,
    "softmax-normalized attention features").

    s: [W, L] logits.  Window row i is prompt position n + i and sees keys
    j <= n + i.  Returns p [W, L] with zeros at masked positions; every row sums
    to one over its visible keys.
    """
    W, L = s.shape
    n = L - W
    j = np.arange(L)[None, :]
    i = np.arange(W)[:, None]
    visible = j <= (n + i)
    masked = np.where(visible, s, -np.inf)
    m = masked.max(axis=1, keepdims=True)
    e = np.where(visible, np.exp(masked - m), 0.0)
    return e / e.sum(axis=1, keepdims=True)


def vote_from_probs(p: np.ndarray) -> np.ndarray:
    """Eq. 1: C[j] = sum over the W window rows of p[i, j], prefix columns only."""
    W, L = p.shape
    n = L - W
    return p[:, :n].sum(axis=0)


def window_votes(q_head: np.ndarray, k_head: np.ndarray) -> np.ndarray:
    """Steps score -> softmax -> vote for one head: [W,d],[L,d] -> [n]."""
    return vote_from_probs(window_softmax(window_logits(q_head, k_head)))


def window_lse(s: np.ndarray) -> np.ndarray:
    """Natural-log sum-exp of every window row over the keys it sees (the normaliser of
    Sec. 4's softmax, as a prefill attention kernel would hand it on): [W, L] -> [W]."""
    W, L = s.shape
    n = L - W
    out = np.empty(W, dtype=np.float64)
    for i in range(W):
        row = s[i, : n + i + 1]
        m = row.max()
        out[i] = m + math.log(np.exp(row - m).sum())
    return out


def votes_given_lse(s: np.ndarray, lse: np.ndarray) -> np.ndarray:
    """Eq. 1 with the normaliser supplied: C[j] = sum_i exp(s[i, j] - lse[i]) over the W
    window rows, prefix columns only (every prefix key is visible to every window row).
    Not in the paper's listing, which recomputes the softmax; same result when `lse` is
    the rows' own log-sum-exp."""
    W, L = s.shape
    n = L - W
    return np.exp(s[:, :n] - lse[:, None]).sum(axis=0)


def lse_obs(q_obs: np.ndarray, k: np.ndarray) -> np.ndarray:
    """window_lse for every (batch, query head): bf16 bits in, fp64 [B, Hq, W] out."""
    B, Hq, W, d = q_obs.shape
    _, Hkv, L, _ = k.shape
    g = Hq // Hkv
    out = np.empty((B, Hq, W), dtype=np.float64)
    for b in range(B):
        for c in range(Hkv):
            kf = bf16_bits_to_f64(k[b, c])
            for h in range(c * g, (c + 1) * g):
                out[b, h] = window_lse(window_logits(bf16_bits_to_f64(q_obs[b, h]), kf))
    return out


def pool1d(vote: np.ndarray, pool_kernel: int, pool_type: int) -> np.ndarray:
    """Listing 1's pool1d(kernel_size, padding=kernel_size//2, stride=1) on one row.

    max: maximum over the in-range neighbours |t| <= r.
    avg: sum over the in-range neighbours divided by pool_kernel (zero padding
    counted in the divisor).
    """
    if pool_kernel < 1 or pool_kernel % 2 == 0:
        raise ValueError("pool_kernel must be odd and >= 1")
    if pool_type not in (POOL_MAX, POOL_AVG):
        raise ValueError("pool_type must be POOL_MAX or POOL_AVG")
    n = vote.shape[0]
    r = pool_kernel // 2
    # Pad r positions on both sides with the neutral element, then look at the
    # pool_kernel shifted copies: copy t holds vote[j + t - r] at position j.
    fill = -np.inf if pool_type == POOL_MAX else 0.0
    padded = np.concatenate([np.full(r, fill), vote.astype(np.float64), np.full(r, fill)])
    shifted = np.stack([padded[t:t + n] for t in range(pool_kernel)])
    if pool_type == POOL_MAX:
        return shifted.max(axis=0)
    return shifted.sum(axis=0) / pool_kernel


def topk_positions(pooled: np.ndarray, k: int) -> np.ndarray:
    """Eq. 2: the k positions of largest pooled vote, ties to the lower position,
    returned in ascending position order (int64)."""
    n = pooled.shape[0]
    if not 0 <= k <= n:
        raise ValueError("k out of range")
    order = np.argsort(-pooled, kind="stable")  # value descending, index ascending
    return np.sort(order[:k])


def kv_head_of(h: int, Hq: int, Hkv: int) -> int:
    """Consecutive query heads share one KV head."""
    return h // (Hq // Hkv)


def _check_shapes(q_obs, k, v):
    B, Hq, W, d = q_obs.shape
    Bk, Hkv, L, dk = k.shape
    if v.shape != k.shape or Bk != B or dk != d:
        raise ValueError("inconsistent shapes")
    if Hq % Hkv != 0:
        raise ValueError("Hq must be a multiple of Hkv")
    if W > L:
        raise ValueError("window longer than the prompt")
    return B, Hq, Hkv, L, d, W


def votes(q_obs: np.ndarray, k: np.ndarray, workers: int = 1) -> np.ndarray:
    """Votes for every (batch, query head): bf16 bits in, fp64 [B, Hq, n] out."""
    B, Hq, W, d = q_obs.shape
    _, Hkv, L, _ = k.shape
    n = L - W
    out = np.empty((B, Hq, n), dtype=np.float64)

    def unit(bc):
        b, c = bc
        kf = bf16_bits_to_f64(k[b, c])
        g = Hq // Hkv
        for h in range(c * g, (c + 1) * g):
            out[b, h] = window_votes(bf16_bits_to_f64(q_obs[b, h]), kf)

    units = [(b, c) for b in range(B) for c in range(Hkv)]
    if workers > 1:
        with ThreadPoolExecutor(max_workers=workers) as ex:
            list(ex.map(unit, units))
    else:
        for u in units:
            unit(u)
    return out


def compress(q_obs: np.ndarray, k: np.ndarray, v: np.ndarray, pool_kernel: int,
             pool_type: int, budget: int, workers: int = 1, heads=None, lse=None):
    """The whole step (Listing 1) on bf16 bit patterns.

    Returns a dict with
      out_k, out_v : uint16 [B, Hq, rows, d], rows = min(budget, L)
      out_idx      : int64  [B, Hq, rows - W] ascending prefix positions
      vote, pooled : fp64   [B, Hq, n] (None on the identity path)
    `heads` optionally restricts the work to a list of (b, h) pairs (other heads
    are left zero) so that sampled checks at large sizes stay affordable.
    `lse` (fp64 [B, Hq, W]) switches to the supplied-normaliser variant: votes are
    votes_given_lse instead of window_votes; everything after the vote is the same.
    """
    B, Hq, Hkv, L, d, W = _check_shapes(q_obs, k, v)
    if budget <= W:
        raise ValueError("budget must exceed the window")
    n = L - W
    g = Hq // Hkv
    if budget >= L:  # Listing 1's early return: nothing is dropped
        kv_of = [kv_head_of(h, Hq, Hkv) for h in range(Hq)]
        return {
            "out_k": np.ascontiguousarray(k[:, kv_of]),
            "out_v": np.ascontiguousarray(v[:, kv_of]),
            "out_idx": np.broadcast_to(np.arange(n, dtype=np.int64), (B, Hq, n)).copy(),
            "vote": None,
            "pooled": None,
        }
    ksel = budget - W
    out_k = np.zeros((B, Hq, budget, d), dtype=np.uint16)
    out_v = np.zeros((B, Hq, budget, d), dtype=np.uint16)
    out_idx = np.zeros((B, Hq, ksel), dtype=np.int64)
    vote = np.zeros((B, Hq, n), dtype=np.float64)
    pooled = np.zeros((B, Hq, n), dtype=np.float64)

    wanted = None if heads is None else set(heads)

    def unit(bc):
        b, c = bc
        hs = [h for h in range(c * g, (c + 1) * g) if wanted is None or (b, h) in wanted]
        if not hs:
            return
        kf = bf16_bits_to_f64(k[b, c])
        for h in hs:
            if lse is None:
                vt = window_votes(bf16_bits_to_f64(q_obs[b, h]), kf)
            else:
                vt = votes_given_lse(window_logits(bf16_bits_to_f64(q_obs[b, h]), kf), lse[b, h])
            pv = pool1d(vt, pool_kernel, pool_type)
            idx = topk_positions(pv, ksel)
            vote[b, h] = vt
            pooled[b, h] = pv
            out_idx[b, h] = idx
            out_k[b, h, :ksel] = k[b, c, idx]
            out_v[b, h, :ksel] = v[b, c, idx]
            out_k[b, h, ksel:] = k[b, c, n:]
            out_v[b, h, ksel:] = v[b, c, n:]

    units = [(b, c) for b in range(B) for c in range(Hkv)]
    if workers > 1:
        with ThreadPoolExecutor(max_workers=workers) as ex:
            list(ex.map(unit, units))
    else:
        for u in units:
            unit(u)
    return {"out_k": out_k, "out_v": out_v, "out_idx": out_idx, "vote": vote, "pooled": pooled}


def group_votes(vote_heads: np.ndarray) -> np.ndarray:
    """Shared selection under grouped-query attention: all window queries of all query
    heads of a group vote on the keys of the KV head they share,
    C_group[j] = sum over the group's heads h and window rows i of p_h[i, j]
    (Eq. 1 with the sum extended over the group's heads).  [g, n] -> [n]."""
    g, n = vote_heads.shape
    out = np.zeros(n, dtype=np.float64)
    for h in range(g):
        out = out + vote_heads[h]
    return out


def compress_grouped(q_obs: np.ndarray, k: np.ndarray, v: np.ndarray, pool_kernel: int,
                     pool_type: int, budget: int, lse=None, kv_heads=None):
    """The step with ONE selection per KV head (Listing 1 applied to the KV head with the
    votes of its whole query group): score and vote per query head as in `compress`, sum the
    votes over the group (group_votes), then pool, top-k and gather per KV head.

    Returns a dict with
      out_k, out_v : uint16 [B, Hkv, rows, d], rows = min(budget, L)
      out_idx      : int64  [B, Hkv, rows - W] ascending prefix positions
      vote, pooled : fp64   [B, Hkv, n] group votes (None on the identity path)
    With Hq == Hkv this is `compress`.  `lse` as in `compress`; `kv_heads` optionally
    restricts the work to a list of (b, c) pairs.
    """
    B, Hq, Hkv, L, d, W = _check_shapes(q_obs, k, v)
    if budget <= W:
        raise ValueError("budget must exceed the window")
    n = L - W
    g = Hq // Hkv
    if budget >= L:
        return {
            "out_k": np.ascontiguousarray(k),
            "out_v": np.ascontiguousarray(v),
            "out_idx": np.broadcast_to(np.arange(n, dtype=np.int64), (B, Hkv, n)).copy(),
            "vote": None,
            "pooled": None,
        }
    ksel = budget - W
    out_k = np.zeros((B, Hkv, budget, d), dtype=np.uint16)
    out_v = np.zeros((B, Hkv, budget, d), dtype=np.uint16)
    out_idx = np.zeros((B, Hkv, ksel), dtype=np.int64)
    vote = np.zeros((B, Hkv, n), dtype=np.float64)
    pooled = np.zeros((B, Hkv, n), dtype=np.float64)
    wanted = None if kv_heads is None else set(kv_heads)
    for b in range(B):
        for c in range(Hkv):
            if wanted is not None and (b, c) not in wanted:
                continue
            kf = bf16_bits_to_f64(k[b, c])
            per_head = np.empty((g, n), dtype=np.float64)
            for t, h in enumerate(range(c * g, (c + 1) * g)):
                qf = bf16_bits_to_f64(q_obs[b, h])
                if lse is None:
                    per_head[t] = window_votes(qf, kf)
                else:
                    per_head[t] = votes_given_lse(window_logits(qf, kf), lse[b, h])
            vt = group_votes(per_head)
            pv = pool1d(vt, pool_kernel, pool_type)
            idx = topk_positions(pv, ksel)
            vote[b, c] = vt
            pooled[b, c] = pv
            out_idx[b, c] = idx
            out_k[b, c, :ksel] = k[b, c, idx]
            out_v[b, c, :ksel] = v[b, c, idx]
            out_k[b, c, ksel:] = k[b, c, n:]
            out_v[b, c, ksel:] = v[b, c, n:]
    return {"out_k": out_k, "out_v": out_v, "out_idx": out_idx, "vote": vote, "pooled": pooled}


def shard_lse(q_head: np.ndarray, k_shard_head: np.ndarray, pos0: int, n_total: int) -> np.ndarray:
    """One head, one shard holding positions [pos0, pos0 + Ls) of the prompt: for every window
    row i the log of the sum of exp(logit) over the shard's keys the row may see (global
    position <= n_total + i).  -inf where the row sees none of them.  [W] fp64."""
    W = q_head.shape[0]
    Ls = k_shard_head.shape[0]
    s = window_logits(q_head, k_shard_head)          # [W, Ls]
    out = np.full(W, -np.inf)
    for i in range(W):
        seen = min(Ls, n_total + i - pos0 + 1)       # local keys 0 .. seen-1
        if seen > 0:
            row = s[i, :seen]
            m = row.max()
            out[i] = m + math.log(np.exp(row - m).sum())
    return out


def merge_lse(parts: np.ndarray) -> np.ndarray:
    """log sum_r exp(parts[r]) over the first axis (the shards' shares of a normaliser)."""
    m = parts.max(axis=0)
    safe = np.where(np.isfinite(m), m, 0.0)
    return safe + np.log(np.exp(parts - safe).sum(axis=0))


def shard_votes(q_head: np.ndarray, k_shard_head: np.ndarray, lse: np.ndarray, n_vote: int) -> np.ndarray:
    """Eq. 1 for the first n_vote keys of a shard, given every window row's log-sum-exp over
    the WHOLE prompt: vote_j = sum_i exp(logit_ij - lse_i).  Prefix keys are seen by every row,
    so no mask is involved.  [n_vote] fp64."""
    s = window_logits(q_head, k_shard_head[:n_vote])
    return np.exp(s - lse[:, None]).sum(axis=0)


def read_paged(pool: np.ndarray, table_row, page_size: int, length: int) -> np.ndarray:
    """The first `length` positions of one sequence of a paged cache as a dense
    [Hkv, length, d] array.  pool: [num_pages, Hkv, page_size, d]; table_row: page numbers."""
    num_pages, Hkv, ps, d = pool.shape
    assert ps == page_size
    out = np.empty((Hkv, length, d), dtype=pool.dtype)
    for p in range(length):
        page = int(table_row[p // page_size])
        if 0 <= page < num_pages:
            out[:, p, :] = pool[page, :, p % page_size, :]
        else:
            out[:, p, :] = 0      # an entry that names no page of the pool reads as zeros
    return out


def compress_paged(q_obs: np.ndarray, k_pool: np.ndarray, v_pool: np.ndarray, page_table,
                   page_size: int, seq_lens, pool_kernel: int, pool_type: int, budget: int,
                   lse=None):
    """Listing 1 per sequence on a paged cache.  q_obs [B, Hq, W, d]; pools
    [num_pages, Hkv, page_size, d] (bf16 bit patterns); page_table [B, pages_per_seq];
    seq_lens: B prompt lengths.  Returns one `compress` result per sequence."""
    results = []
    for b, length in enumerate(seq_lens):
        k = read_paged(k_pool, page_table[b], page_size, int(length))[None]
        v = read_paged(v_pool, page_table[b], page_size, int(length))[None]
        results.append(compress(q_obs[b:b + 1], k, v, pool_kernel, pool_type, budget,
                                lse=None if lse is None else lse[b:b + 1]))
    return results


def hit_counts(a_cur: np.ndarray, idx: np.ndarray, theta) -> np.ndarray:
    """Sec. 3, Eq. 3-7 per head: a_cur fp32 [N, L_prefix] (attention of one generated query over
    the prefix keys), idx int [N, k] (positions chosen by the vote).  Builds the two masks of
    the definition, M_vote_obs (ones at idx) and M_threshold_cur (a_cur > theta, compared in
    fp32 as given), and returns int64 [N, 2]: per head the overlap sum(O) and sum(M_threshold_cur).
    """
    a = np.asarray(a_cur, dtype=np.float32)
    N, n = a.shape
    m_vote = np.zeros((N, n), dtype=bool)
    for h in range(N):
        m_vote[h, np.asarray(idx[h], dtype=np.int64)] = True
    m_thr = a > np.float32(theta)
    overlap = np.logical_and(m_thr, m_vote)
    return np.stack([overlap.sum(axis=1), m_thr.sum(axis=1)], axis=1).astype(np.int64)


def hit_rate(a_cur: np.ndarray, idx: np.ndarray, theta) -> float:
    """Eq. 7: H = sum(O) / sum(M_threshold_cur) over all heads (nan when nothing is important)."""
    c = hit_counts(a_cur, idx, theta)
    return float(c[:, 0].sum()) / float(c[:, 1].sum()) if c[:, 1].sum() > 0 else float("nan")


def decode_attention(q_cur: np.ndarray, cache_k: np.ndarray, cache_v: np.ndarray):
    """One generation step's attention over the compressed cache (Sec. 4.1: the compressed
    keys and values are what later steps attend to; Sec. 5.1.2 measures exactly this
    decoding).  bf16 bit patterns in: q_cur [B, Hq, d] (the generated token's queries),
    cache_k / cache_v [B, Hc, R, d] with Hc dividing Hq (query head h reads cache head
    h // (Hq // Hc): Hc = Hq for the expanded cache, Hc = Hkv for one selection per KV head).
    Every cache row is visible (they all precede the generated token).  Returns fp64
      out   [B, Hq, d]  sum_j p_j v_j,  p = softmax_j(q . k_j / sqrt(d))
      lse   [B, Hq]     natural-log sum-exp of the logits
      scale [B, Hq, d]  sum_j p_j |v_j|: the magnitude rounding errors are judged against.
    """
    B, Hq, d = q_cur.shape
    _, Hc, R, _ = cache_k.shape
    if Hq % Hc != 0 or cache_v.shape != cache_k.shape or cache_k.shape[0] != B or cache_k.shape[3] != d:
        raise ValueError("shapes do not fit")
    g = Hq // Hc
    out = np.zeros((B, Hq, d), dtype=np.float64)
    lse = np.zeros((B, Hq), dtype=np.float64)
    scale = np.zeros((B, Hq, d), dtype=np.float64)
    for b in range(B):
        for h in range(Hq):
            q = bf16_bits_to_f64(q_cur[b, h])
            kf = bf16_bits_to_f64(cache_k[b, h // g])
            vf = bf16_bits_to_f64(cache_v[b, h // g])
            s = kf @ q / math.sqrt(d)
            m = s.max()
            e = np.exp(s - m)
            z = e.sum()
            p = e / z
            out[b, h] = p @ vf
            scale[b, h] = p @ np.abs(vf)
            lse[b, h] = m + math.log(z)
    return out, lse, scale
