"""ctypes binding of libsnapkv.so: argument marshalling only.

Every step of the compression path runs in the library's CUDA kernels; torch is
used here for device memory (outputs, workspace) and for the current stream.  The
functions carry the names of the C entry points declared in include/snapkv.h.
If the library has not been built, or a call returns an error status, a
RuntimeError is raised: there is no fallback path.
"""
from __future__ import annotations

import ctypes
import os

import torch

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libsnapkv.so")

POOL_MAX = 0
POOL_AVG = 1
OK = 0

SYMBOLS = [
    "snapkv_status_string", "snapkv_out_rows", "snapkv_workspace_size", "snapkv_compress",
    "snapkv_window_scores", "snapkv_pool_topk_workspace_size", "snapkv_pool_topk", "snapkv_gather",
    "snapkv_host_staging_size", "snapkv_compress_host", "snapkv_device_status",
    "snapkv_last_launch_count", "snapkv_pool_topk_static",
    "snapkv_window_scores_lse", "snapkv_compress_lse", "snapkv_compress_strided",
    "snapkv_compress_grouped", "snapkv_compress_varlen",
    "snapkv_hit_counts", "snapkv_decode_workspace_size", "snapkv_decode_attention",
    "snapkv_set_wait_limit_ns", "snapkv_selftest_stalled_scores", "snapkv_schedule_items",
    "snapkv_compress_paged",
    "snapkv_shard_lse", "snapkv_lse_merge", "snapkv_shard_votes", "snapkv_gather_range",
]

_lib = None


class SnapKVError(RuntimeError):
    pass


def lib() -> ctypes.CDLL:
    """Load the shared library (once); raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise SnapKVError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2404_14469_b200.build` "
            "(there is no CPU or framework fallback)")
    L = ctypes.CDLL(LIB_PATH)
    c_int, c_sz, c_vp = ctypes.c_int, ctypes.c_size_t, ctypes.c_void_p
    L.snapkv_status_string.restype = ctypes.c_char_p
    L.snapkv_status_string.argtypes = [c_int]
    L.snapkv_out_rows.restype = c_int
    L.snapkv_out_rows.argtypes = [c_int, c_int]
    L.snapkv_workspace_size.restype = c_sz
    L.snapkv_workspace_size.argtypes = [c_int] * 9
    L.snapkv_compress.restype = c_int
    L.snapkv_compress.argtypes = [c_vp] * 3 + [c_int] * 9 + [c_vp] * 3 + [c_vp, c_sz, c_vp]
    L.snapkv_window_scores.restype = c_int
    L.snapkv_window_scores.argtypes = [c_vp] * 2 + [c_int] * 6 + [c_vp, c_vp, c_sz, c_vp]
    L.snapkv_window_scores_lse.restype = c_int
    L.snapkv_window_scores_lse.argtypes = [c_vp] * 3 + [c_int] * 6 + [c_vp, c_vp, c_sz, c_vp]
    L.snapkv_compress_lse.restype = c_int
    L.snapkv_compress_lse.argtypes = [c_vp] * 4 + [c_int] * 9 + [c_vp] * 3 + [c_vp, c_sz, c_vp]
    L.snapkv_compress_strided.restype = c_int
    L.snapkv_compress_strided.argtypes = ([c_vp] * 3 + [ctypes.POINTER(ctypes.c_int64)] * 2 + [c_vp]
                                          + [c_int] * 9 + [c_vp] * 3 + [c_vp, c_sz, c_vp])
    L.snapkv_compress_grouped.restype = c_int
    L.snapkv_compress_grouped.argtypes = L.snapkv_compress_strided.argtypes
    p64, p32 = ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(ctypes.c_int32)
    L.snapkv_compress_varlen.restype = c_int
    L.snapkv_compress_varlen.argtypes = ([c_vp] * 3 + [p64] * 4 + [p32, c_vp] + [c_int] * 9 + [c_vp] * 3
                                         + [c_vp, c_sz, c_vp])
    L.snapkv_compress_paged.restype = c_int
    L.snapkv_compress_paged.argtypes = ([c_vp] * 3 + [p64] * 2 + [c_vp] + [c_int] * 3 + [p32, c_vp]
                                        + [c_int] * 9 + [c_vp] * 3 + [c_vp, c_sz, c_vp])
    L.snapkv_shard_lse.restype = c_int
    L.snapkv_shard_lse.argtypes = [c_vp] * 2 + [c_int] * 7 + [c_vp, c_vp, c_sz, c_vp]
    L.snapkv_lse_merge.restype = c_int
    L.snapkv_lse_merge.argtypes = [c_vp, c_int, c_int, c_vp, c_vp]
    L.snapkv_shard_votes.restype = c_int
    L.snapkv_shard_votes.argtypes = [c_vp] * 3 + [c_int] * 7 + [c_vp, c_vp, c_sz, c_vp]
    L.snapkv_gather_range.restype = c_int
    L.snapkv_gather_range.argtypes = [c_vp] * 3 + [c_int] * 8 + [c_vp, c_vp, c_int, c_vp, c_vp]
    L.snapkv_hit_counts.restype = c_int
    L.snapkv_hit_counts.argtypes = [c_vp, c_vp, c_int, c_int, c_int, ctypes.c_float, c_vp, c_vp]
    L.snapkv_decode_workspace_size.restype = c_sz
    L.snapkv_decode_workspace_size.argtypes = [c_int] * 4
    L.snapkv_decode_attention.restype = c_int
    L.snapkv_decode_attention.argtypes = [c_vp] * 3 + [c_int] * 5 + [c_vp, c_vp, c_vp, c_sz, c_vp]
    L.snapkv_pool_topk_workspace_size.restype = c_sz
    L.snapkv_pool_topk_workspace_size.argtypes = [c_int, c_int]
    L.snapkv_pool_topk.restype = c_int
    L.snapkv_pool_topk.argtypes = [c_vp] + [c_int] * 5 + [c_vp, c_vp, c_sz, c_vp]
    L.snapkv_pool_topk_static.restype = c_int
    L.snapkv_pool_topk_static.argtypes = [c_vp] + [c_int] * 5 + [c_vp, c_vp]
    L.snapkv_gather.restype = c_int
    L.snapkv_gather.argtypes = [c_vp] * 3 + [c_int] * 7 + [c_vp] * 3
    L.snapkv_host_staging_size.restype = c_sz
    L.snapkv_host_staging_size.argtypes = [c_int] * 9
    L.snapkv_compress_host.restype = c_int
    L.snapkv_compress_host.argtypes = [c_vp] * 3 + [c_int] * 9 + [c_vp] * 3 + [c_vp, c_sz, c_vp]
    L.snapkv_device_status.restype = c_int
    L.snapkv_device_status.argtypes = [c_vp, c_vp, ctypes.POINTER(c_int)]
    L.snapkv_last_launch_count.restype = c_int
    L.snapkv_last_launch_count.argtypes = []
    L.snapkv_schedule_items.restype = c_int
    L.snapkv_schedule_items.argtypes = [c_int] * 9 + [ctypes.POINTER(ctypes.c_int32), c_int,
                                                      ctypes.POINTER(ctypes.c_int32)]
    L.snapkv_set_wait_limit_ns.restype = ctypes.c_ulonglong
    L.snapkv_set_wait_limit_ns.argtypes = [ctypes.c_ulonglong]
    L.snapkv_selftest_stalled_scores.restype = c_int
    L.snapkv_selftest_stalled_scores.argtypes = L.snapkv_window_scores.argtypes
    _lib = L
    return L


def status_string(code: int) -> str:
    return lib().snapkv_status_string(int(code)).decode()


def _check(code: int, what: str):
    if code != OK:
        raise SnapKVError(f"{what} failed: {status_string(code)}")


def _stream_ptr() -> int:
    return int(torch.cuda.current_stream().cuda_stream)


def _dev_bf16(t: torch.Tensor, name: str) -> torch.Tensor:
    if not (t.is_cuda and t.dtype == torch.bfloat16 and t.is_contiguous()):
        raise SnapKVError(f"{name} must be a contiguous CUDA bf16 tensor")
    return t


def _dev_bf16_rows(t: torch.Tensor, name: str) -> torch.Tensor:
    """A 4-D [B, Hkv, L, d] view whose rows of d elements are contiguous; the other strides are free."""
    if not (t.is_cuda and t.dtype == torch.bfloat16 and t.dim() == 4 and t.stride(3) == 1):
        raise SnapKVError(f"{name} must be a CUDA bf16 [B, Hkv, L, d] view with contiguous rows")
    return t


def _shapes(q_obs, k):
    B, Hq, W, d = q_obs.shape
    Bk, Hkv, L, dk = k.shape
    if Bk != B or dk != d:
        raise SnapKVError("q_obs and k disagree on batch or head dimension")
    return B, Hq, Hkv, L, d, W


def _alloc_ws(nbytes: int, device) -> torch.Tensor:
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)


def snapkv_out_rows(L: int, budget: int) -> int:
    return lib().snapkv_out_rows(L, budget)


def snapkv_workspace_size(B, Hq, Hkv, L, d, W, pool_kernel, pool_type, budget) -> int:
    return lib().snapkv_workspace_size(B, Hq, Hkv, L, d, W, pool_kernel, pool_type, budget)


def _lse_arg(lse_obs, B, Hq, W):
    if not (lse_obs.is_cuda and lse_obs.dtype == torch.float32 and lse_obs.is_contiguous()
            and tuple(lse_obs.shape) == (B, Hq, W)):
        raise SnapKVError("lse_obs must be a contiguous CUDA fp32 [B, Hq, W] tensor")
    return lse_obs.data_ptr()


def snapkv_compress_lse(q_obs, k, v, lse_obs, pool_kernel: int, pool_type: int, budget: int,
                        out_k=None, out_v=None, out_idx=None, workspace=None):
    """snapkv_compress with the window rows' log-sum-exp supplied (fp32 [B, Hq, W])."""
    return snapkv_compress(q_obs, k, v, pool_kernel, pool_type, budget, out_k, out_v, out_idx,
                           workspace, lse_obs=lse_obs)


def snapkv_compress_grouped(q_obs, k, v, pool_kernel: int, pool_type: int, budget: int,
                            out_k=None, out_v=None, out_idx=None, workspace=None, lse_obs=None):
    """One selection per KV head: the query heads of a group vote together and the cache keeps
    Hkv heads.  Returns (out_k, out_v [B, Hkv, rows, d], out_idx [B, Hkv, rows - W], workspace)."""
    return snapkv_compress(q_obs, k, v, pool_kernel, pool_type, budget, out_k, out_v, out_idx,
                           workspace, lse_obs=lse_obs, grouped=True)


def snapkv_compress(q_obs, k, v, pool_kernel: int, pool_type: int, budget: int,
                    out_k=None, out_v=None, out_idx=None, workspace=None, lse_obs=None,
                    grouped: bool = False):
    """Whole step on device tensors.  Returns (out_k, out_v, out_idx, workspace).

    k, v: bf16 [B, Hkv, L, d], dense or any view of that shape with contiguous rows (strides
    that are multiples of 8 elements), which goes through snapkv_compress_strided.

    out_k/out_v: bf16 [B, Hq, min(budget, L), d]; out_idx: int32 [B, Hq, rows - W].
    """
    _dev_bf16(q_obs, "q_obs"), _dev_bf16_rows(k, "k"), _dev_bf16_rows(v, "v")
    if tuple(v.shape) != tuple(k.shape):
        raise SnapKVError("k and v must have the same shape")
    strided = not (k.is_contiguous() and v.is_contiguous())
    B, Hq, Hkv, L, d, W = _shapes(q_obs, k)
    L_ = lib()
    rows = L_.snapkv_out_rows(L, budget)
    # the library addresses outputs with `budget` rows per head; on the identity path we
    # call it with budget = L so that the tensors stay dense
    eff_budget = rows
    dev = k.device
    Ho = Hkv if grouped else Hq
    if out_k is None:
        out_k = torch.empty(B, Ho, rows, d, dtype=torch.bfloat16, device=dev)
    if out_v is None:
        out_v = torch.empty(B, Ho, rows, d, dtype=torch.bfloat16, device=dev)
    if out_idx is None:
        out_idx = torch.empty(B, Ho, rows - W, dtype=torch.int32, device=dev)
    need = L_.snapkv_workspace_size(B, Hq, Hkv, L, d, W, pool_kernel, pool_type, eff_budget)
    if workspace is None or workspace.numel() < need:
        workspace = _alloc_ws(need, dev)
    tail = (B, Hq, Hkv, L, d, W, pool_kernel, pool_type, eff_budget, out_k.data_ptr(),
            out_v.data_ptr(), out_idx.data_ptr(), workspace.data_ptr(), workspace.numel(),
            _stream_ptr())
    if strided or grouped:
        # any [B, Hkv, L, d] view with contiguous rows, e.g. a permuted [B, L, Hkv, d] cache
        st = ctypes.c_int64 * 3
        fn = L_.snapkv_compress_grouped if grouped else L_.snapkv_compress_strided
        code = fn(
            q_obs.data_ptr(), k.data_ptr(), v.data_ptr(),
            st(*k.stride()[:3]) if strided else None, st(*v.stride()[:3]) if strided else None,
            None if lse_obs is None else _lse_arg(lse_obs, B, Hq, W), *tail)
    elif lse_obs is None:
        code = L_.snapkv_compress(q_obs.data_ptr(), k.data_ptr(), v.data_ptr(), *tail)
    else:
        code = L_.snapkv_compress_lse(q_obs.data_ptr(), k.data_ptr(), v.data_ptr(),
                                      _lse_arg(lse_obs, B, Hq, W), *tail)
    _check(code, "snapkv_compress")
    return out_k, out_v, out_idx, workspace


def snapkv_compress_varlen(q_obs, k, v, seq_lens, pool_kernel: int, pool_type: int, budget: int,
                           cu_seqlens=None, lse_obs=None, workspace=None):
    """Batch of prompts of different lengths.  seq_lens: list of B lengths.

    k, v: either a [B, Hkv, Lmax, d] view with contiguous rows (sequence b at positions
    [0, seq_lens[b])), or, with `cu_seqlens` (list of B starting tokens), a packed
    [total_tokens, Hkv, d] tensor.  Returns (out_k, out_v [B, Hq, budget, d] zero-filled,
    out_idx [B, Hq, budget - W] filled with -1, workspace); a sequence with budget >= its
    length fills only its first rows.
    """
    _dev_bf16(q_obs, "q_obs")
    B, Hq, W, d = q_obs.shape
    lens = [int(x) for x in seq_lens]
    st = ctypes.c_int64 * 3
    if cu_seqlens is None:
        _dev_bf16_rows(k, "k"), _dev_bf16_rows(v, "v")
        Hkv, Lmax = k.shape[1], k.shape[2]
        ks, vs, ko, vo = st(*k.stride()[:3]), st(*v.stride()[:3]), None, None
    else:
        if not (k.is_cuda and k.dtype == torch.bfloat16 and k.dim() == 3 and k.is_contiguous()
                and v.shape == k.shape and v.is_contiguous() and v.dtype == torch.bfloat16):
            raise SnapKVError("packed k and v must be contiguous CUDA bf16 [total_tokens, Hkv, d]")
        Hkv, Lmax = k.shape[1], max(lens)
        row = Hkv * d
        ks = vs = st(row * 8, d, row)       # the batch stride is not used: offsets are given
        ko = vo = (ctypes.c_int64 * B)(*[int(c) * row for c in cu_seqlens])
    L_ = lib()
    dev = k.device
    out_k = torch.zeros(B, Hq, budget, d, dtype=torch.bfloat16, device=dev)
    out_v = torch.zeros_like(out_k)
    out_idx = torch.full((B, Hq, budget - W), -1, dtype=torch.int32, device=dev)
    need = max([L_.snapkv_workspace_size(1, Hq, Hkv, x, d, W, pool_kernel, pool_type, budget)
                for x in set(lens) if x > budget] + [256])
    if workspace is None or workspace.numel() < need:
        workspace = _alloc_ws(need, dev)
    code = L_.snapkv_compress_varlen(
        q_obs.data_ptr(), k.data_ptr(), v.data_ptr(), ks, vs, ko, vo, (ctypes.c_int32 * B)(*lens),
        None if lse_obs is None else _lse_arg(lse_obs, B, Hq, W), B, Hq, Hkv, Lmax, d, W,
        pool_kernel, pool_type, budget, out_k.data_ptr(), out_v.data_ptr(), out_idx.data_ptr(),
        workspace.data_ptr(), workspace.numel(), _stream_ptr())
    _check(code, "snapkv_compress_varlen")
    return out_k, out_v, out_idx, workspace


def snapkv_compress_paged(q_obs, k_pool, v_pool, page_table, L, pool_kernel: int, pool_type: int,
                          budget: int, seq_lens=None, lse_obs=None, workspace=None):
    """The step on a paged cache.  k_pool, v_pool: bf16 CUDA views [num_pages, Hkv, page_size, d]
    with contiguous rows (any other strides, e.g. a permuted [num_pages, page_size, Hkv, d]
    pool); page_table: int32 CUDA [B, pages_per_seq]; L: prompt length (the longest one when
    seq_lens, a list of B lengths, is given).  Returns (out_k, out_v, out_idx, workspace) as
    snapkv_compress does, or, with seq_lens, as snapkv_compress_varlen does."""
    _dev_bf16(q_obs, "q_obs"), _dev_bf16_rows(k_pool, "k_pool"), _dev_bf16_rows(v_pool, "v_pool")
    if not (page_table.is_cuda and page_table.dtype == torch.int32 and page_table.is_contiguous()
            and page_table.dim() == 2 and page_table.shape[0] == q_obs.shape[0]):
        raise SnapKVError("page_table must be a contiguous CUDA int32 [B, pages_per_seq] tensor")
    if tuple(v_pool.shape) != tuple(k_pool.shape):
        raise SnapKVError("k_pool and v_pool must have the same shape")
    B, Hq, W, d = q_obs.shape
    num_pages, Hkv, page_size, dk = k_pool.shape
    if dk != d:
        raise SnapKVError("q_obs and k_pool disagree on the head dimension")
    L_ = lib()
    dev = k_pool.device
    st = ctypes.c_int64 * 3
    if seq_lens is None:
        rows = L_.snapkv_out_rows(L, budget)
        out_k = torch.empty(B, Hq, rows, d, dtype=torch.bfloat16, device=dev)
        out_v = torch.empty_like(out_k)
        out_idx = torch.empty(B, Hq, rows - W, dtype=torch.int32, device=dev)
        eff_budget, lens_arg = rows, None
        need = L_.snapkv_workspace_size(B, Hq, Hkv, L, d, W, pool_kernel, pool_type, eff_budget)
    else:
        lens = [int(x) for x in seq_lens]
        out_k = torch.zeros(B, Hq, budget, d, dtype=torch.bfloat16, device=dev)
        out_v = torch.zeros_like(out_k)
        out_idx = torch.full((B, Hq, budget - W), -1, dtype=torch.int32, device=dev)
        eff_budget, lens_arg = budget, (ctypes.c_int32 * B)(*lens)
        need = max([L_.snapkv_workspace_size(1, Hq, Hkv, x, d, W, pool_kernel, pool_type, budget)
                    for x in set(lens) if x > budget] + [256])
    if workspace is None or workspace.numel() < need:
        workspace = _alloc_ws(need, dev)
    code = L_.snapkv_compress_paged(
        q_obs.data_ptr(), k_pool.data_ptr(), v_pool.data_ptr(), st(*k_pool.stride()[:3]),
        st(*v_pool.stride()[:3]), page_table.data_ptr(), page_table.shape[1], page_size, num_pages,
        lens_arg, None if lse_obs is None else _lse_arg(lse_obs, B, Hq, W), B, Hq, Hkv, L, d, W,
        pool_kernel, pool_type, eff_budget, out_k.data_ptr(), out_v.data_ptr(), out_idx.data_ptr(),
        workspace.data_ptr(), workspace.numel(), _stream_ptr())
    _check(code, "snapkv_compress_paged")
    return out_k, out_v, out_idx, workspace


def snapkv_shard_lse(q_obs, k_shard, mask_n: int, workspace=None):
    """A shard's partial log-sum-exp of every window row: fp32 [B, Hq, W] (and the workspace)."""
    _dev_bf16(q_obs, "q_obs"), _dev_bf16(k_shard, "k_shard")
    B, Hq, Hkv, Ls, d, W = _shapes(q_obs, k_shard)
    L_ = lib()
    need = L_.snapkv_workspace_size(B, Hq, Hkv, Ls, d, W, 1, 0, W + 1)
    if workspace is None or workspace.numel() < need:
        workspace = _alloc_ws(need, k_shard.device)
    out = torch.empty(B, Hq, W, dtype=torch.float32, device=k_shard.device)
    code = L_.snapkv_shard_lse(q_obs.data_ptr(), k_shard.data_ptr(), B, Hq, Hkv, Ls, d, W, int(mask_n),
                               out.data_ptr(), workspace.data_ptr(), workspace.numel(), _stream_ptr())
    _check(code, "snapkv_shard_lse")
    return out, workspace


def snapkv_lse_merge(parts):
    """parts fp32 [R, ...] (CUDA, contiguous) -> log-sum-exp over the first axis, in its order."""
    if not (parts.is_cuda and parts.dtype == torch.float32 and parts.is_contiguous() and parts.dim() >= 2):
        raise SnapKVError("parts must be a contiguous CUDA fp32 [R, ...] tensor")
    out = torch.empty(parts.shape[1:], dtype=torch.float32, device=parts.device)
    code = lib().snapkv_lse_merge(parts.data_ptr(), parts.shape[0], out.numel(), out.data_ptr(), _stream_ptr())
    _check(code, "snapkv_lse_merge")
    return out


def snapkv_shard_votes(q_obs, k_shard, lse_obs, n_vote: int, workspace=None):
    """Votes of a shard's first n_vote keys given the merged normalisers: fp32 [B, Hq, n_vote]."""
    _dev_bf16(q_obs, "q_obs"), _dev_bf16(k_shard, "k_shard")
    B, Hq, Hkv, Ls, d, W = _shapes(q_obs, k_shard)
    L_ = lib()
    need = L_.snapkv_workspace_size(B, Hq, Hkv, Ls, d, W, 1, 0, W + 1)
    if workspace is None or workspace.numel() < need:
        workspace = _alloc_ws(need, k_shard.device)
    out = torch.empty(B, Hq, n_vote, dtype=torch.float32, device=k_shard.device)
    code = L_.snapkv_shard_votes(q_obs.data_ptr(), k_shard.data_ptr(), _lse_arg(lse_obs, B, Hq, W), B, Hq, Hkv,
                                 Ls, d, W, int(n_vote), out.data_ptr(), workspace.data_ptr(),
                                 workspace.numel(), _stream_ptr())
    _check(code, "snapkv_shard_votes")
    return out, workspace


def snapkv_gather_range(k_shard, v_shard, idx, pos0: int, append: int):
    """The shard's segment of every head's selected rows (+ `append` trailing rows of the shard).
    Returns (out_k, out_v [B, Hq, min(ksel, Ls) + append, d], seg int32 [B, Hq, 2])."""
    _dev_bf16(k_shard, "k_shard"), _dev_bf16(v_shard, "v_shard")
    if not (idx.is_cuda and idx.dtype == torch.int32 and idx.is_contiguous() and idx.dim() == 3):
        raise SnapKVError("idx must be a contiguous CUDA int32 [B, Hq, ksel] tensor")
    B, Hkv, Ls, d = k_shard.shape
    _, Hq, ksel = idx.shape
    rows = min(ksel, Ls) + append
    # rows behind a head's segment (and its appended rows) are left as allocated
    out_k = torch.empty(B, Hq, rows, d, dtype=torch.bfloat16, device=k_shard.device)
    out_v = torch.empty_like(out_k)
    seg = torch.empty(B, Hq, 2, dtype=torch.int32, device=k_shard.device)
    code = lib().snapkv_gather_range(k_shard.data_ptr(), v_shard.data_ptr(), idx.data_ptr(), B, Hq, Hkv, Ls, d,
                                     int(pos0), ksel, int(append), out_k.data_ptr(), out_v.data_ptr(), rows,
                                     seg.data_ptr(), _stream_ptr())
    _check(code, "snapkv_gather_range")
    return out_k, out_v, seg


def snapkv_hit_counts(a_cur, idx, theta: float):
    """a_cur fp32 [rows, n], idx int32 [rows, k] (CUDA) -> int32 [rows, 2]: per head the selected
    positions above theta and all positions above theta (Eq. 3-7; H = ratio of the column sums)."""
    if not (a_cur.is_cuda and a_cur.dtype == torch.float32 and a_cur.is_contiguous() and a_cur.dim() == 2):
        raise SnapKVError("a_cur must be a contiguous CUDA fp32 [rows, n] tensor")
    if not (idx.is_cuda and idx.dtype == torch.int32 and idx.is_contiguous() and idx.dim() == 2
            and idx.shape[0] == a_cur.shape[0]):
        raise SnapKVError("idx must be a contiguous CUDA int32 [rows, k] tensor")
    out = torch.empty(a_cur.shape[0], 2, dtype=torch.int32, device=a_cur.device)
    code = lib().snapkv_hit_counts(a_cur.data_ptr(), idx.data_ptr(), a_cur.shape[0], a_cur.shape[1],
                                   idx.shape[1], float(theta), out.data_ptr(), _stream_ptr())
    _check(code, "snapkv_hit_counts")
    return out


def snapkv_decode_attention(q_cur, cache_k, cache_v, workspace=None, want_lse: bool = True):
    """q_cur bf16 [B, Hq, d], cache_k/v bf16 [B, Hc, rows, d] (CUDA, contiguous) ->
    (out fp32 [B, Hq, d], lse fp32 [B, Hq] or None, workspace)."""
    _dev_bf16(q_cur, "q_cur"), _dev_bf16(cache_k, "cache_k"), _dev_bf16(cache_v, "cache_v")
    B, Hq, d = q_cur.shape
    Bc, Hc, rows, dc = cache_k.shape
    if Bc != B or dc != d or tuple(cache_v.shape) != tuple(cache_k.shape):
        raise SnapKVError("q_cur, cache_k and cache_v disagree on their shapes")
    L_ = lib()
    need = L_.snapkv_decode_workspace_size(B, Hq, rows, d)
    if workspace is None or workspace.numel() < need:
        workspace = _alloc_ws(need, q_cur.device)
    out = torch.empty(B, Hq, d, dtype=torch.float32, device=q_cur.device)
    lse = torch.empty(B, Hq, dtype=torch.float32, device=q_cur.device) if want_lse else None
    code = L_.snapkv_decode_attention(q_cur.data_ptr(), cache_k.data_ptr(), cache_v.data_ptr(), B, Hq, Hc,
                                      rows, d, out.data_ptr(), lse.data_ptr() if want_lse else None,
                                      workspace.data_ptr(), workspace.numel(), _stream_ptr())
    _check(code, "snapkv_decode_attention")
    return out, lse, workspace


def snapkv_window_scores_lse(q_obs, k, lse_obs, out_vote=None, workspace=None):
    """snapkv_window_scores with the window rows' log-sum-exp supplied (fp32 [B, Hq, W])."""
    return snapkv_window_scores(q_obs, k, out_vote, workspace, lse_obs=lse_obs)


def snapkv_window_scores(q_obs, k, out_vote=None, workspace=None, lse_obs=None):
    """Votes fp32 [B, Hq, n].  Returns (out_vote, workspace)."""
    _dev_bf16(q_obs, "q_obs"), _dev_bf16(k, "k")
    B, Hq, Hkv, L, d, W = _shapes(q_obs, k)
    L_ = lib()
    dev = k.device
    if out_vote is None:
        out_vote = torch.empty(B, Hq, L - W, dtype=torch.float32, device=dev)
    need = L_.snapkv_workspace_size(B, Hq, Hkv, L, d, W, 1, 0, W + 1)
    if workspace is None or workspace.numel() < need:
        workspace = _alloc_ws(need, dev)
    tail = (B, Hq, Hkv, L, d, W, out_vote.data_ptr(), workspace.data_ptr(), workspace.numel(),
            _stream_ptr())
    if lse_obs is None:
        code = L_.snapkv_window_scores(q_obs.data_ptr(), k.data_ptr(), *tail)
    else:
        code = L_.snapkv_window_scores_lse(q_obs.data_ptr(), k.data_ptr(),
                                           _lse_arg(lse_obs, B, Hq, W), *tail)
    _check(code, "snapkv_window_scores")
    return out_vote, workspace


def snapkv_schedule_items(B, Hq, Hkv, L, d, W, grid, cta, votes_only=False):
    """The scoring kernel's work items for block `cta` of `grid` (host only).  Returns
    (items, plan): items is a list of (unit, t0, t1, vote, slot, nseg); plan a dict."""
    L_ = lib()
    plan = (ctypes.c_int32 * 8)()
    n = L_.snapkv_schedule_items(B, Hq, Hkv, L, d, W, int(votes_only), grid, cta, None, 0, plan)
    if n < 0:
        raise SnapKVError("snapkv_schedule_items: arguments not acceptable")
    buf = (ctypes.c_int32 * (6 * max(n, 1)))()
    L_.snapkv_schedule_items(B, Hq, Hkv, L, d, W, int(votes_only), grid, cta, buf, n, plan)
    items = [tuple(buf[6 * i:6 * i + 6]) for i in range(n)]
    names = ("units", "units_per_wave", "waves", "tiles_stats", "tiles_vote", "maxseg", "lag", "ncols")
    return items, dict(zip(names, plan))


def snapkv_set_wait_limit_ns(limit_ns: int) -> int:
    """Sets the time limit of device-side waits; returns the previous one."""
    return int(lib().snapkv_set_wait_limit_ns(int(limit_ns)))


def snapkv_selftest_stalled_scores(q_obs, k, out_vote=None, workspace=None):
    """Launches the vote sweep with statistics that never arrive (time-out self-test).
    Returns (out_vote, workspace); read the outcome with snapkv_device_status."""
    _dev_bf16(q_obs, "q_obs"), _dev_bf16(k, "k")
    B, Hq, Hkv, L, d, W = _shapes(q_obs, k)
    L_ = lib()
    if out_vote is None:
        out_vote = torch.empty(B, Hq, L - W, dtype=torch.float32, device=k.device)
    need = L_.snapkv_workspace_size(B, Hq, Hkv, L, d, W, 1, 0, W + 1)
    if workspace is None or workspace.numel() < need:
        workspace = _alloc_ws(need, k.device)
    code = L_.snapkv_selftest_stalled_scores(q_obs.data_ptr(), k.data_ptr(), B, Hq, Hkv, L, d, W,
                                             out_vote.data_ptr(), workspace.data_ptr(),
                                             workspace.numel(), _stream_ptr())
    _check(code, "snapkv_selftest_stalled_scores")
    return out_vote, workspace


def snapkv_pool_topk(vote, pool_kernel: int, pool_type: int, ksel: int, out_idx=None,
                     workspace=None):
    """vote fp32 [rows, n] (CUDA) -> int32 [rows, ksel] ascending positions."""
    if not (vote.is_cuda and vote.dtype == torch.float32 and vote.is_contiguous() and vote.dim() == 2):
        raise SnapKVError("vote must be a contiguous CUDA fp32 [rows, n] tensor")
    rows, n = vote.shape
    L_ = lib()
    if out_idx is None:
        out_idx = torch.empty(rows, max(ksel, 0), dtype=torch.int32, device=vote.device)
    elif not (out_idx.is_cuda and out_idx.dtype == torch.int32 and out_idx.is_contiguous()
              and tuple(out_idx.shape) == (rows, ksel)):
        raise SnapKVError("out_idx must be a contiguous CUDA int32 [rows, ksel] tensor")
    need = L_.snapkv_pool_topk_workspace_size(rows, n)
    if need and (workspace is None or workspace.numel() < need):
        workspace = _alloc_ws(need, vote.device)
    code = L_.snapkv_pool_topk(vote.data_ptr(), rows, n, pool_kernel, pool_type, ksel,
                               out_idx.data_ptr(), workspace.data_ptr() if workspace is not None else None,
                               workspace.numel() if workspace is not None else 0, _stream_ptr())
    _check(code, "snapkv_pool_topk")
    return out_idx


STATIC_MAX_KEYS = 4 * 1024 * 1024


def snapkv_pool_topk_static(vote, pool_kernel: int, pool_type: int, ksel: int, out_idx):
    """snapkv_pool_topk for callers that cannot allocate: the scratch is an array built
    into the library (rows * n <= STATIC_MAX_KEYS).  `out_idx` (int32 [rows, ksel], CUDA)
    must be passed in; this wrapper allocates nothing either."""
    if not (vote.is_cuda and vote.dtype == torch.float32 and vote.is_contiguous() and vote.dim() == 2):
        raise SnapKVError("vote must be a contiguous CUDA fp32 [rows, n] tensor")
    rows, n = vote.shape
    if not (torch.is_tensor(out_idx) and out_idx.is_cuda and out_idx.dtype == torch.int32
            and out_idx.is_contiguous() and tuple(out_idx.shape) == (rows, ksel)
            and out_idx.device == vote.device):
        raise SnapKVError("out_idx must be a contiguous CUDA int32 [rows, ksel] tensor on vote's device")
    code = lib().snapkv_pool_topk_static(vote.data_ptr(), rows, n, pool_kernel, pool_type, ksel,
                                         out_idx.data_ptr(), _stream_ptr())
    _check(code, "snapkv_pool_topk_static")
    return out_idx


def snapkv_gather(k, v, idx, W: int):
    """k, v bf16 [B,Hkv,L,d]; idx int32 [B,Hq,ksel] -> out_k, out_v [B,Hq,ksel+W,d]."""
    _dev_bf16(k, "k"), _dev_bf16(v, "v")
    if not (idx.is_cuda and idx.dtype == torch.int32 and idx.is_contiguous()):
        raise SnapKVError("idx must be a contiguous CUDA int32 tensor")
    B, Hkv, L, d = k.shape
    _, Hq, ksel = idx.shape
    out_k = torch.empty(B, Hq, ksel + W, d, dtype=torch.bfloat16, device=k.device)
    out_v = torch.empty_like(out_k)
    code = lib().snapkv_gather(k.data_ptr(), v.data_ptr(), idx.data_ptr(), B, Hq, Hkv, L, d, W, ksel,
                               out_k.data_ptr(), out_v.data_ptr(), _stream_ptr())
    _check(code, "snapkv_gather")
    return out_k, out_v


def snapkv_host_staging_size(B, Hq, Hkv, L, d, W, pool_kernel, pool_type, budget) -> int:
    return lib().snapkv_host_staging_size(B, Hq, Hkv, L, d, W, pool_kernel, pool_type, budget)


def snapkv_compress_host(q_obs, k, v, pool_kernel, pool_type, budget, out_k, out_v, out_idx,
                         staging):
    """Host (ideally pinned) tensors in and out; `staging` is a CUDA uint8 tensor.
    Enqueues copies and kernels on the current stream and returns without synchronising."""
    for t, name in ((q_obs, "q_obs"), (k, "k"), (v, "v"), (out_k, "out_k"), (out_v, "out_v"),
                    (out_idx, "out_idx")):
        if t.is_cuda or not t.is_contiguous():
            raise SnapKVError(f"{name} must be a contiguous host tensor")
    B, Hq, Hkv, L, d, W = _shapes(q_obs, k)
    code = lib().snapkv_compress_host(q_obs.data_ptr(), k.data_ptr(), v.data_ptr(), B, Hq, Hkv, L, d,
                                      W, pool_kernel, pool_type, budget, out_k.data_ptr(),
                                      out_v.data_ptr(), out_idx.data_ptr(), staging.data_ptr(),
                                      staging.numel(), _stream_ptr())
    _check(code, "snapkv_compress_host")


def snapkv_device_status(workspace):
    """Synchronises the current stream; returns (status, detail)."""
    detail = ctypes.c_int(0)
    code = lib().snapkv_device_status(workspace.data_ptr(), _stream_ptr(), ctypes.byref(detail))
    return code, detail.value


def snapkv_last_launch_count() -> int:
    return lib().snapkv_last_launch_count()
