"""Seeded synthetic Q/K/V for the SnapKV compression step.

This module only draws numbers.  It contains none of the method's arithmetic and
is the one piece of code that both the CUDA tests/benchmark and the CPU oracle
tests feed from (each side receives the same bits).

The tensors stand in for the post-RoPE prompt queries, keys and values of the
7B-class long-context models the paper evaluates (Sec. 5: LWM-Text-Chat-1M,
LongChat-7B, Mistral-7B, Mixtral-8x7B) on its long-context workloads; the real
activations need trained weights and the benchmark texts, neither of which is
used here.  Shapes, window/kernels and budgets follow Sec. 5.1-5.3.

Recipe (per sequence b of a layer, all draws fp32 then rounded to bf16):
  * seed = 1000*workload_id + layer + 100000*b (a torch Generator on the target
    device; the stream of a CPU and of a CUDA generator differ, so a given
    (workload, layer, device kind) is reproducible, and both sides of a parity
    test always read the very same tensor);
  * K, V ~ N(0, 1); with `key_norm_sigma` each key position is scaled by
    exp(sigma * z_j), z_j ~ N(0, 1) shared by all heads (heavy-tailed norms);
  * one unit direction u_c per KV head; with GQA query head h uses
    normalize(u_c + 0.5 * r_h), r_h a random unit vector, so the heads of a
    group agree on the planted clusters and differ at the margin;
  * `clusters` runs of 8 contiguous prefix keys get 3*u_c added (planted
    important spans: the synthetic stand-in for the spans the paper's models
    attend to); starts are drawn on a CPU generator so they do not depend on the
    device; `edge_clusters` forces one run at position 0 and one ending at n-1;
  * window queries q_i = 4*u_h + 0.3*N(0, I).
"""
from __future__ import annotations

from dataclasses import dataclass

import torch

CLUSTER_LEN = 8


@dataclass(frozen=True)
class Workload:
    wid: int
    name: str
    B: int
    Hq: int
    Hkv: int
    d: int
    L: int
    W: int
    pool_kernel: int
    pool_type: str          # "max" | "avg"
    budgets: tuple
    layers: int
    clusters: int
    key_norm_sigma: float = 0.0
    edge_clusters: bool = False

    @property
    def n(self) -> int:
        return self.L - self.W

    @property
    def group(self) -> int:
        return self.Hq // self.Hkv


def _nclusters(L, W, frac=0.01):
    return int(round(frac * (L - W) / CLUSTER_LEN))


WORKLOADS = {
    0: Workload(0, "tiny-mha-1k", 1, 4, 4, 64, 1024, 32, 7, "max", (256,), 1, 3),
    1: Workload(1, "lwm7b-mha-16k", 1, 32, 32, 128, 16384, 32, 7, "max", (1024, 2048, 4096), 32,
                _nclusters(16384, 32)),
    2: Workload(2, "mistral7b-gqa-32k", 4, 32, 8, 128, 32768, 32, 5, "avg", (4096,), 32,
                _nclusters(32768, 32)),
    3: Workload(3, "mixtral-gqa-128k", 1, 32, 8, 128, 131072, 64, 7, "max", (2048, 8192), 32, 16,
                key_norm_sigma=0.5, edge_clusters=True),
    4: Workload(4, "mha-380k-needle", 1, 32, 32, 128, 380000, 32, 7, "max", (4096,), 1, 1),
}


def cluster_starts(w: Workload, layer: int, b: int) -> torch.Tensor:
    """Start positions (int64, ascending) of the planted runs of one sequence."""
    gen = torch.Generator(device="cpu")
    gen.manual_seed(7919 + 1000 * w.wid + layer + 100000 * b)
    slots = w.n // CLUSTER_LEN
    if w.edge_clusters:
        inner = w.clusters - 2
        pick = torch.randperm(slots - 3, generator=gen)[:inner] + 1
        starts = torch.cat([pick * CLUSTER_LEN, torch.tensor([0, w.n - CLUSTER_LEN])])
    else:
        pick = torch.randperm(slots, generator=gen)[: w.clusters]
        starts = pick * CLUSTER_LEN
    return torch.sort(starts).values


def _unit(x: torch.Tensor) -> torch.Tensor:
    return x / x.norm(dim=-1, keepdim=True)


def make_layer(w: Workload, layer: int = 0, device: str = "cpu", want_v: bool = True):
    """Draw one layer's inputs.

    Returns {"q_obs": bf16 [B,Hq,W,d], "k": bf16 [B,Hkv,L,d], "v": bf16 [B,Hkv,L,d],
    "starts": list of B int64 tensors with the planted run starts}.
    """
    dev = torch.device(device)
    q_obs = torch.empty(w.B, w.Hq, w.W, w.d, dtype=torch.bfloat16, device=dev)
    k = torch.empty(w.B, w.Hkv, w.L, w.d, dtype=torch.bfloat16, device=dev)
    v = torch.empty(w.B, w.Hkv, w.L, w.d, dtype=torch.bfloat16, device=dev) if want_v else None
    starts_all = []
    g = w.group
    for b in range(w.B):
        gen = torch.Generator(device=dev)
        gen.manual_seed(1000 * w.wid + layer + 100000 * b)
        u_c = _unit(torch.randn(w.Hkv, w.d, generator=gen, device=dev))
        if g > 1:
            r_h = _unit(torch.randn(w.Hq, w.d, generator=gen, device=dev))
            u_h = _unit(u_c.repeat_interleave(g, dim=0) + 0.5 * r_h)
        else:
            u_h = u_c
        qf = 4.0 * u_h[:, None, :] + 0.3 * torch.randn(w.Hq, w.W, w.d, generator=gen, device=dev)
        q_obs[b] = qf.to(torch.bfloat16)
        scale = None
        if w.key_norm_sigma > 0.0:
            z = torch.randn(w.L, generator=gen, device=dev)
            scale = torch.exp(w.key_norm_sigma * z)[:, None]
        starts = cluster_starts(w, layer, b)
        starts_all.append(starts)
        pos = (starts[:, None] + torch.arange(CLUSTER_LEN)[None, :]).reshape(-1).to(dev)
        for c in range(w.Hkv):  # one KV head at a time keeps the fp32 staging small
            kf = torch.randn(w.L, w.d, generator=gen, device=dev)
            if scale is not None:
                kf *= scale
            kf[pos] += 3.0 * u_c[c]
            k[b, c] = kf.to(torch.bfloat16)
            if want_v:
                v[b, c] = torch.randn(w.L, w.d, generator=gen, device=dev).to(torch.bfloat16)
    return {"q_obs": q_obs, "k": k, "v": v, "starts": starts_all}


def make_random(B, Hq, Hkv, L, d, W, seed=0, device="cpu", q_scale=1.0):
    """Unstructured N(0,1) inputs of an arbitrary shape (edge-case tests)."""
    dev = torch.device(device)
    gen = torch.Generator(device=dev)
    gen.manual_seed(seed)
    q_obs = (q_scale * torch.randn(B, Hq, W, d, generator=gen, device=dev)).to(torch.bfloat16)
    k = torch.randn(B, Hkv, L, d, generator=gen, device=dev).to(torch.bfloat16)
    v = torch.randn(B, Hkv, L, d, generator=gen, device=dev).to(torch.bfloat16)
    return {"q_obs": q_obs, "k": k, "v": v}


def bf16_bits(t: torch.Tensor):
    """bf16 tensor -> numpy uint16 bit patterns on the host (no arithmetic)."""
    import numpy as np

    return t.detach().contiguous().cpu().view(torch.int16).numpy().view(np.uint16)
