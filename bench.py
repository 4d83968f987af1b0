"""Benchmark of the SnapKV prompt KV-cache compression step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--workload ID] [--budget B] [--layers NL]

One step = the whole compression path (score, vote, pool, top-k, gather) over every
layer of the workload, each layer with its own seeded synthetic Q/K/V resident in HBM
(distinct buffers per layer, far larger than L2, so no layer is timed on cached data).
Prints one JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

# dram__bytes_read.sum + dram__bytes_write.sum per launch from the committed ncu summaries
# (profiles/): (stage, workload id) -> (bytes, source file of the kernel, first 12 hex digits of
# that file's SHA-256 when the counters were taken).  A figure is reported only while the
# kernel's source is unchanged; after any edit it reads null until the capture is redone.
NCU_TRAFFIC = {
    ("score", 2): (477.26e6, "snapkv_score.cu", "389ce5121ee8"),
    ("score-lse", 2): (276.65e6, "snapkv_score.cu", "389ce5121ee8"),
    ("gather", 2): (339.06e6, "snapkv_gather.cu", "6ef533532da0"),
}


def ncu_traffic(stage, wid):
    import hashlib
    ent = NCU_TRAFFIC.get((stage, wid))
    if ent is None:
        return None
    nbytes, src, digest = ent
    path = os.path.join(ROOT, "paper_2404_14469_b200", "csrc", src)
    try:
        with open(path, "rb") as f:
            now = hashlib.sha256(f.read()).hexdigest()[:12]
    except OSError:
        return None
    return nbytes if now == digest else None

METRIC = "prompt_tokens_compressed_per_s"
UNIT = "prompt tokens/s"


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            with open(path) as f:
                p = json.load(f)
            return float(p["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


def algorithmic_bytes(w, budget, heads_out=None):
    """Per layer: K read once + Q_obs + selected K/V rows read + compressed K/V written +
    out_idx written (fp32 vote scratch traffic is extra and not counted).  `heads_out`: heads of
    the compressed cache (Hq, or Hkv with one selection per KV head)."""
    rows = min(budget, w.L)
    ksel = rows - w.W
    ho = heads_out or w.Hq
    k_read = w.B * w.Hkv * w.L * w.d * 2
    q_read = w.B * w.Hq * w.W * w.d * 2
    sel = 2 * w.B * ho * rows * w.d * 2
    idx = w.B * ho * ksel * 4
    return {"score": k_read + q_read, "gather": 2 * sel + idx, "total": k_read + q_read + 2 * sel + idx}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            pass
        sm, smax, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0]))
                smax = float(parts[1])
            except ValueError:
                continue
            for name, val in zip(names, parts[2:6]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": smax,
                "reasons": sorted(reasons), "samples": len(sm)}


# ------------------------------------------------------------------ reference arm (CPU oracle)
def oracle_sample(w, budget, seconds_hint=15.0):
    """Time the CPU oracle, as it stands, on a bounded sample of one layer of the workload:
    whole (batch, KV-head) groups until about `seconds_hint` seconds are spent.  Returns
    (tokens_per_s extrapolated to the full layer stack, cores, description)."""
    from oracle import snapkv_oracle as orc
    from paper_2404_14469_b200 import synth

    cores = len(os.sched_getaffinity(0))
    one = synth.Workload(w.wid, w.name, 1, w.Hq, w.Hkv, w.d, w.L, w.W, w.pool_kernel, w.pool_type,
                         w.budgets, 1, w.clusters, w.key_norm_sigma, w.edge_clusters)
    ptype = orc.POOL_MAX if w.pool_type == "max" else orc.POOL_AVG
    g = w.Hq // w.Hkv
    done_heads, t_total, seq = 0, 0.0, 0
    # one sequence of one layer at a time, drawn on the host, until the time hint is used up
    while t_total < seconds_hint and seq < 64:
        data = synth.make_layer(one, seq)
        q, k, v = (synth.bf16_bits(data[x]) for x in ("q_obs", "k", "v"))
        c = 0
        while c < w.Hkv and (t_total < seconds_hint or done_heads == 0):
            take = min(max(1, cores // g), w.Hkv - c)
            heads = [(0, h) for h in range(c * g, (c + take) * g)]
            t0 = time.perf_counter()
            orc.compress(q, k, v, w.pool_kernel, ptype, budget, workers=cores, heads=heads)
            t_total += time.perf_counter() - t0
            done_heads += len(heads)
            c += take
        seq += 1
    t_layer = t_total / done_heads * (w.B * w.Hq)
    tokens_per_s = w.B * w.L / (t_layer * w.layers)
    desc = (f"{done_heads} (batch, head) rows of {w.name} ({w.B * w.Hq} per layer), "
            f"{t_total:.1f} s of oracle time, extrapolated to {w.layers} layers")
    return tokens_per_s, cores, desc, t_total


def run_reference(args, w, budget, rank, world):
    if rank != 0:
        return
    vals, times = [], []
    desc, cores = "", 0
    for _ in range(args.warmup + args.steps):
        tps, cores, desc, t_sample = oracle_sample(w, budget, seconds_hint=8.0)
        vals.append(tps)
        times.append(t_sample)
    vals = vals[args.warmup:] or vals
    times = times[args.warmup:] or times
    value = sum(vals) / len(vals)
    # a step of this arm is a bounded sample of the workload: ms_per_step is the time one such
    # sample really took; what the whole 32-layer step would take is given separately
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": sum(times) / len(times) * 1e3,
        "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(w, budget, args.layers or w.layers),
        "extrapolated": {"ms_per_full_step": w.B * w.L / value * 1e3,
                         "note": "value and ms_per_full_step scale the sampled (batch, head) rows "
                                 "to the whole layer stack; ms_per_step is the sample itself"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def workload_config(w, budget, layers):
    return {"workload": w.name, "B": w.B, "Hq": w.Hq, "Hkv": w.Hkv, "d": w.d, "L": w.L, "W": w.W,
            "pool": f"{w.pool_type}{w.pool_kernel}", "budget": budget, "layers": layers,
            "l2": "every layer has its own buffers (inputs per step far larger than L2)"}


def launch_ranks(n, argv):
    """`python bench.py --gpus N` outside a launcher: run N ranks of this script through
    torch.distributed.run on 127.0.0.1 (one process per GPU) and pass their exit code on."""
    import socket

    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + list(argv)
    return subprocess.call(cmd)


# ------------------------------------------------------------------ our arm
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=60)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", type=int, default=2)
    ap.add_argument("--budget", type=int, default=0)
    ap.add_argument("--layers", type=int, default=0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--lse-in", action="store_true",
                    help="time the supplied-normaliser variant (snapkv_compress_lse): the window "
                         "rows' log-sum-exp is an input, K is swept once; not the paper's path")
    ap.add_argument("--grouped", action="store_true",
                    help="time the shared-selection variant (snapkv_compress_grouped): one "
                         "selection per KV head, the compressed cache keeps Hkv heads")
    args = ap.parse_args()

    if args.gpus > 1 and "RANK" not in os.environ:
        # not under a launcher: start one rank per GPU ourselves, the way the launcher would
        sys.exit(launch_ranks(args.gpus, sys.argv[1:]))

    from paper_2404_14469_b200 import synth

    w = synth.WORKLOADS[args.workload]
    budget = args.budget or w.budgets[-1]
    if args.impl == "reference":
        # the CPU oracle runs on rank 0 alone; the other ranks have nothing to do
        run_reference(args, w, budget, int(os.environ.get("RANK", "0")),
                      int(os.environ.get("WORLD_SIZE", "1")))
        return
    from paper_2404_14469_b200 import replicas

    rank, world, local = replicas.init()
    barrier = replicas.barrier

    def max_over_ranks(x, world_):
        return replicas.max_over_ranks(x, world_, device="cuda")

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the compression path has no CPU fallback")
    from paper_2404_14469_b200 import binding as sk
    from paper_2404_14469_b200 import build as sk_build

    if rank == 0:
        sk_build.build()
    barrier(world)
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    layers = args.layers or w.layers
    ptype = sk.POOL_MAX if w.pool_type == "max" else sk.POOL_AVG
    ksel = budget - w.W

    # resident inputs and outputs, one set per layer (seeds differ per rank: weak scaling,
    # every rank compresses its own batch of sequences)
    ins = []
    for layer in range(layers):
        d = synth.make_layer(w, layer + replicas.layer_seed_offset(rank), device=str(dev))
        ins.append((d["q_obs"], d["k"], d["v"]))
    ho = w.Hkv if args.grouped else w.Hq
    out_k = [torch.empty(w.B, ho, budget, w.d, dtype=torch.bfloat16, device=dev) for _ in range(layers)]
    out_v = [torch.empty_like(t) for t in out_k]
    out_idx = [torch.empty(w.B, ho, ksel, dtype=torch.int32, device=dev) for _ in range(layers)]
    ws = torch.empty(sk.snapkv_workspace_size(w.B, w.Hq, w.Hkv, w.L, w.d, w.W, w.pool_kernel, ptype, budget),
                     dtype=torch.uint8, device=dev)
    vote = torch.empty(w.B * w.Hq, w.n, dtype=torch.float32, device=dev)
    lses = [None] * layers
    if args.lse_in:
        # Input preparation for the variant, untimed: what the prompt phase's attention kernel
        # would hand over.  Plain framework ops on the synthetic q and k; the library's own
        # results with these inputs are checked against the oracle in tests/test_gpu_lse.py.
        g = w.Hq // w.Hkv
        pos = torch.arange(w.L, device=dev)[None, :] <= (w.n + torch.arange(w.W, device=dev))[:, None]
        for i, (q, k, _) in enumerate(ins):
            rows = []
            for b in range(w.B):
                kk = k[b].float().repeat_interleave(g, dim=0)                      # [Hq, L, d]
                lg = torch.matmul(q[b].float(), kk.transpose(1, 2)) / (w.d ** 0.5)   # [Hq, W, L]
                rows.append(torch.logsumexp(lg.masked_fill(~pos, float("-inf")), dim=-1))
            lses[i] = torch.stack(rows).contiguous()

    def step():
        for i in range(layers):
            q, k, v = ins[i]
            sk.snapkv_compress(q, k, v, w.pool_kernel, ptype, budget, out_k[i], out_v[i], out_idx[i], ws,
                               lse_obs=lses[i], grouped=args.grouped)

    for _ in range(max(args.warmup, 3)):
        step()
    launches_per_layer = sk.snapkv_last_launch_count()
    torch.cuda.synchronize()
    barrier(world)

    # nvidia-smi numbers the GPUs of the machine, CUDA those this process may see: go by UUID
    try:
        smi_id = "GPU-" + str(torch.cuda.get_device_properties(local).uuid)
    except Exception:
        smi_id = str(local)
    sampler = ClockSampler(smi_id)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    barrier(world)
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    torch.cuda.synchronize()
    barrier(world)
    ms_total = max_over_ranks(e0.elapsed_time(e1), world)
    code, detail = sk.snapkv_device_status(ws)
    if code != sk.OK:
        raise SystemExit(f"device status {sk.status_string(code)} (detail {detail})")

    # per-stage timing through the staged entry points, same buffers, same stream: one event
    # pair per stage per layer (the events sit on the launching stream)
    stage_ms = {"score": 0.0, "select": 0.0, "gather": 0.0}
    reps = max(1, min(args.steps, 3))
    lib = sk.lib()
    for _ in range(reps):
        # all layers are enqueued before the one synchronisation, so that the device runs
        # them back to back and an interval never contains host launch time
        evs = []
        for i in range(layers):
            q, k, v = ins[i]
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
            evs.append(ev)
            ev[0].record()
            sk.snapkv_window_scores(q, k, vote.view(w.B, w.Hq, w.n), ws, lse_obs=lses[i])
            ev[1].record()
            # (the staged select has no group sum: with --grouped only the gather stage, on the
            # indices the fused call left, and the scoring stage are timed separately)
            if not args.grouped:
                sk.snapkv_pool_topk(vote, w.pool_kernel, ptype, ksel, out_idx[i].view(w.B * w.Hq, ksel), ws)
            ev[2].record()
            lib.snapkv_gather(k.data_ptr(), v.data_ptr(), out_idx[i].data_ptr(), w.B, ho, w.Hkv, w.L,
                              w.d, w.W, ksel, out_k[i].data_ptr(), out_v[i].data_ptr(),
                              int(torch.cuda.current_stream().cuda_stream))
            ev[3].record()
        torch.cuda.synchronize()
        for ev in evs[1:] if layers > 1 else evs:  # the first layer starts on an idle device
            stage_ms["score"] += ev[0].elapsed_time(ev[1])
            stage_ms["select"] += ev[1].elapsed_time(ev[2])
            stage_ms["gather"] += ev[2].elapsed_time(ev[3])
    for kname in stage_ms:
        stage_ms[kname] /= reps * (layers - 1 if layers > 1 else 1)
    # The scoring stage once more, on its own: every layer's scoring call back to back
    # between ONE pair of events, so that no event sits between the launches of a call (the
    # scoring kernel is made resident while the clear kernel before it still runs, which an
    # event in between prevents).  Each layer has its own K: nothing is served from L2.
    e2, e3 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sk.snapkv_window_scores(ins[0][0], ins[0][1], vote.view(w.B, w.Hq, w.n), ws, lse_obs=lses[0])
    e2.record()
    for _ in range(reps):
        for i in range(layers):
            sk.snapkv_window_scores(ins[i][0], ins[i][1], vote.view(w.B, w.Hq, w.n), ws, lse_obs=lses[i])
    e3.record()
    torch.cuda.synchronize()
    stage_ms["score_with_events"] = stage_ms["score"]
    stage_ms["score"] = e2.elapsed_time(e3) / (reps * layers)
    clocks = sampler.stop() if rank == 0 else None

    ms_step = ms_total / args.steps
    ms_layer = ms_step / layers
    tokens = w.B * w.L * world
    value = tokens / (ms_step * 1e-3)
    ab = algorithmic_bytes(w, budget, ho)
    if args.grouped:
        stage_ms["select"] = None
    peak, peak_kind = load_peaks()

    # roofline of the dominant stage; the gather is one launch per layer, the scoring is a
    # pair of launches (statistics pass, vote pass) per wave of units
    dom = max(("score", "gather"), key=lambda s: stage_ms[s])
    dom_bytes = ab[dom]
    achieved = dom_bytes / (stage_ms[dom] * 1e-3) / 1e9
    roofline = {
        "bound": "hbm", "kernel": {"score": "score_kernel (vote pass only)" if args.lse_in
                                    else "score_kernel (statistics + vote passes)",
                                    "gather": "gather_kernel"}[dom],
        "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
        "peak_kind": f"of {peak_kind}",
        "traffic": ncu_traffic("score-lse" if args.lse_in and dom == "score" else dom, w.wid),
        "algorithmic_bytes_per_launch": dom_bytes, "ms_per_launch": stage_ms[dom],
        "stage_ms_per_layer": stage_ms,
        "whole_step": {"algorithmic_bytes_per_layer": ab["total"], "ms_per_layer": ms_layer,
                       "achieved": ab["total"] / (ms_layer * 1e-3) / 1e9,
                       "frac_of_peak": ab["total"] / (ms_layer * 1e-3) / 1e9 / peak,
                       "frac_of_8TBps": ab["total"] / (ms_layer * 1e-3) / 8.0e12},
    }

    # end to end through the host-buffer entry point: pinned host tensors in, pinned out
    e2e = None
    if not args.no_e2e and not args.lse_in and not args.grouped:
        q, k, v = (t.cpu().pin_memory() for t in ins[0])
        hk = torch.empty(w.B, w.Hq, budget, w.d, dtype=torch.bfloat16).pin_memory()
        hv = torch.empty_like(hk).pin_memory()
        hi = torch.empty(w.B, w.Hq, ksel, dtype=torch.int32).pin_memory()
        staging = torch.empty(sk.snapkv_host_staging_size(w.B, w.Hq, w.Hkv, w.L, w.d, w.W, w.pool_kernel,
                                                          ptype, budget), dtype=torch.uint8, device=dev)
        e2e_layers = layers

        def e2e_step():
            for _ in range(e2e_layers):
                sk.snapkv_compress_host(q, k, v, w.pool_kernel, ptype, budget, hk, hv, hi, staging)

        e2e_step()
        torch.cuda.synchronize()
        barrier(world)
        e2e_steps = max(1, min(args.steps, 2))
        a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a0.record()
        for _ in range(e2e_steps):
            e2e_step()
        a1.record()
        torch.cuda.synchronize()
        barrier(world)
        e2e_ms = max_over_ranks(a0.elapsed_time(a1), world) / e2e_steps
        h2d = (q.numel() + k.numel() + v.numel()) * 2 * e2e_layers
        d2h = (hk.numel() + hv.numel()) * 2 * e2e_layers + hi.numel() * 4 * e2e_layers
        e2e = {"value": tokens / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms, "steps": e2e_steps,
               "api": "snapkv_compress_host (pinned host buffers)"}

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        tps, cores, desc, _ = oracle_sample(w, budget, seconds_hint=12.0)
        cpu_baseline = {"value": tps, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc}

    if rank == 0:
        cfg = workload_config(w, budget, layers)
        if args.lse_in:
            cfg["variant"] = ("lse-in: the window rows' log-sum-exp is an input, one sweep over K "
                              "(snapkv_compress_lse; not the paper's path)")
        if args.grouped:
            cfg["variant"] = (cfg.get("variant", "") + " grouped: one selection per KV head from the "
                              "group's summed votes, cache of Hkv heads (snapkv_compress_grouped; "
                              "not the paper's path)").strip()
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "dtype_note": "bf16 operands on the tensor cores, fp32 accumulation, softmax and votes",
            "ms_per_layer": ms_layer,
            "parallelism": "replicas: each GPU compresses its own batch, no collective",
            "config": cfg, "clocks": clocks, "e2e": e2e,
            "gpu_launches": launches_per_layer * layers * args.steps,
            "roofline": roofline, "cpu_baseline": cpu_baseline,
        }
        print(json.dumps(line))
    replicas.finish(world)


if __name__ == "__main__":
    main()
