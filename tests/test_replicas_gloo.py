"""The multi-GPU host logic (replicas, barrier, max-over-ranks timing) on two gloo ranks."""
import os
import socket
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    from paper_2404_14469_b200 import replicas, synth

    r, w, local = replicas.init("gloo")
    assert (r, w, local) == (rank, world, rank)
    # each rank draws different sequences of the same workload
    wl = synth.Workload(60, "t", 1, 2, 2, 64, 256, 16, 5, "max", (64,), 1, 1)
    data = synth.make_layer(wl, replicas.layer_seed_offset(r))
    replicas.barrier(w)
    my_ms = 10.0 + 5.0 * r                      # pretend rank 1 was slower
    slowest = replicas.max_over_ranks(my_ms, w)
    value = replicas.aggregate_throughput(wl.B * wl.L, w, slowest)
    out.put((r, slowest, value, float(data["k"].float().sum())))
    replicas.finish(w)


def test_two_replicas_agree_on_the_slowest_time():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, s0, v0, k0), (r1, s1, v1, k1) = res
    assert s0 == s1 == 15.0                      # max over ranks, seen by both
    assert v0 == v1 == 256 * 2 / 15e-3           # both ranks' tokens over the slowest time
    assert k0 != k1                              # different sequences per rank


def test_single_process_defaults():
    sys.path.insert(0, ROOT)
    from paper_2404_14469_b200 import replicas

    for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK"):
        os.environ.pop(k, None)
    assert replicas.env_rank_world() == (0, 1, 0)
    assert replicas.max_over_ranks(3.5, 1) == 3.5
    assert replicas.aggregate_throughput(100, 1, 10.0) == 10000.0


def test_bench_launches_its_own_ranks_when_asked_for_two_gpus():
    # `bench.py --gpus 2` outside a launcher starts two ranks itself.  The reference arm needs
    # no GPU: rank 0 times the oracle on a small sample and prints the line, rank 1 exits 0.
    import json
    import subprocess

    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--impl", "reference",
                          "--workload", "0", "--steps", "1", "--warmup", "0"],
                         capture_output=True, text=True, timeout=600, env=env, cwd=ROOT)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [json.loads(x) for x in res.stdout.splitlines() if x.startswith("{")]
    assert len(lines) == 1                       # one line for the whole job, from rank 0
    line = lines[0]
    assert line["impl"] == "reference" and line["n_gpus"] == 2
    assert line["config"]["workload"] == "tiny-1k" or line["config"]["L"] == 1024
    assert line["value"] > 0 and line["cpu_baseline"]["kind"] == "oracle"
    assert line["extrapolated"]["ms_per_full_step"] > 0
