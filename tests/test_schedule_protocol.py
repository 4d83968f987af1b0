"""Host-side checks of the scoring kernel's schedule and of the hand-over of the softmax
statistics between its blocks (Eq. 1 needs each window row's normaliser over ALL keys before
any probability can be summed, so blocks that share a unit exchange partial log-sum-exps).

The item lists come from the library itself (snapkv_schedule_items runs the kernel's own item
walk on the host).  The hand-over is modelled with one CPU thread per block: publish a
partial and count it; before a vote item, wait (with a time limit) until the unit's count
says that all partials are there, then fold them in slot order.  The model shows that the
schedule cannot deadlock, that every block folds the same value whatever the thread timing,
and that a block which never arrives turns into time-outs, not into a hang."""
import threading
import time

import pytest

from paper_2404_14469_b200 import binding as sk

SHAPES = [
    # B, Hq, Hkv, L, d, W, grid
    (4, 32, 8, 32768, 128, 32, 148),    # workload 2
    (1, 32, 32, 16384, 128, 32, 148),   # workload 1
    (1, 32, 8, 131072, 128, 64, 148),   # workload 3: two head sub-groups per KV head
    (1, 32, 32, 380000, 128, 32, 148),  # workload 4: one unit per wave
    (1, 4, 4, 1024, 64, 32, 148),       # fewer tiles than blocks
    (2, 4, 2, 1000, 128, 32, 7),        # ragged, small grid
    (3, 2, 2, 257, 64, 32, 192),
    (1, 8, 1, 900, 64, 32, 33),
]


def _all_items(B, Hq, Hkv, L, d, W, grid, votes_only=False):
    per_cta, plan = [], None
    for c in range(grid):
        items, plan = sk.snapkv_schedule_items(B, Hq, Hkv, L, d, W, grid, c, votes_only)
        per_cta.append(items)
    return per_cta, plan


@pytest.mark.parametrize("B,Hq,Hkv,L,d,W,grid", SHAPES)
def test_every_tile_is_covered_once_and_slots_are_dense(B, Hq, Hkv, L, d, W, grid):
    per_cta, plan = _all_items(B, Hq, Hkv, L, d, W, grid)
    for vote, T in ((0, plan["tiles_stats"]), (1, plan["tiles_vote"])):
        seen = {}
        for c, items in enumerate(per_cta):
            for unit, t0, t1, v, slot, nseg in items:
                if v != vote:
                    continue
                assert 0 <= t0 < t1 <= T and 0 <= unit < plan["units"]
                for t in range(t0, t1):
                    assert (unit, t) not in seen, "a tile is handed out twice"
                    seen[(unit, t)] = c
        assert len(seen) == plan["units"] * T
    # statistics sweep: the blocks that share a unit hold slots 0 .. nseg-1, once each, and
    # all of them agree on nseg, which fits the workspace's partial slots
    slots = {}
    for items in per_cta:
        for unit, t0, t1, v, slot, nseg in items:
            if v == 0:
                slots.setdefault(unit, []).append((slot, nseg))
    for unit, lst in slots.items():
        nsegs = {n for _, n in lst}
        assert len(nsegs) == 1
        nseg = nsegs.pop()
        assert sorted(s for s, _ in lst) == list(range(nseg))
        assert nseg <= plan["maxseg"]
    # vote items carry the nseg of their unit's statistics sweep
    for items in per_cta:
        for unit, t0, t1, v, slot, nseg in items:
            if v == 1:
                assert nseg == len(slots[unit])


@pytest.mark.parametrize("B,Hq,Hkv,L,d,W,grid", SHAPES)
def test_a_block_reaches_a_units_votes_only_after_its_own_statistics(B, Hq, Hkv, L, d, W, grid):
    per_cta, plan = _all_items(B, Hq, Hkv, L, d, W, grid)
    # where each block has its statistics items of a unit
    own = [{} for _ in per_cta]
    for c, items in enumerate(per_cta):
        for i, (unit, t0, t1, v, slot, nseg) in enumerate(items):
            if v == 0:
                own[c][unit] = max(own[c].get(unit, -1), i)
    for c, items in enumerate(per_cta):
        for i, (unit, t0, t1, v, slot, nseg) in enumerate(items):
            if v == 1 and unit in own[c]:
                assert own[c][unit] < i   # else the block would wait for itself


def test_votes_only_schedule_is_one_phase_without_statistics():
    per_cta, plan = _all_items(2, 8, 2, 5000, 128, 32, 148, votes_only=True)
    assert plan["waves"] == 1
    assert all(v == 1 for items in per_cta for (_, _, _, v, _, _) in items)
    tiles = sum(t1 - t0 for items in per_cta for (_, t0, t1, _, _, _) in items)
    assert tiles == plan["units"] * plan["tiles_vote"]


class _Model:
    """One thread per block; `absent` blocks never run."""

    def __init__(self, per_cta, units, limit_s):
        self.per_cta, self.limit = per_cta, limit_s
        self.partials = [dict() for _ in range(units)]
        self.count = [0] * units
        self.lock = threading.Lock()
        self.abort = [0] * len(per_cta)
        self.folds = [[] for _ in per_cta]

    def run_block(self, c, jitter):
        for k, (unit, t0, t1, vote, slot, nseg) in enumerate(self.per_cta[c]):
            if jitter:
                time.sleep(((c * 7 + k * 3) % 5) * 1e-4)
            if not vote:
                value = (unit + 1) * 1000 + slot        # stands for the block's partial
                self.partials[unit][slot] = value        # the data first ...
                with self.lock:
                    self.count[unit] += 1                # ... then the count (release)
            else:
                t_end = time.monotonic() + self.limit / 2   # a wait on other blocks: half the limit
                while True:
                    with self.lock:
                        ready = self.count[unit] >= nseg
                    if ready:
                        break
                    if time.monotonic() > t_end:
                        self.abort[c] = 7                # the code of the wait for a unit's statistics
                        return
                    time.sleep(1e-4)
                acc = 0
                for s in range(nseg):                    # slot order: the same in every block
                    acc = acc * 31 + self.partials[unit][s]
                self.folds[c].append((unit, acc))

    def run(self, absent=(), jitter=True):
        threads = [threading.Thread(target=self.run_block, args=(c, jitter))
                   for c in range(len(self.per_cta)) if c not in absent]
        t0 = time.monotonic()
        for t in threads:
            t.start()
        for t in threads:
            t.join(timeout=30)
        assert not any(t.is_alive() for t in threads), "the model hangs"
        return time.monotonic() - t0


@pytest.mark.parametrize("shape", [(2, 8, 2, 3000, 128, 32, 24), (1, 4, 4, 1024, 64, 32, 40)])
def test_hand_over_completes_and_every_block_folds_the_same_value(shape):
    per_cta, plan = _all_items(*shape)
    m = _Model(per_cta, plan["units"], limit_s=5.0)
    m.run()
    assert not any(m.abort)
    by_unit = {}
    for folds in m.folds:
        for unit, acc in folds:
            by_unit.setdefault(unit, set()).add(acc)
    assert set(by_unit) == set(range(plan["units"]))
    assert all(len(v) == 1 for v in by_unit.values())


def test_a_block_that_never_arrives_becomes_time_outs_not_a_hang():
    shape = (2, 8, 2, 3000, 128, 32, 24)
    per_cta, plan = _all_items(*shape)
    m = _Model(per_cta, plan["units"], limit_s=0.4)
    took = m.run(absent={5})
    # blocks that share a unit with block 5 give up at half the limit with the code of that
    # wait; nobody waits longer than the limit
    units_of_5 = {u for (u, _, _, v, _, _) in per_cta[5] if v == 0}
    waiting = [c for c, items in enumerate(per_cta)
               if c != 5 and any(v == 1 and u in units_of_5 for (u, _, _, v, _, _) in items)]
    assert waiting and all(m.abort[c] == 7 for c in waiting)
    assert took < 5.0


def test_wait_limit_setter_returns_the_previous_value_and_has_a_floor():
    prev = sk.snapkv_set_wait_limit_ns(5)            # raised to one millisecond
    try:
        assert sk.snapkv_set_wait_limit_ns(20_000_000) == 1_000_000
        assert sk.snapkv_set_wait_limit_ns(30_000_000) == 20_000_000
    finally:
        sk.snapkv_set_wait_limit_ns(prev)
    assert prev == 1_000_000_000
