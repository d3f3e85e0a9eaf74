"""Gated block pool + controller: the C++ implementation against the plain model in oracle/ on random
operation sequences (integer work: exact agreement), the model against a hand-worked trace, and the
invariants the paper states (elastic ids are never handed out while gated; a drain leaves none in use)."""
import os
import random

import pytest

import paper_2608_23658_b200 as ekv
from oracle.blockpool_model import BlockPoolModel, ControllerModel

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "blockpool_trace.txt")
ACT = {0: "NONE", 1: "COMMIT", 2: "DECOMMIT"}


class LibPool:
    """Same verbs as the model, on the library."""

    def __init__(self, base, elastic):
        self.h = ekv.ekv_blockpool_create(base, elastic)
        self.cap = base + elastic

    def close(self):
        ekv.ekv_blockpool_destroy(self.h)

    def alloc(self, n):
        try:
            return ekv.ekv_blockpool_alloc(self.h, n)
        except ekv.EkvError as e:
            assert e.status == ekv.Status.ERR_OOM
            return None

    def free(self, ids):
        try:
            ekv.ekv_blockpool_free(self.h, ids)
            return True
        except ekv.EkvError as e:
            assert e.status in (ekv.Status.ERR_INVALID, ekv.Status.ERR_STATE)
            return False if e.status == ekv.Status.ERR_INVALID else "state"

    def admit(self):
        try:
            ekv.ekv_blockpool_admit_elastic(self.h)
            return True
        except ekv.EkvError as e:
            assert e.status == ekv.Status.ERR_STATE
            return False

    def gate(self):
        return ekv.ekv_blockpool_gate_elastic(self.h)

    def drain_plan(self):
        try:
            return ekv.ekv_blockpool_drain_plan(self.h, self.cap)
        except ekv.EkvError as e:
            return {ekv.Status.ERR_OOM: "oom", ekv.Status.ERR_STATE: "state"}[e.status]

    def drain_commit(self):
        ekv.ekv_blockpool_drain_commit(self.h)

    def num_gpu_blocks(self):
        return ekv.ekv_blockpool_stats(self.h).num_gpu_blocks


def _run_trace(pool_factory, ctrl_factory):
    pool, ctrl = pool_factory(3, 2), None
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line[0] == "#":
            continue
        if line.startswith("ctrl"):
            _, n, thr = line.split()
            ctrl = ctrl_factory(int(n), int(thr))
            continue
        lhs, want = [x.strip() for x in line.split("->")]
        op, *args = lhs.split()
        args = [int(a) for a in args]
        if op == "alloc":
            got = pool.alloc(args[0])
            got = "OOM" if got is None else " ".join(map(str, got))
        elif op == "free":
            got = "ok" if pool.free(args) else "BAD"
        elif op == "admit":
            got = "ok" if pool.admit() else "STATE"
        elif op == "gate":
            got = str(pool.gate())
        elif op == "numblocks":
            got = str(pool.num_gpu_blocks())
        elif op == "plan":
            r = pool.drain_plan()
            got = r.upper() if isinstance(r, str) else " ".join(f"{a}:{b}" for a, b in zip(*r))
        elif op == "commit":
            pool.drain_commit()
            got = "ok"
        elif op == "decide":
            got = ACT[ctrl(args[0])]
        assert got == want, (line, got)
    return pool


def test_model_follows_the_hand_worked_trace():
    def ctrl(n, thr):
        c = ControllerModel(n, thr)
        return c.decide
    _run_trace(BlockPoolModel, ctrl)


def test_library_follows_the_hand_worked_trace():
    def ctrl(n, thr):
        h = ekv.ekv_controller_create(n, thr)
        return lambda t: ekv.ekv_controller_decide(h, t)
    _run_trace(LibPool, ctrl).close()


@pytest.mark.parametrize("seed", range(6))
def test_library_matches_model_on_random_operations(seed):
    rng = random.Random(seed)
    base, elastic = rng.randint(1, 40), rng.randint(0, 24)
    lib, mod = LibPool(base, elastic), BlockPoolModel(base, elastic)
    held = []
    try:
        for step in range(3000):
            op = rng.random()
            if op < 0.40:
                n = rng.randint(0, 6)
                a, b = lib.alloc(n), mod.alloc(n)
                assert a == b
                if a:
                    held += a
                    if not mod.admitted:
                        assert all(i < base for i in a), "an elastic id was handed out while gated"
            elif op < 0.70 and held:
                k = rng.randint(1, min(5, len(held)))
                ids = rng.sample(held, k)
                if rng.random() < 0.1:
                    ids = ids + [ids[0]]                            # duplicate: must be refused, nothing freed
                if mod.plan and any(i in mod.plan[0] or i in mod.plan[1] for i in ids):
                    continue                                        # blocks of an outstanding drain are not the caller's to free
                a, b = lib.free(ids), mod.free(ids)
                assert a == b
                if a:
                    held = [i for i in held if i not in ids]
            elif op < 0.76:
                assert lib.admit() == mod.admit()
            elif op < 0.82:
                assert lib.gate() == mod.gate()
            elif op < 0.90:
                a, b = lib.drain_plan(), mod.drain_plan()
                assert a == (b if isinstance(b, str) else (b[0], b[1]))
                if not isinstance(b, str):
                    src, dst = b
                    assert src == sorted(src) and all(i >= base for i in src) and all(i < base for i in dst)
                    held = [dst[src.index(i)] if i in src else i for i in held]   # the caller rewrites its tables
                    lib.drain_commit()
                    mod.drain_commit()
                    assert mod.elastic_in_use() == []               # nothing left in the range that goes away
            else:
                assert lib.free([base + elastic + 5]) is False and mod.free([base + elastic + 5]) is False
            st = ekv.ekv_blockpool_stats(lib.h)
            assert (st.free_base, st.free_elastic, st.elastic_in_use, st.num_gpu_blocks, st.admitted) == \
                (len(mod.free_base), len(mod.free_elastic), len(mod.elastic_in_use()), mod.num_gpu_blocks(), int(mod.admitted))
            assert st.free_base + st.free_elastic + len(set(held)) == base + elastic and len(set(held)) == len(held)
    finally:
        lib.close()


def test_ids_of_an_outstanding_drain_plan_cannot_be_freed():
    """Between drain_plan and drain_commit both sides of every pair belong to the plan: freeing one would let the
    commit push the id onto a free list a second time.  Hand-worked: base 4, elastic 2; six allocations use ids
    0..5; freeing 1 and 2 leaves two base ids free; the plan pairs 4 -> 2 and 5 -> 1 (most recently freed first)."""
    for make in (LibPool, BlockPoolModel):
        pool = make(4, 2)
        assert pool.admit() is True
        assert pool.alloc(6) == [0, 1, 2, 3, 4, 5]
        assert pool.free([1, 2]) is True
        assert pool.gate() == 2
        plan = pool.drain_plan()
        assert (list(plan[0]), list(plan[1])) == ([4, 5], [2, 1])
        for ids in ([4], [1], [0, 5], [2, 3]):
            assert pool.free(ids) == "state"
        assert pool.free([0]) is True                              # an id outside the plan is still the caller's
        pool.drain_commit()
        assert pool.free([4]) is False                             # the elastic side is free now
        assert pool.free([2, 1]) is True                           # the base side became ordinary allocated blocks
        assert pool.alloc(3) == [1, 2, 0]                          # stack order: most recently freed first
        assert pool.alloc(1) is None                               # 3 is held, the elastic ids are gated
        if make is LibPool:
            pool.close()


@pytest.mark.parametrize("seed", range(4))
def test_controller_matches_model_and_respects_hysteresis(seed):
    rng = random.Random(100 + seed)
    n, thr = rng.randint(1, 8), rng.choice([1, 2048, 8192])
    start = bool(seed % 2)
    h, mod = ekv.ekv_controller_create(n, thr, start), ControllerModel(n, thr, start)
    quiet, committed, commits, decommits = 0, start, 0, 0
    for _ in range(5000):
        tokens = 0 if rng.random() < 0.85 else rng.choice([1, thr - 1, thr, thr + 1, 32768])
        tokens = max(tokens, 0)
        a, b = ekv.ekv_controller_decide(h, tokens), mod.decide(tokens)
        assert a == b
        if tokens >= thr:
            assert a != ekv.EKV_ACT_COMMIT
            assert (a == ekv.EKV_ACT_DECOMMIT) == committed          # the reserve is back before every large prefill
            committed, quiet = False, 0
        else:
            quiet += 1
            if a == ekv.EKV_ACT_COMMIT:
                assert quiet >= n and not committed                   # never earlier than the hysteresis window
                committed = True
            else:
                assert a == ekv.EKV_ACT_NONE
        commits += a == ekv.EKV_ACT_COMMIT
        decommits += a == ekv.EKV_ACT_DECOMMIT
    st = ekv.ekv_controller_stats(h)
    assert (st.steps, st.commits, st.decommits, st.committed) == (5000, commits, decommits, int(committed))
    ekv.ekv_controller_destroy(h)
