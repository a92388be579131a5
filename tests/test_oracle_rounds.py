"""Invariants of whole rounds and of the trace replay, checked on the oracle's outputs.

These hold for any correct implementation (capacity, level membership, legal chunks, no
shared unit, prefix property, conservation); the CUDA parity tests reuse `check_round`.
"""
import numpy as np
import pytest

from workloads import POOL_API, POOL_CPU, POOL_GPU, Pool, generate, make_workload, random_round

GANG = 0x80


def allowed_units(unit, mask, pool: Pool):
    g, gang = int(unit) & 0x7F, bool(int(unit) & GANG) and pool.type == POOL_GPU
    out = []
    for r in range(1, 33):
        if int(mask) >> (r - 1) & 1:
            k = g * r
            if gang and not (k & (k - 1) == 0 and k <= pool.group):
                continue
            out.append(k)
    return out


def check_round(pools, a, o, now_us=0):
    """Assert every single-round invariant on outputs `o` for inputs `a`."""
    S, N = a["pool"].shape
    node0 = []
    acc = 0
    for p in pools:
        node0.append(acc)
        if p.type == POOL_GPU:
            acc += p.capacity // p.group
    for sc in range(S):
        n = int(a["n_actions"][sc])
        alloc, node, off, act = (o[k][sc] for k in ("alloc_units", "place_node", "place_off", "act_us"))
        assert np.all(alloc[n:] == 0) and np.all(act[n:] == -1)
        if o["status"][sc] != 0:
            assert np.all(alloc == 0) and o["n_selected"][sc] == 0
            continue
        sel = alloc[:n] > 0
        assert o["n_selected"][sc] == sel.sum()
        assert np.all(act[:n][~sel] == -1) and np.all(node[:n][~sel] == -1) and np.all(off[:n][~sel] == -1)
        assert o["total_act_us"][sc] == act[:n][sel].sum()
        # selected actions form, per pool, a prefix of that pool's queue, and nothing behind the
        # global candidate prefix is selected
        last_selected = np.flatnonzero(sel).max() if sel.any() else -1
        for j, p in enumerate(pools):
            mine = np.flatnonzero(a["pool"][sc, :n] == j)
            picked = sel[mine]
            if picked.any():
                assert picked[: picked.sum()].all(), "selection is not a prefix of the pool's queue"
            used = int(alloc[mine].sum())
            busy_before = 0
            if p.type == POOL_GPU and a.get("gpu_busy") is not None:
                nodes = p.capacity // p.group
                busy_before = int(sum(bin(int(b)).count("1") for b in a["gpu_busy"][sc, node0[j]:node0[j] + nodes]))
            assert used + busy_before <= p.capacity, "pool oversubscribed"
            for i in mine[picked]:
                assert alloc[i] in allowed_units(a["unit"][sc, i], a["level_mask"][sc, i], p)
                arr = 0 if a.get("arrival_us") is None else int(a["arrival_us"][sc, i])
                r = alloc[i] // (int(a["unit"][sc, i]) & 0x7F)
                s_, p_ = min(max(int(a["s_us"][sc, i]), 0), 1 << 40), min(max(int(a["p_us"][sc, i]), 0), 1 << 40)
                assert act[i] == now_us - arr + s_ + p_ // r
            if p.type == POOL_GPU:
                for i in mine[picked]:
                    g = int(a["unit"][sc, i]) & 0x7F
                    size = alloc[i] if int(a["unit"][sc, i]) & GANG else g
                    assert 0 <= node[i] < p.capacity // p.group
                    assert off[i] % size == 0 and off[i] + size <= p.group, "illegal chunk"
                    if a.get("gpu_busy") is not None:
                        b = int(a["gpu_busy"][sc, node0[j] + node[i]])
                        assert b & (((1 << size) - 1) << off[i]) == 0, "chunk on a busy GPU"
            if p.type == POOL_CPU:
                for i in mine[picked]:
                    assert 0 <= off[i] < p.capacity and node[i] == off[i] // p.group
        # a waiting action ahead of the last selected one in another pool is allowed (eviction),
        # but nothing is selected behind the first action that was not even a candidate
        assert last_selected < n


POOLSETS = [
    (Pool(POOL_CPU, 16, 4), Pool(POOL_GPU, 16, 8), Pool(POOL_API, 5, 0, 1_000_000)),
    (Pool(POOL_GPU, 24, 8),),
    (Pool(POOL_CPU, 40, 8), Pool(POOL_GPU, 8, 4)),
    (Pool(POOL_CPU, 6, 2), Pool(POOL_API, 3, 0, 0)),
]


@pytest.mark.parametrize("seed", range(8))
def test_random_rounds_satisfy_invariants(oracle, seed):
    pools = POOLSETS[seed % len(POOLSETS)]
    w, a = random_round(100 + seed, 24, 40, pools, small_durations=0.3 if seed % 2 else 0.0,
                        busy_fraction=0.3 if seed % 3 == 0 else 0.0)
    o = oracle.schedule_batch(pools, a, depth=2, now_us=777)
    check_round(pools, a, o, now_us=777)
    assert (o["n_selected"] > 0).sum() > 5


@pytest.mark.parametrize("name,S", [("cfg0", 1), ("cfg1", 6), ("cfg3", 6), ("cfg4", 3)])
def test_named_configs_satisfy_invariants(oracle, name, S):
    w = make_workload(name, n_scenarios=S)
    a = generate(w)
    o = oracle.schedule_batch(w.pools, a, depth=w.depth)
    check_round(w.pools, a, o)
    assert np.all(o["status"] == 0) and np.all(o["n_selected"] > 0)
    # the tight pool is used to the last unit wherever a waiting action of one unit remains
    if name in ("cfg1", "cfg4"):
        gpu = [j for j, p in enumerate(w.pools) if p.type == POOL_GPU][0]
        used = (o["alloc_units"] * (a["pool"] == gpu)).sum(1)
        assert np.all(used <= w.pools[gpu].capacity) and np.median(used) >= 0.9 * w.pools[gpu].capacity


def test_scenarios_are_independent_of_batching(oracle):
    w = make_workload("cfg1", n_scenarios=5)
    a = generate(w)
    whole = oracle.schedule_batch(w.pools, a)
    for sc in (0, 3):
        one = oracle.schedule_batch(w.pools, a, lo=sc, hi=sc + 1)
        for k in whole:
            assert np.array_equal(one[k][0], whole[k][sc])
    # generating a slice alone gives the same records (seed = base + scenario id)
    part = generate(w, 3, 5)
    assert np.array_equal(part["s_us"], a["s_us"][3:5]) and np.array_equal(part["level_mask"], a["level_mask"][3:5])


# ------------------------------------------------------------------ trace replay
def check_replay(pools, a, o, round_us, max_rounds):
    S, N = a["pool"].shape
    for sc in range(S):
        n = int(a["n_actions"][sc])
        if o["status"][sc] != 0:
            continue
        act, alloc = o["act_us"][sc, :n], o["alloc_units"][sc, :n]
        started = act >= 0
        assert o["n_selected"][sc] == started.sum()
        assert np.all(alloc[started] > 0) and np.all(alloc[~started] == 0)
        arr = a["arrival_us"][sc, :n]
        g = a["unit"][sc, :n].astype(np.int64) & 0x7F
        r = np.where(started, alloc // g, 1)
        T = np.clip(a["s_us"][sc, :n], 0, 1 << 40) + np.clip(a["p_us"][sc, :n], 0, 1 << 40) // r
        start_t = arr + act - T                                     # ACT = (start - arrival) + T
        assert np.all(start_t[started] >= arr[started])
        assert np.all(start_t[started] % round_us == 0), "actions start on round boundaries"
        finish = start_t + T
        R = int(o["rounds_used"][sc])
        # occupancy of round r = units of actions running just after that round's scheduling
        occ = o["occupancy"][sc]
        for j, p in enumerate(pools):
            mine = started & (a["pool"][sc, :n] == j)
            assert occ[:, j].max() <= p.capacity
            for rr in np.linspace(0, max(R - 1, 0), 25).astype(int):
                now = rr * round_us
                if p.type == POOL_API and p.window_us > 0:
                    w0 = now // p.window_us * p.window_us
                    expect = alloc[mine & (start_t >= w0) & (start_t <= now)].sum()
                else:
                    expect = alloc[mine & (start_t <= now) & (finish > now)].sum()
                assert occ[rr, j] == expect, (sc, j, rr)
        assert np.all(occ[R:] == 0)
        if started.all():
            assert R <= max_rounds and R * round_us >= finish.max()


def test_replay_conservation_small(oracle):
    w = make_workload("cfg2", n_scenarios=3, max_actions=600)
    a = generate(w)
    max_rounds = 4000
    o = oracle.replay_trace(w.pools, a, depth=2, round_us=w.round_us, max_rounds=max_rounds)
    assert np.all(o["status"] == 0) and np.all(o["n_selected"] == 600)
    check_replay(w.pools, a, o, w.round_us, max_rounds)
    # with GPUs scarce some reward-model actions queue, so some ACT exceeds the bare duration
    T1 = a["s_us"] + a["p_us"]
    assert (o["act_us"] > T1).any()


def test_replay_idle_cluster_runs_everything_at_once(oracle):
    # arrivals far apart on an empty, ample cluster: each action starts at the first round
    # boundary at or after its arrival, with every unit it can use
    pools = (Pool(POOL_CPU, 64, 8),)
    n = 5
    arr = np.array([[0, 25_000, 50_001, 99_999, 200_000]], np.int64)
    a = dict(pool=np.zeros((1, n), np.uint8), unit=np.ones((1, n), np.uint8),
             level_mask=np.full((1, n), 0x8B, np.uint32), s_us=np.full((1, n), 100, np.int64),
             p_us=np.full((1, n), 8000, np.int64), arrival_us=arr, n_actions=np.array([n], np.int32), gpu_busy=None)
    o = oracle.replay_trace(pools, a, round_us=10_000, max_rounds=100)
    start = (arr + 9_999) // 10_000 * 10_000
    assert list(o["alloc_units"][0]) == [8] * n
    assert np.array_equal(o["act_us"], start - arr + 100 + 1000)
    assert o["rounds_used"][0] == 22                                  # drained at the round after the last finish


def test_replay_quota_window_and_unsorted_trace(oracle):
    # one token per second: one call starts per window, in queue order
    pools = (Pool(POOL_API, 1, 0, 1_000_000),)
    n = 3
    a = dict(pool=np.zeros((1, n), np.uint8), unit=np.ones((1, n), np.uint8), level_mask=np.ones((1, n), np.uint32),
             s_us=np.full((1, n), 5, np.int64), p_us=np.zeros((1, n), np.int64), arrival_us=np.zeros((1, n), np.int64),
             n_actions=np.array([n], np.int32), gpu_busy=None)
    o = oracle.replay_trace(pools, a, round_us=250_000, max_rounds=20)
    assert list(o["act_us"][0]) == [5, 1_000_005, 2_000_005]
    a["arrival_us"] = np.array([[5, 4, 6]], np.int64)
    o = oracle.replay_trace(pools, a, round_us=250_000, max_rounds=20)
    assert o["status"][0] == 2 and o["n_selected"][0] == 0


def test_cfg0_matches_stored_schedule(oracle):
    """Regression fixture written by tests/golden/make_cfg0_golden.py (oracle only): guards the
    input generator and the oracle against silent drift."""
    import os
    w = make_workload("cfg0")
    a = generate(w)
    o = oracle.schedule_batch(w.pools, a, depth=w.depth)
    rows = [l for l in open(os.path.join(os.path.dirname(__file__), "golden", "cfg0_schedule.txt")) if l[0] != "#"]
    assert len(rows) == 64
    for line in rows:
        left, right = line.split("|")
        i, pool, unit, mask, s, p = (int(x) for x in left.split())
        alloc, node, off, act = (int(x) for x in right.split())
        assert (a["pool"][0, i], a["unit"][0, i], a["level_mask"][0, i], a["s_us"][0, i], a["p_us"][0, i]) == \
            (pool, unit, mask, s, p)
        assert (o["alloc_units"][0, i], o["place_node"][0, i], o["place_off"][0, i], o["act_us"][0, i]) == \
            (alloc, node, off, act)
