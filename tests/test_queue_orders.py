"""Other queue orders (Section 4.2: the scheduling algorithm works with other ordering algorithms than
first come first served) and per-node CPU scheduling with trajectories pinned to nodes (Section 5.2).
CPU pins worked by hand; the GPU tests compare the CUDA path with the oracle."""
import numpy as np
import pytest

from workloads import POOL_API, POOL_CPU, POOL_GPU, Pool, add_trajectories, random_round

SJF, LJF, ARRIVAL = 1, 2, 3


def _arrays(rows, arrival=None):
    """rows: (pool, unit, mask, s, p); one scenario."""
    n = len(rows)
    return dict(pool=np.array([[r[0] for r in rows]], np.uint8), unit=np.array([[r[1] for r in rows]], np.uint8),
                level_mask=np.array([[r[2] for r in rows]], np.uint32), s_us=np.array([[r[3] for r in rows]], np.int64),
                p_us=np.array([[r[4] for r in rows]], np.int64),
                arrival_us=None if arrival is None else np.array([arrival], np.int64),
                n_actions=np.array([n], np.int32), gpu_busy=None)


def test_keys_and_ties_of_the_three_orders(oracle):
    pools = [Pool(POOL_CPU, 8, 8)]
    # least levels: a: r = 2 -> 10 + 100 / 2 = 60; b: r = 1 -> 60; c: r = 4 -> 0 + 90 / 4 = 22; d: r = 1 -> 300
    rows = [(0, 1, 0b1010, 10, 100), (0, 1, 0b1, 60, 0), (0, 1, 0b1000, 0, 90), (0, 1, 0b11, 100, 200)]
    a = _arrays(rows, arrival=[40, 10, 30, 10])
    assert list(oracle.order_queue(pools, a, SJF)[0]) == [2, 0, 1, 3]          # 22, 60 (a before b: queue order), 300
    assert list(oracle.order_queue(pools, a, LJF)[0]) == [3, 0, 1, 2]
    assert list(oracle.order_queue(pools, a, ARRIVAL)[0]) == [1, 3, 2, 0]      # 10 (b before d), 30, 40
    assert list(oracle.order_queue(pools, a, 0)[0]) == [0, 1, 2, 3]
    a["n_actions"][0] = 3                                                       # positions behind the queue map to themselves
    assert list(oracle.order_queue(pools, a, SJF)[0]) == [2, 0, 1, 3]
    assert list(oracle.order_queue(pools, a, LJF)[0]) == [0, 1, 2, 3]


def test_shortest_first_schedules_the_shortest_actions_that_fit(oracle):
    # 3 cores, five one-core actions of 50, 10, 40, 20, 30 us: first come first served takes the first three,
    # shortest first the three shortest (10, 20, 30), longest first 50, 40, 30; results stay at the actions' positions
    pools = [Pool(POOL_CPU, 3, 3)]
    a = _arrays([(0, 1, 1, t, 0) for t in (50, 10, 40, 20, 30)])
    assert list(oracle.schedule_batch(pools, a)["alloc_units"][0]) == [1, 1, 1, 0, 0]
    o = oracle.schedule_batch_ordered(pools, a, SJF)
    assert list(o["alloc_units"][0]) == [0, 1, 0, 1, 1] and list(o["act_us"][0]) == [-1, 10, -1, 20, 30]
    assert list(o["place_off"][0]) == [-1, 0, -1, 1, 2]                         # cores are handed out in the sorted order
    o = oracle.schedule_batch_ordered(pools, a, LJF)
    assert list(o["alloc_units"][0]) == [1, 0, 1, 0, 1] and list(o["place_off"][0]) == [0, -1, 1, -1, 2]


@pytest.mark.parametrize("policy", (SJF, LJF, ARRIVAL))
def test_order_is_a_stable_sort_and_the_round_is_the_plain_round_on_the_sorted_queue(oracle, policy):
    pools = (Pool(POOL_CPU, 24, 8), Pool(POOL_GPU, 16, 8), Pool(POOL_API, 9, 0, 0))
    w, a = random_round(40 + policy, 12, 70, pools, max_mult=4, small_durations=0.4)
    a["arrival_us"] = np.random.default_rng(policy).integers(0, 50, a["pool"].shape).astype(np.int64)
    perm = oracle.order_queue(pools, a, policy)
    o = oracle.schedule_batch_ordered(pools, a, policy, now_us=60)
    for sc in range(12):
        n = int(a["n_actions"][sc])
        pm = perm[sc, :n]
        assert sorted(pm) == list(range(n))
        r = np.array([int(m & -m).bit_length() for m in a["level_mask"][sc, :n].astype(np.int64)])
        T = a["s_us"][sc, :n] + a["p_us"][sc, :n] // np.maximum(r, 1)
        key = {SJF: T, LJF: -T, ARRIVAL: a["arrival_us"][sc, :n]}[policy][pm]
        assert np.all(np.diff(key) >= 0)
        assert np.all(np.diff(pm)[np.diff(key) == 0] > 0)                       # equal keys keep their queue order
        # the plain round on the permuted records gives the same schedule, position by position
        b = {k: (v[sc:sc + 1, :n][:, pm] if k in ("pool", "unit", "level_mask", "s_us", "p_us", "arrival_us") else None)
             for k, v in a.items()}
        b["n_actions"] = np.array([n], np.int32)
        b["gpu_busy"] = a["gpu_busy"][sc:sc + 1] if a["gpu_busy"] is not None else None
        plain = oracle.schedule_batch(pools, b, now_us=60)
        for k in ("alloc_units", "place_node", "place_off", "act_us"):
            assert np.array_equal(plain[k][0, :n], o[k][sc, :n][pm]), (sc, k)
        assert plain["n_selected"][0] == o["n_selected"][sc] and plain["total_act_us"][0] == o["total_act_us"][sc]


# ------------------------------------------------------------------ trajectories pinned to CPU nodes
def _traj(rows, traj, mem, node, free):
    a = _arrays(rows)
    a["trajectory"], a["traj_mem"] = np.array([traj], np.int32), np.array([mem], np.uint32)
    a["traj_node"], a["node_mem_free"] = np.array([node], np.int32), np.array([free], np.int64)
    return a


NODES = [Pool(POOL_CPU, 8, 8), Pool(POOL_CPU, 16, 8), Pool(POOL_GPU, 8, 8), Pool(POOL_CPU, 16, 8)]


def test_a_trajectory_goes_to_the_node_with_the_most_free_memory_and_stays_there(oracle):
    one = (0, 1, 1, 100, 0)
    # free memory 50 / 70 / - / 70: trajectory 0 (20) -> node 1 (most free, lower index of the tie), 50 left;
    # trajectory 1 (30) -> node 3 (70), 40 left; trajectory 0 again -> node 1, nothing more set aside;
    # trajectory 2 (45) -> node 0 (50 / 50 / 40: lower index), 5 left; the action without a trajectory keeps its pool
    a = _traj([one] * 5, [0, 1, 0, 2, -1], [20, 30, 20, 45, 9], [-1, -1, -1], [50, 70, 999, 70])
    o = oracle.pin_trajectories(NODES, a, a["traj_node"], a["node_mem_free"])
    assert list(o["pool"][0]) == [1, 3, 1, 0, 0] and o["n_admitted"][0] == 5
    assert list(o["traj_node"][0]) == [1, 3, 0] and list(o["node_mem_free"][0]) == [5, 50, 999, 40]


def test_nodes_without_the_cores_or_the_memory_are_filtered_out(oracle):
    # the action needs at least 4 x 3 = 12 cores: node 0 (8 cores) is out although it has the most memory
    a = _traj([(0, 4, 0b1100, 100, 0)], [0], [10], [-1], [90, 20, 999, 30])
    o = oracle.pin_trajectories(NODES, a, a["traj_node"], a["node_mem_free"])
    assert o["pool"][0, 0] == 3 and list(o["node_mem_free"][0]) == [90, 20, 999, 20]
    # the memory of the whole trajectory has to be free: 25 fits node 3 only
    a = _traj([(0, 1, 1, 100, 0)], [0], [25], [-1], [24, 20, 999, 30])
    assert oracle.pin_trajectories(NODES, a, a["traj_node"], a["node_mem_free"])["pool"][0, 0] == 3
    # a pinned trajectory is not moved, whatever the memory says now; a GPU action is none of the CPU manager's
    a = _traj([(0, 1, 1, 100, 0), (2, 1 | 0x80, 1, 100, 0)], [0, 1], [25, 5], [0, -1], [0, 20, 999, 30])
    o = oracle.pin_trajectories(NODES, a, a["traj_node"], a["node_mem_free"])
    assert list(o["pool"][0]) == [0, 2] and list(o["traj_node"][0]) == [0, -1] and list(o["node_mem_free"][0]) == [0, 20, 999, 30]


def test_a_trajectory_that_finds_no_node_ends_the_admitted_queue(oracle):
    one = (0, 1, 1, 100, 0)
    a = _traj([one] * 4, [0, 1, 2, 0], [10, 80, 5, 10], [-1, -1, -1], [50, 60, 999, 70])
    o = oracle.pin_trajectories(NODES, a, a["traj_node"], a["node_mem_free"])
    # trajectory 0 -> node 3 (60 left); trajectory 1 needs 80: nowhere; what stands behind it waits as well
    assert o["n_admitted"][0] == 1 and list(o["traj_node"][0]) == [3, -1, -1]
    assert list(o["pool"][0]) == [3, 0, 0, 0] and list(o["node_mem_free"][0]) == [50, 60, 999, 60]
