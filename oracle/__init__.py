"""ctypes front end of the CPU oracle (TEST INFRASTRUCTURE, not part of the product).

Only tests, the smoke check and the CPU-baseline leg of the benchmark may import this
package.  It compiles `tangram_oracle.cpp` with g++ on first use and exposes the whole
round, the trace replay and the single pieces (duration, chunk test, DPArrange,
estimate, chunk allocation) as numpy-in / numpy-out functions.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Dict, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "tangram_oracle.cpp")
_LIB = os.path.join(_HERE, "libtangram_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle into a shared library next to its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["g++", "-O2", "-std=c++17", "-shared", "-fPIC", "-o", _LIB, _SRC])
    return _LIB


def _p(a: Optional[np.ndarray], ctype):
    if a is None:
        return C.cast(None, C.POINTER(ctype))
    return a.ctypes.data_as(C.POINTER(ctype))


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.oracle_duration.restype = C.c_longlong
        _lib.oracle_duration.argtypes = [C.c_longlong, C.c_longlong, C.c_int]
        _lib.oracle_encode.restype = C.c_longlong
        _lib.oracle_estimate.restype = C.c_longlong
    return _lib


def _pools_flat(pools: Sequence) -> np.ndarray:
    return np.array([[p.type, p.capacity, p.group, p.window_us] for p in pools], dtype=np.int32).ravel()


def _n_nodes(pools: Sequence) -> int:
    return sum(p.capacity // p.group for p in pools if p.type == 1)


def _c(a, dt):
    return None if a is None else np.ascontiguousarray(a, dtype=dt)


def _cache_args(arrays, sl, S, pools, cache_slots):
    """service / restore_us / cache state of scenarios `sl` (copies: the oracle updates the state in place)."""
    service = _c(arrays["service"][sl], np.uint16) if arrays.get("service") is not None else None
    restore = _c(arrays["restore_us"][sl], np.int64) if arrays.get("restore_us") is not None else None
    tag = use = None
    if cache_slots > 0:
        n = _n_nodes(pools) * 8 * cache_slots
        tag = (np.array(arrays["cache_tag"][sl], dtype=np.uint32, order="C", copy=True).reshape(S, n)
               if arrays.get("cache_tag") is not None else np.zeros((S, n), np.uint32))
        use = (np.array(arrays["cache_use"][sl], dtype=np.int64, order="C", copy=True).reshape(S, n)
               if arrays.get("cache_use") is not None else np.zeros((S, n), np.int64))
    return service, restore, tag, use


def _side_args(arrays, sl):
    """Further entries of the cost vectors, [n_side][scenario][action] (pool 0xff: none)."""
    if arrays.get("side_pool") is None:
        return 0, None, None
    sp = _c(arrays["side_pool"][:, sl], np.uint8)
    su = _c(arrays["side_units"][:, sl], np.uint16)
    return sp.shape[0], sp, su


def schedule_batch(pools: Sequence, arrays: Dict[str, Optional[np.ndarray]], *, depth: int = 2,
                   now_us: int = 0, lo: int = 0, hi: Optional[int] = None, cache_slots: int = 0) -> Dict[str, np.ndarray]:
    """One scheduling round for scenarios [lo, hi) of the given input arrays.  With cache_slots > 0 the
    GPU pools keep a service cache (arrays "service", "restore_us", "cache_tag", "cache_use"); the
    updated cache state comes back as "cache_tag" / "cache_use"."""
    S_all, N = arrays["pool"].shape
    hi = S_all if hi is None else hi
    S = hi - lo
    sl = slice(lo, hi)
    pool = _c(arrays["pool"][sl], np.uint8)
    unit = _c(arrays["unit"][sl], np.uint8)
    mask = _c(arrays["level_mask"][sl], np.uint32)
    s = _c(arrays["s_us"][sl], np.int64)
    p = _c(arrays["p_us"][sl], np.int64)
    arr = _c(arrays["arrival_us"][sl], np.int64) if arrays.get("arrival_us") is not None else None
    busy = _c(arrays["gpu_busy"][sl], np.uint8) if arrays.get("gpu_busy") is not None else None
    n_act = _c(arrays["n_actions"][sl], np.int32)
    out = dict(
        alloc_units=np.empty((S, N), np.int32), place_node=np.empty((S, N), np.int32),
        place_off=np.empty((S, N), np.int32), act_us=np.empty((S, N), np.int64),
        total_act_us=np.empty(S, np.int64), n_selected=np.empty(S, np.int32),
        status=np.empty(S, np.int32))
    pf = _pools_flat(pools)
    service, restore, tag, use = _cache_args(arrays, sl, S, pools, cache_slots)
    n_side, side_pool, side_units = _side_args(arrays, sl)
    rc = lib().oracle_schedule_batch_ext(
        C.c_int(S), C.c_int(N), C.c_int(len(pools)), _p(pf, C.c_int), C.c_int(depth),
        C.c_int(_n_nodes(pools)), _p(n_act, C.c_int), _p(pool, C.c_uint8), _p(unit, C.c_uint8),
        _p(mask, C.c_uint32), _p(s, C.c_longlong), _p(p, C.c_longlong), _p(arr, C.c_longlong),
        _p(busy, C.c_uint8), C.c_longlong(now_us),
        _p(out["alloc_units"], C.c_int), _p(out["place_node"], C.c_int), _p(out["place_off"], C.c_int),
        _p(out["act_us"], C.c_longlong), _p(out["total_act_us"], C.c_longlong),
        _p(out["n_selected"], C.c_int), _p(out["status"], C.c_int),
        _p(service, C.c_uint16), _p(restore, C.c_longlong), C.c_int(cache_slots), _p(tag, C.c_uint32),
        _p(use, C.c_longlong), C.c_int(n_side), _p(side_pool, C.c_uint8), _p(side_units, C.c_uint16))
    assert rc == 0
    if cache_slots > 0:
        out["cache_tag"], out["cache_use"] = tag, use
    return out


def replay_trace(pools: Sequence, arrays: Dict[str, Optional[np.ndarray]], *, depth: int = 2,
                 round_us: int = 10_000, max_rounds: int, lo: int = 0, hi: Optional[int] = None,
                 want_occupancy: bool = True, cache_slots: int = 0, policy: int = 0) -> Dict[str, np.ndarray]:
    """Trace replay of scenarios [lo, hi).  policy 1 / 2: the waiting queue is kept in shortest / longest
    least-level duration order (equal keys in arrival order) instead of first come first served."""
    S_all, N = arrays["pool"].shape
    hi = S_all if hi is None else hi
    S = hi - lo
    sl = slice(lo, hi)
    pool = _c(arrays["pool"][sl], np.uint8)
    unit = _c(arrays["unit"][sl], np.uint8)
    mask = _c(arrays["level_mask"][sl], np.uint32)
    s = _c(arrays["s_us"][sl], np.int64)
    p = _c(arrays["p_us"][sl], np.int64)
    arr = _c(arrays["arrival_us"][sl], np.int64) if arrays.get("arrival_us") is not None else None
    busy = _c(arrays["gpu_busy"][sl], np.uint8) if arrays.get("gpu_busy") is not None else None
    n_act = _c(arrays["n_actions"][sl], np.int32)
    out = dict(
        alloc_units=np.empty((S, N), np.int32), place_node=np.empty((S, N), np.int32),
        place_off=np.empty((S, N), np.int32), act_us=np.empty((S, N), np.int64),
        total_act_us=np.empty(S, np.int64), n_selected=np.empty(S, np.int32),
        status=np.empty(S, np.int32), rounds_used=np.empty(S, np.int32),
        occupancy=np.empty((S, max_rounds, len(pools)), np.int32) if want_occupancy else None)
    pf = _pools_flat(pools)
    service, restore, tag, use = _cache_args(arrays, sl, S, pools, cache_slots)
    n_side, side_pool, side_units = _side_args(arrays, sl)
    rc = lib().oracle_replay_trace_ext(
        C.c_int(S), C.c_int(N), C.c_int(len(pools)), _p(pf, C.c_int), C.c_int(depth),
        C.c_int(_n_nodes(pools)), C.c_longlong(round_us), C.c_int(max_rounds),
        _p(n_act, C.c_int), _p(pool, C.c_uint8), _p(unit, C.c_uint8), _p(mask, C.c_uint32),
        _p(s, C.c_longlong), _p(p, C.c_longlong), _p(arr, C.c_longlong), _p(busy, C.c_uint8),
        _p(out["alloc_units"], C.c_int), _p(out["place_node"], C.c_int), _p(out["place_off"], C.c_int),
        _p(out["act_us"], C.c_longlong), _p(out["total_act_us"], C.c_longlong),
        _p(out["n_selected"], C.c_int), _p(out["status"], C.c_int), _p(out["occupancy"], C.c_int),
        _p(out["rounds_used"], C.c_int),
        _p(service, C.c_uint16), _p(restore, C.c_longlong), C.c_int(cache_slots), _p(tag, C.c_uint32),
        _p(use, C.c_longlong), C.c_int(n_side), _p(side_pool, C.c_uint8), _p(side_units, C.c_uint16), C.c_int(policy))
    assert rc == 0
    if cache_slots > 0:
        out["cache_tag"], out["cache_use"] = tag, use
    return out


def replay_trace_pinned(pools: Sequence, arrays: Dict[str, Optional[np.ndarray]], *, depth: int = 2,
                        round_us: int = 10_000, max_rounds: int, policy: int = 0) -> Dict[str, np.ndarray]:
    """Trace replay with the trajectories pinned to CPU nodes as their actions arrive (arrays "trajectory",
    "traj_mem", "traj_last", state "traj_node", "node_mem_free").  Returns the replay's outputs plus "pool"
    (the pool every action ran on) and the final state "traj_node" / "node_mem_free" (copies)."""
    S, N = arrays["pool"].shape
    pool, unit, mask, s, p, arr, n_act = _record_args(arrays, slice(0, S))
    busy = _c(arrays["gpu_busy"], np.uint8) if arrays.get("gpu_busy") is not None else None
    out = dict(
        alloc_units=np.empty((S, N), np.int32), place_node=np.empty((S, N), np.int32),
        place_off=np.empty((S, N), np.int32), act_us=np.empty((S, N), np.int64),
        total_act_us=np.empty(S, np.int64), n_selected=np.empty(S, np.int32),
        status=np.empty(S, np.int32), rounds_used=np.empty(S, np.int32),
        occupancy=np.empty((S, max_rounds, len(pools)), np.int32), pool=np.empty((S, N), np.uint8),
        traj_node=np.array(arrays["traj_node"], dtype=np.int32, order="C", copy=True),
        node_mem_free=np.array(arrays["node_mem_free"], dtype=np.int64, order="C", copy=True))
    traj, mem, last = _c(arrays["trajectory"], np.int32), _c(arrays["traj_mem"], np.uint32), _c(arrays["traj_last"], np.uint8)
    pf = _pools_flat(pools)
    rc = lib().oracle_replay_trace_pin(
        C.c_int(S), C.c_int(N), C.c_int(len(pools)), _p(pf, C.c_int), C.c_int(depth),
        C.c_int(_n_nodes(pools)), C.c_longlong(round_us), C.c_int(max_rounds),
        _p(n_act, C.c_int), _p(pool, C.c_uint8), _p(unit, C.c_uint8), _p(mask, C.c_uint32),
        _p(s, C.c_longlong), _p(p, C.c_longlong), _p(arr, C.c_longlong), _p(busy, C.c_uint8),
        _p(out["alloc_units"], C.c_int), _p(out["place_node"], C.c_int), _p(out["place_off"], C.c_int),
        _p(out["act_us"], C.c_longlong), _p(out["total_act_us"], C.c_longlong),
        _p(out["n_selected"], C.c_int), _p(out["status"], C.c_int), _p(out["occupancy"], C.c_int),
        _p(out["rounds_used"], C.c_int),
        None, None, C.c_int(0), None, None, C.c_int(0), None, None, C.c_int(policy),
        _p(traj, C.c_int), _p(mem, C.c_uint32), _p(last, C.c_uint8), C.c_int(out["traj_node"].shape[1]),
        _p(out["traj_node"], C.c_int), _p(out["node_mem_free"], C.c_longlong), _p(out["pool"], C.c_uint8))
    assert rc == 0
    return out


def _record_args(arrays, sl):
    return (_c(arrays["pool"][sl], np.uint8), _c(arrays["unit"][sl], np.uint8), _c(arrays["level_mask"][sl], np.uint32),
            _c(arrays["s_us"][sl], np.int64), _c(arrays["p_us"][sl], np.int64),
            _c(arrays["arrival_us"][sl], np.int64) if arrays.get("arrival_us") is not None else None,
            _c(arrays["n_actions"][sl], np.int32))


def order_queue(pools: Sequence, arrays: Dict[str, Optional[np.ndarray]], policy: int) -> np.ndarray:
    """Permutation [scenario][position] -> action index that sorts every queue by the policy's key
    (1: shortest least-level duration, 2: longest, 3: earliest arrival), equal keys in queue order."""
    S, N = arrays["pool"].shape
    pool, unit, mask, s, p, arr, n_act = _record_args(arrays, slice(0, S))
    perm = np.empty((S, N), np.int32)
    pf = _pools_flat(pools)
    rc = lib().oracle_order_queue(C.c_int(S), C.c_int(N), C.c_int(len(pools)), _p(pf, C.c_int), _p(n_act, C.c_int),
                                  _p(pool, C.c_uint8), _p(unit, C.c_uint8), _p(mask, C.c_uint32), _p(s, C.c_longlong),
                                  _p(p, C.c_longlong), _p(arr, C.c_longlong), C.c_int(policy), _p(perm, C.c_int))
    assert rc == 0
    return perm


def schedule_batch_ordered(pools: Sequence, arrays: Dict[str, Optional[np.ndarray]], policy: int, *, depth: int = 2,
                           now_us: int = 0) -> Dict[str, np.ndarray]:
    """One round on every queue sorted by `policy`; results at the actions' own positions."""
    S, N = arrays["pool"].shape
    pool, unit, mask, s, p, arr, n_act = _record_args(arrays, slice(0, S))
    busy = _c(arrays["gpu_busy"], np.uint8) if arrays.get("gpu_busy") is not None else None
    out = dict(
        alloc_units=np.empty((S, N), np.int32), place_node=np.empty((S, N), np.int32),
        place_off=np.empty((S, N), np.int32), act_us=np.empty((S, N), np.int64),
        total_act_us=np.empty(S, np.int64), n_selected=np.empty(S, np.int32), status=np.empty(S, np.int32))
    pf = _pools_flat(pools)
    rc = lib().oracle_schedule_batch_ordered(
        C.c_int(S), C.c_int(N), C.c_int(len(pools)), _p(pf, C.c_int), C.c_int(depth), C.c_int(_n_nodes(pools)),
        _p(n_act, C.c_int), _p(pool, C.c_uint8), _p(unit, C.c_uint8), _p(mask, C.c_uint32), _p(s, C.c_longlong),
        _p(p, C.c_longlong), _p(arr, C.c_longlong), _p(busy, C.c_uint8), C.c_longlong(now_us), C.c_int(policy),
        _p(out["alloc_units"], C.c_int), _p(out["place_node"], C.c_int), _p(out["place_off"], C.c_int),
        _p(out["act_us"], C.c_longlong), _p(out["total_act_us"], C.c_longlong), _p(out["n_selected"], C.c_int),
        _p(out["status"], C.c_int))
    assert rc == 0
    return out


def pin_trajectories(pools: Sequence, arrays: Dict[str, Optional[np.ndarray]], traj_node: np.ndarray,
                     node_mem_free: np.ndarray) -> Dict[str, np.ndarray]:
    """Pins the trajectories of every queue to CPU nodes (arrays "trajectory" int32, "traj_mem" uint32).
    Returns pool (the rewritten column), n_admitted and the updated state (copies)."""
    S, N = arrays["pool"].shape
    pool, unit, mask, s, p, arr, n_act = _record_args(arrays, slice(0, S))
    traj = _c(arrays["trajectory"], np.int32)
    mem = _c(arrays["traj_mem"], np.uint32)
    tn = np.array(traj_node, dtype=np.int32, order="C", copy=True)
    mf = np.array(node_mem_free, dtype=np.int64, order="C", copy=True)
    out = dict(pool=np.empty((S, N), np.uint8), n_admitted=np.empty(S, np.int32), traj_node=tn, node_mem_free=mf)
    pf = _pools_flat(pools)
    rc = lib().oracle_pin_trajectories(
        C.c_int(S), C.c_int(N), C.c_int(len(pools)), _p(pf, C.c_int), _p(n_act, C.c_int), _p(pool, C.c_uint8),
        _p(unit, C.c_uint8), _p(mask, C.c_uint32), _p(traj, C.c_int), _p(mem, C.c_uint32), C.c_int(tn.shape[1]),
        _p(tn, C.c_int), _p(mf, C.c_longlong), _p(out["pool"], C.c_uint8), _p(out["n_admitted"], C.c_int))
    assert rc == 0
    return out


# ------------------------------------------------------------------ single pieces
def duration(s: int, p: int, r: int) -> int:
    return int(lib().oracle_duration(int(s), int(p), int(r)))


def free_blocks(busy: Sequence[int], group: int = 8) -> np.ndarray:
    b = np.asarray(busy, dtype=np.uint8)
    F = np.zeros(4, np.int32)
    lib().oracle_free_blocks(C.c_int(len(b)), _p(b, C.c_uint8), C.c_int(group), _p(F, C.c_int))
    return F


def chunks_fit(n: Sequence[int], F: Sequence[int]) -> bool:
    n = np.asarray(n, dtype=np.int32)
    F = np.asarray(F, dtype=np.int32)
    return bool(lib().oracle_chunks_fit(_p(n, C.c_int), _p(F, C.c_int)))


def encode(n: Sequence[int], N: Sequence[int]) -> int:
    n = np.asarray(n, dtype=np.int32)
    N = np.asarray(N, dtype=np.int32)
    return int(lib().oracle_encode(_p(n, C.c_int), _p(N, C.c_int)))


def decode(j: int, N: Sequence[int]) -> np.ndarray:
    N = np.asarray(N, dtype=np.int32)
    n = np.zeros(4, np.int32)
    lib().oracle_decode(C.c_longlong(j), _p(N, C.c_int), _p(n, C.c_int))
    return n


def dp_arrange(unit, mask, s, p, *, pool_type: int, capacity: int, group: int,
               free_units: int = 0, busy: Optional[Sequence[int]] = None, prune: bool = True):
    """DPArrange for every prefix.  Returns (rc, value[m], alloc[m, m]) with alloc[q-1, :q]
    the units granted to the first q tasks; rc = 0, or the first prefix that does not fit."""
    unit = np.ascontiguousarray(unit, dtype=np.uint8)
    mask = np.ascontiguousarray(mask, dtype=np.uint32)
    s = np.ascontiguousarray(s, dtype=np.int64)
    p = np.ascontiguousarray(p, dtype=np.int64)
    m = len(unit)
    value = np.zeros(m, np.int64)
    alloc = np.zeros((m, m), np.int32)
    b = np.asarray(busy if busy is not None else [], dtype=np.uint8)
    rc = lib().oracle_dp_arrange(
        C.c_int(m), _p(unit, C.c_uint8), _p(mask, C.c_uint32), _p(s, C.c_longlong), _p(p, C.c_longlong),
        C.c_int(pool_type), C.c_int(capacity), C.c_int(group), C.c_int(free_units), C.c_int(len(b)),
        _p(b, C.c_uint8), C.c_int(1 if prune else 0), _p(value, C.c_longlong), _p(alloc, C.c_int))
    return int(rc), value, alloc


def estimate(heap: Sequence[int], unit, mask, s, p, depth: int = 2) -> int:
    heap = np.ascontiguousarray(heap, dtype=np.int64)
    unit = np.ascontiguousarray(unit, dtype=np.uint8)
    mask = np.ascontiguousarray(mask, dtype=np.uint32)
    s = np.ascontiguousarray(s, dtype=np.int64)
    p = np.ascontiguousarray(p, dtype=np.int64)
    return int(lib().oracle_estimate(
        C.c_int(len(heap)), _p(heap, C.c_longlong), C.c_int(len(unit)), _p(unit, C.c_uint8),
        _p(mask, C.c_uint32), _p(s, C.c_longlong), _p(p, C.c_longlong), C.c_int(depth)))


def chunk_alloc(busy: Sequence[int], m: int, group: int = 8):
    """Section 5.3 allocation of m GPUs; returns (rc, node, start, size, busy_after)."""
    b = np.array(busy, dtype=np.uint8)
    node, start, size = C.c_int(-1), C.c_int(-1), C.c_int(0)
    rc = lib().oracle_chunk_alloc(C.c_int(len(b)), _p(b, C.c_uint8), C.c_int(group), C.c_int(m),
                                  C.byref(node), C.byref(start), C.byref(size))
    return int(rc), node.value, start.value, size.value, b
