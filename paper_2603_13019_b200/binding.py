"""ctypes binding of libtangram.so: the same calls as include/tangram.h, with torch tensors
(device memory, or pinned host memory in host-buffer mode) marshalled to raw pointers.

There is no fallback: without the compiled CUDA library every call raises.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Dict, Optional, Sequence

POOL_CPU, POOL_GPU, POOL_API = 0, 1, 2
UNIT_GANG = 0x80
STATUS_OK, STATUS_BAD_ACTION, STATUS_UNSORTED, STATUS_WORKSPACE = 0, 1, 2, 4

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libtangram.so")
_lib = None


class TangramError(RuntimeError):
    pass


class _PoolDesc(C.Structure):
    _fields_ = [("type", C.c_int32), ("capacity", C.c_int32), ("group", C.c_int32), ("window_us", C.c_int32)]


class _RoundDesc(C.Structure):
    _fields_ = [("n_scenarios", C.c_int32), ("max_actions", C.c_int32), ("n_pools", C.c_int32),
                ("depth", C.c_int32), ("round_us", C.c_int64), ("max_rounds", C.c_int32),
                ("host_buffers", C.c_int32), ("workspace_bytes", C.c_int64), ("slot_wait_us", C.c_int64),
                ("cache_slots", C.c_int32), ("side_costs", C.c_int32), ("pools", C.POINTER(_PoolDesc))]


class _Actions(C.Structure):
    _fields_ = [("pool", C.c_void_p), ("unit", C.c_void_p), ("level_mask", C.c_void_p), ("s_us", C.c_void_p),
                ("p_us", C.c_void_p), ("arrival_us", C.c_void_p), ("n_actions", C.c_void_p),
                ("gpu_busy", C.c_void_p), ("service", C.c_void_p), ("restore_us", C.c_void_p),
                ("gpu_cache_tag", C.c_void_p), ("gpu_cache_use", C.c_void_p),
                ("side_pool", C.c_void_p), ("side_units", C.c_void_p)]


class _Pinning(C.Structure):
    _fields_ = [("trajectory", C.c_void_p), ("traj_mem", C.c_void_p), ("max_trajectories", C.c_int32),
                ("traj_node", C.c_void_p), ("node_mem_free", C.c_void_p), ("pool_out", C.c_void_p),
                ("n_admitted", C.c_void_p), ("traj_last", C.c_void_p)]


class _Result(C.Structure):
    _fields_ = [("alloc_units", C.c_void_p), ("place_node", C.c_void_p), ("place_off", C.c_void_p),
                ("act_us", C.c_void_p), ("total_act_us", C.c_void_p), ("n_selected", C.c_void_p),
                ("status", C.c_void_p), ("occupancy", C.c_void_p), ("rounds_used", C.c_void_p)]


EXPORTS = ("tangram_round_create", "tangram_schedule_batch", "tangram_replay_trace",
           "tangram_round_destroy", "tangram_kernel_launches", "tangram_strerror",
           "tangram_last_cuda_error", "tangram_set_profiling", "tangram_kernel_time_ms",
           "tangram_kernel_name", "tangram_schedule_batch_static", "tangram_order_queue",
           "tangram_schedule_batch_ordered", "tangram_pin_trajectories", "tangram_replay_trace_ordered", "tangram_replay_trace_pinned")


def load_library(path: Optional[str] = None):
    """dlopen the CUDA library (built in-tree by paper_2603_13019_b200.build)."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or _LIB_PATH
    if not os.path.exists(p):
        raise TangramError(f"{p} is missing: build it with `python -m paper_2603_13019_b200.build` "
                           "(there is no CPU fallback)")
    lib = C.CDLL(p)
    lib.tangram_round_create.restype = C.c_int
    lib.tangram_round_create.argtypes = [C.POINTER(_RoundDesc), C.POINTER(C.c_void_p)]
    lib.tangram_schedule_batch.restype = C.c_int
    lib.tangram_schedule_batch.argtypes = [C.c_void_p, C.POINTER(_Actions), C.c_int64, C.POINTER(_Result), C.c_void_p]
    lib.tangram_replay_trace.restype = C.c_int
    lib.tangram_replay_trace.argtypes = [C.c_void_p, C.POINTER(_Actions), C.POINTER(_Result), C.c_void_p]
    lib.tangram_round_destroy.restype = None
    lib.tangram_round_destroy.argtypes = [C.c_void_p]
    lib.tangram_kernel_launches.restype = C.c_int64
    lib.tangram_kernel_launches.argtypes = [C.c_void_p]
    lib.tangram_strerror.restype = C.c_char_p
    lib.tangram_strerror.argtypes = [C.c_int]
    lib.tangram_last_cuda_error.restype = C.c_char_p
    lib.tangram_set_profiling.restype = C.c_int
    lib.tangram_set_profiling.argtypes = [C.c_void_p, C.c_int]
    lib.tangram_kernel_time_ms.restype = C.c_int
    lib.tangram_kernel_time_ms.argtypes = [C.c_void_p, C.c_int, C.POINTER(C.c_double), C.POINTER(C.c_int64)]
    lib.tangram_kernel_name.restype = C.c_char_p
    lib.tangram_kernel_name.argtypes = [C.c_int]
    lib.tangram_schedule_batch_static.restype = C.c_int
    lib.tangram_order_queue.restype = C.c_int
    lib.tangram_order_queue.argtypes = [C.c_void_p, C.POINTER(_Actions), C.c_int, C.c_void_p, C.c_void_p]
    lib.tangram_schedule_batch_ordered.restype = C.c_int
    lib.tangram_schedule_batch_ordered.argtypes = [C.c_void_p, C.POINTER(_Actions), C.c_int, C.c_int64,
                                                   C.POINTER(_Result), C.c_void_p]
    lib.tangram_replay_trace_ordered.restype = C.c_int
    lib.tangram_replay_trace_ordered.argtypes = [C.c_void_p, C.POINTER(_Actions), C.c_int, C.POINTER(_Result), C.c_void_p]
    lib.tangram_replay_trace_pinned.restype = C.c_int
    lib.tangram_replay_trace_pinned.argtypes = [C.c_void_p, C.POINTER(_Actions), C.c_int, C.POINTER(_Pinning),
                                                C.POINTER(_Result), C.c_void_p]
    lib.tangram_pin_trajectories.restype = C.c_int
    lib.tangram_pin_trajectories.argtypes = [C.c_void_p, C.POINTER(_Actions), C.POINTER(_Pinning), C.c_void_p]
    lib.tangram_schedule_batch_static.argtypes = [C.POINTER(_RoundDesc), C.POINTER(_Actions), C.c_int64,
                                                  C.POINTER(_Result), C.c_void_p]
    if path is None:
        _lib = lib
    return lib


@dataclass(frozen=True)
class PoolDesc:
    type: int
    capacity: int
    group: int
    window_us: int = 0


def _dtypes():
    import torch
    ins = dict(pool=torch.uint8, unit=torch.uint8, level_mask=torch.int32, s_us=torch.int64,
               p_us=torch.int64, arrival_us=torch.int64, n_actions=torch.int32, gpu_busy=torch.uint8,
               service=torch.int16, restore_us=torch.int64, cache_tag=torch.int32, cache_use=torch.int64,
               side_pool=torch.uint8, side_units=torch.int16)
    outs = dict(alloc_units=torch.int32, place_node=torch.int32, place_off=torch.int32,
                act_us=torch.int64, total_act_us=torch.int64, n_selected=torch.int32,
                status=torch.int32, occupancy=torch.int32, rounds_used=torch.int32)
    return ins, outs


def _check(rc: int):
    if rc != 0:
        lib = load_library()
        msg = lib.tangram_strerror(rc).decode()
        detail = lib.tangram_last_cuda_error().decode()
        raise TangramError(f"tangram call failed: {msg}" + (f" ({detail})" if detail else ""))


class Round:
    """Owner of a tangram_round handle (device workspace)."""

    def __init__(self, n_scenarios: int, max_actions: int, pools: Sequence, *, depth: int = 2,
                 round_us: int = 10_000, max_rounds: int = 0, host_buffers: bool = False,
                 workspace_bytes: int = 0, slot_wait_us: int = 0, cache_slots: int = 0, side_costs: int = 0):
        self._lib = load_library()
        self._h = None
        self.n_scenarios, self.max_actions, self.pools = int(n_scenarios), int(max_actions), tuple(pools)
        self.max_rounds, self.host_buffers = int(max_rounds), bool(host_buffers)
        self.cache_slots = int(cache_slots)
        self.side_costs = int(side_costs)
        arr = (_PoolDesc * len(pools))(*[_PoolDesc(p.type, p.capacity, p.group, p.window_us) for p in pools])
        desc = _RoundDesc(n_scenarios, max_actions, len(pools), depth, round_us, max_rounds,
                          1 if host_buffers else 0, workspace_bytes, slot_wait_us, cache_slots, side_costs, arr)
        h = C.c_void_p()
        _check(self._lib.tangram_round_create(C.byref(desc), C.byref(h)))
        self._h = h

    # -- marshalling ---------------------------------------------------------------
    def _ptr(self, name: str, t, dtype, numel: Optional[int]):
        if t is None:
            return None
        if t.dtype != dtype:
            raise TangramError(f"{name}: expected {dtype}, got {t.dtype}")
        if not t.is_contiguous():
            raise TangramError(f"{name}: tensor must be contiguous")
        if self.host_buffers == t.is_cuda:
            raise TangramError(f"{name}: tensor must be on the {'host' if self.host_buffers else 'device'}")
        if numel is not None and t.numel() != numel:
            raise TangramError(f"{name}: expected {numel} elements, got {t.numel()}")
        return t.data_ptr()

    def _actions(self, a: Dict) -> _Actions:
        ins, _ = _dtypes()
        SN = self.n_scenarios * self.max_actions
        nodes = sum(p.capacity // p.group for p in self.pools if p.type == POOL_GPU)
        ncache = self.n_scenarios * nodes * 8 * self.cache_slots
        sizes = dict(pool=SN, unit=SN, level_mask=SN, s_us=SN, p_us=SN, arrival_us=SN,
                     n_actions=self.n_scenarios, gpu_busy=self.n_scenarios * nodes,
                     service=SN, restore_us=SN, cache_tag=ncache, cache_use=ncache,
                     side_pool=SN * self.side_costs, side_units=SN * self.side_costs)
        # the cache and cost-vector columns are only handed over when the round was created with them
        off = set()
        if self.cache_slots == 0:
            off |= {"service", "restore_us", "cache_tag", "cache_use"}
        if self.side_costs == 0:
            off |= {"side_pool", "side_units"}
        return _Actions(*[self._ptr(k, None if k in off else a.get(k), ins[k], sizes[k]) for k in
                          ("pool", "unit", "level_mask", "s_us", "p_us", "arrival_us", "n_actions", "gpu_busy",
                           "service", "restore_us", "cache_tag", "cache_use", "side_pool", "side_units")])

    def new_result(self, replay: bool = False) -> Dict:
        """Output tensors of the right shapes (device, or pinned host in host-buffer mode)."""
        import torch
        _, outs = _dtypes()
        S, N = self.n_scenarios, self.max_actions
        kw = dict(pin_memory=True) if self.host_buffers else dict(device="cuda")
        shapes = dict(alloc_units=(S, N), place_node=(S, N), place_off=(S, N), act_us=(S, N),
                      total_act_us=(S,), n_selected=(S,), status=(S,))
        if replay:
            shapes.update(occupancy=(S, self.max_rounds, len(self.pools)), rounds_used=(S,))
        return {k: torch.empty(shp, dtype=outs[k], **kw) for k, shp in shapes.items()}

    def _result(self, r: Dict) -> _Result:
        _, outs = _dtypes()
        S, N = self.n_scenarios, self.max_actions
        sizes = dict(alloc_units=S * N, place_node=S * N, place_off=S * N, act_us=S * N, total_act_us=S,
                     n_selected=S, status=S, occupancy=S * self.max_rounds * len(self.pools), rounds_used=S)
        return _Result(*[self._ptr(k, r.get(k), outs[k], sizes[k]) for k in
                         ("alloc_units", "place_node", "place_off", "act_us", "total_act_us", "n_selected",
                          "status", "occupancy", "rounds_used")])

    @staticmethod
    def _stream(stream) -> int:
        import torch
        if stream is None:
            stream = torch.cuda.current_stream()
        return int(stream.cuda_stream)

    # -- the calls --------------------------------------------------------------------
    def schedule_batch(self, actions: Dict, now_us: int = 0, result: Optional[Dict] = None, stream=None) -> Dict:
        """tangram_schedule_batch: one round for every scenario, asynchronous on `stream`."""
        result = self.new_result() if result is None else result
        a, r = self._actions(actions), self._result(result)
        _check(self._lib.tangram_schedule_batch(self._h, C.byref(a), int(now_us), C.byref(r), self._stream(stream)))
        return result

    def replay_trace(self, actions: Dict, result: Optional[Dict] = None, stream=None, policy: int = 0) -> Dict:
        """tangram_replay_trace (policy 0) / tangram_replay_trace_ordered: device-resident replay of every
        scenario's arrival trace."""
        result = self.new_result(replay=True) if result is None else result
        a, r = self._actions(actions), self._result(result)
        if policy:
            _check(self._lib.tangram_replay_trace_ordered(self._h, C.byref(a), int(policy), C.byref(r), self._stream(stream)))
        else:
            _check(self._lib.tangram_replay_trace(self._h, C.byref(a), C.byref(r), self._stream(stream)))
        return result

    def order_queue(self, actions: Dict, policy: int, stream=None):
        """tangram_order_queue: the permutation that sorts every queue by the policy's key (device int32 [S][N])."""
        import torch
        perm = torch.empty((self.n_scenarios, self.max_actions), dtype=torch.int32, device="cuda")
        a = self._actions(actions)
        _check(self._lib.tangram_order_queue(self._h, C.byref(a), int(policy), C.c_void_p(perm.data_ptr()),
                                             self._stream(stream)))
        return perm

    def schedule_batch_ordered(self, actions: Dict, policy: int, now_us: int = 0, result: Optional[Dict] = None,
                               stream=None) -> Dict:
        """tangram_schedule_batch_ordered: one round on every queue sorted by `policy`."""
        result = self.new_result() if result is None else result
        a, r = self._actions(actions), self._result(result)
        _check(self._lib.tangram_schedule_batch_ordered(self._h, C.byref(a), int(policy), int(now_us), C.byref(r),
                                                        self._stream(stream)))
        return result

    def pin_trajectories(self, actions: Dict, stream=None) -> Dict:
        """tangram_pin_trajectories: actions["trajectory"] (int32), ["traj_mem"] (int32 bit pattern of uint32),
        state ["traj_node"] (int32 [S][T]) and ["node_mem_free"] (int64 [S][P]) are updated in place; returns
        the rewritten pool column and n_admitted (device tensors)."""
        import torch
        S, N = self.n_scenarios, self.max_actions
        T = actions["traj_node"].shape[1]
        out = dict(pool=torch.empty((S, N), dtype=torch.uint8, device="cuda"),
                   n_admitted=torch.empty((S,), dtype=torch.int32, device="cuda"))
        pin = _Pinning(self._ptr("trajectory", actions["trajectory"], torch.int32, S * N),
                       self._ptr("traj_mem", actions["traj_mem"], torch.int32, S * N), T,
                       self._ptr("traj_node", actions["traj_node"], torch.int32, S * T),
                       self._ptr("node_mem_free", actions["node_mem_free"], torch.int64, S * len(self.pools)),
                       out["pool"].data_ptr(), out["n_admitted"].data_ptr(), None)
        a = self._actions(actions)
        _check(self._lib.tangram_pin_trajectories(self._h, C.byref(a), C.byref(pin), self._stream(stream)))
        return out

    def replay_trace_pinned(self, actions: Dict, policy: int = 0, result: Optional[Dict] = None, stream=None) -> Dict:
        """tangram_replay_trace_pinned: the replay with trajectories pinned as their actions arrive
        (actions["trajectory"], ["traj_mem"], ["traj_last"] uint8; state ["traj_node"], ["node_mem_free"] updated
        in place).  The result gets "pool": the pool every action ran or waits on."""
        import torch
        S, N = self.n_scenarios, self.max_actions
        T = actions["traj_node"].shape[1]
        result = self.new_result(replay=True) if result is None else result
        result["pool"] = torch.empty((S, N), dtype=torch.uint8, device="cuda")
        pin = _Pinning(self._ptr("trajectory", actions["trajectory"], torch.int32, S * N),
                       self._ptr("traj_mem", actions["traj_mem"], torch.int32, S * N), T,
                       self._ptr("traj_node", actions["traj_node"], torch.int32, S * T),
                       self._ptr("node_mem_free", actions["node_mem_free"], torch.int64, S * len(self.pools)),
                       result["pool"].data_ptr(), None,
                       self._ptr("traj_last", actions.get("traj_last"), torch.uint8, S * N))
        a, r = self._actions(actions), self._result(result)
        _check(self._lib.tangram_replay_trace_pinned(self._h, C.byref(a), int(policy), C.byref(pin), C.byref(r),
                                                     self._stream(stream)))
        return result

    def set_profiling(self, enable: bool):
        """tangram_set_profiling: record CUDA events around every kernel of the following calls."""
        _check(self._lib.tangram_set_profiling(self._h, 1 if enable else 0))

    def kernel_times(self) -> Dict[str, tuple]:
        """tangram_kernel_time_ms for every kernel: name -> (total ms, launches).  Synchronise first."""
        out = {}
        for k in range(8):
            ms, n = C.c_double(0.0), C.c_int64(0)
            _check(self._lib.tangram_kernel_time_ms(self._h, k, C.byref(ms), C.byref(n)))
            out[self._lib.tangram_kernel_name(k).decode()] = (ms.value, n.value)
        return out

    @property
    def kernel_launches(self) -> int:
        return int(self._lib.tangram_kernel_launches(self._h))

    def destroy(self):
        if getattr(self, "_h", None):
            self._lib.tangram_round_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def round_create(n_scenarios: int, max_actions: int, pools: Sequence, **kw) -> Round:
    """tangram_round_create."""
    return Round(n_scenarios, max_actions, pools, **kw)


def to_device(arrays: Dict, device: str = "cuda", pin: bool = False) -> Dict:
    """numpy input arrays -> torch tensors (device memory, or pinned host memory)."""
    import numpy as np
    import torch
    out = {}
    for k, v in arrays.items():
        if v is None:
            out[k] = None
            continue
        if v.dtype == np.uint32:
            v = v.view(np.int32)
        if v.dtype == np.uint16:
            v = v.view(np.int16)
        t = torch.from_numpy(np.ascontiguousarray(v))
        out[k] = t.pin_memory() if pin else t.to(device)
    return out


STATIC_SCRATCH_BYTES = 32 << 20


def schedule_batch_static(pools: Sequence, actions: Dict, result: Dict, *, depth: int = 2, now_us: int = 0,
                          stream=None) -> int:
    """tangram_schedule_batch_static: one round without a Round object and without any device
    allocation by the library -- for callers that may not call cudaMalloc (their framework owns
    all device memory, or an allocation's implicit synchronisation is unacceptable).  `actions`
    and `result` are caller-owned DEVICE tensors shaped like those of Round.schedule_batch.
    The library's scratch is a fixed 32 MiB array inside the library image, shared by all calls:
    serialise calls that could overlap on the GPU, and make the first call on a device outside
    stream capture.  Returns the C return code (0, or -4 when the batch is too large for the
    array) instead of raising, so that callers can fall back to a Round."""
    lib = load_library()
    ins, outs = _dtypes()
    S, N = actions["pool"].shape
    arr = (_PoolDesc * len(pools))(*[_PoolDesc(p.type, p.capacity, p.group, p.window_us) for p in pools])
    desc = _RoundDesc(S, N, len(pools), depth, 0, 0, 0, 0, 0, 0, 0, arr)

    def ptr(t):
        return None if t is None else t.data_ptr()

    for k, t in list(actions.items()) + list(result.items()):
        if t is not None and not (t.is_cuda and t.is_contiguous()):
            raise TangramError(f"{k}: a contiguous device tensor is required")
    a = _Actions(*([ptr(actions.get(k)) for k in
                    ("pool", "unit", "level_mask", "s_us", "p_us", "arrival_us", "n_actions", "gpu_busy")] + [None] * 6))
    r = _Result(*[ptr(result.get(k)) for k in
                  ("alloc_units", "place_node", "place_off", "act_us", "total_act_us", "n_selected", "status",
                   "occupancy", "rounds_used")])
    return int(lib.tangram_schedule_batch_static(C.byref(desc), C.byref(a), int(now_us), C.byref(r),
                                                 Round._stream(stream)))
