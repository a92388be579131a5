"""The C-ABI library builds, loads without a GPU and exports every symbol the header declares."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "tangram.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(tangram_[a-z_]+)\s*\(", text)))


def test_header_declares_the_three_entry_points():
    names = _declared()
    for n in ("tangram_round_create", "tangram_schedule_batch", "tangram_replay_trace", "tangram_round_destroy"):
        assert n in names


def test_library_exports_every_declared_symbol():
    from paper_2603_13019_b200 import build
    path = build.build()
    lib = ctypes.CDLL(path)
    for n in _declared():
        assert hasattr(lib, n), n


def test_binding_lists_the_same_symbols():
    from paper_2603_13019_b200 import binding, build
    build.build()
    assert sorted(binding.EXPORTS) == _declared()
    lib = binding.load_library()
    assert lib.tangram_strerror(0) == b"ok" and lib.tangram_strerror(-1) == b"invalid argument"


# ---------------------------------------------------------------- argument validation on the host
# Every rejected call below returns before the library touches CUDA, so this runs without a GPU.
def _desc(binding, pools, **kw):
    arr = (binding._PoolDesc * max(len(pools), 1))(*[binding._PoolDesc(*p) for p in pools])
    d = binding._RoundDesc(kw.get("n_scenarios", 4), kw.get("max_actions", 16), kw.get("n_pools", len(pools)),
                           kw.get("depth", 2), kw.get("round_us", 10_000), kw.get("max_rounds", 0),
                           kw.get("host_buffers", 0), kw.get("workspace_bytes", 0), kw.get("slot_wait_us", 0),
                           kw.get("cache_slots", 0), kw.get("side_costs", 0), arr)
    return d, arr


def test_round_create_rejects_bad_descriptions():
    from paper_2603_13019_b200 import binding, build
    build.build()
    lib = binding.load_library()
    EINVAL = -1
    out = ctypes.c_void_p()
    good = [(0, 64, 8, 0), (1, 16, 8, 0), (2, 10, 0, 1_000_000)]

    def create(pools, **kw):
        d, keep = _desc(binding, pools, **kw)
        return lib.tangram_round_create(ctypes.byref(d), ctypes.byref(out))

    assert lib.tangram_round_create(None, ctypes.byref(out)) == EINVAL            # null description
    d, keep = _desc(binding, good)
    assert lib.tangram_round_create(ctypes.byref(d), None) == EINVAL              # null result slot
    d.pools = ctypes.cast(None, ctypes.POINTER(binding._PoolDesc))
    assert lib.tangram_round_create(ctypes.byref(d), ctypes.byref(out)) == EINVAL  # null pool array
    assert create(good, n_pools=0) == EINVAL
    assert create([(0, 8, 8, 0)] * 9, n_pools=9) == EINVAL                         # more than TANGRAM_MAX_POOLS
    assert create(good, n_scenarios=0) == EINVAL
    assert create(good, max_actions=0) == EINVAL
    assert create(good, depth=0) == EINVAL
    assert create(good, depth=33) == EINVAL
    assert create(good, max_rounds=-1) == EINVAL
    assert create(good, workspace_bytes=-1) == EINVAL
    assert create(good, slot_wait_us=-1) == EINVAL
    assert create(good, cache_slots=5) == EINVAL
    assert create(good, cache_slots=1, host_buffers=1) == EINVAL                    # no service cache through host buffers
    assert create(good, side_costs=3) == EINVAL and create(good, side_costs=-1) == EINVAL
    assert create(good, side_costs=1, host_buffers=1) == EINVAL                     # no cost vectors through host buffers
    assert create(good, n_scenarios=1 << 20, max_actions=1 << 12) == EINVAL         # more than 2^31 records
    assert create([(1, 24, 3, 0)]) == EINVAL                                        # nodes of 3 GPUs
    assert create([(1, 20, 8, 0)]) == EINVAL                                        # capacity not whole nodes
    assert create([(0, 70, 8, 0)]) == EINVAL                                        # capacity not whole NUMA domains
    assert create([(0, 64, 0, 0)]) == EINVAL                                        # NUMA domain of 0 cores
    assert create([(0, 0, 8, 0)]) == EINVAL                                         # empty pool
    assert create([(3, 8, 8, 0)]) == EINVAL                                         # unknown pool type
    assert create([(2, 10, 0, -5)]) == EINVAL                                       # negative quota window
    assert out.value is None                                                        # never set on failure


def test_calls_reject_null_handles_and_buffers():
    from paper_2603_13019_b200 import binding, build
    build.build()
    lib = binding.load_library()
    EINVAL = -1
    a, r = binding._Actions(), binding._Result()
    assert lib.tangram_schedule_batch(None, ctypes.byref(a), 0, ctypes.byref(r), None) == EINVAL
    assert lib.tangram_replay_trace(None, ctypes.byref(a), ctypes.byref(r), None) == EINVAL
    assert lib.tangram_set_profiling(None, 1) == EINVAL
    assert lib.tangram_kernel_launches(None) == 0
    assert lib.tangram_kernel_name(-1) == b"" and lib.tangram_kernel_name(0) != b""
    lib.tangram_round_destroy(None)                                                 # a no-op
    pin = binding._Pinning()
    assert lib.tangram_order_queue(None, ctypes.byref(a), 1, None, None) == EINVAL
    assert lib.tangram_schedule_batch_ordered(None, ctypes.byref(a), 1, 0, ctypes.byref(r), None) == EINVAL
    assert lib.tangram_pin_trajectories(None, ctypes.byref(a), ctypes.byref(pin), None) == EINVAL
    assert lib.tangram_replay_trace_ordered(None, ctypes.byref(a), 1, ctypes.byref(r), None) == EINVAL
    assert lib.tangram_replay_trace_pinned(None, ctypes.byref(a), 0, ctypes.byref(pin), ctypes.byref(r), None) == EINVAL
    # the allocation-free entry point validates its description and buffers the same way
    d, keep = _desc(binding, [(0, 64, 8, 0)])
    assert lib.tangram_schedule_batch_static(None, ctypes.byref(a), 0, ctypes.byref(r), None) == EINVAL
    assert lib.tangram_schedule_batch_static(ctypes.byref(d), ctypes.byref(a), 0, ctypes.byref(r), None) == EINVAL  # null buffers
    assert lib.tangram_strerror(-4) != lib.tangram_strerror(-99)
