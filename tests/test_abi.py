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
