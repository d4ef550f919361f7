"""Host-side checks of the C-ABI library: it builds, loads, and exports every declared symbol.
No compute call is made (there is no GPU here)."""
import ctypes
import os
import re

from paper_2608_18183_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "hbsjd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(hbsjd_[a-z_0-9]+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    path = build.build()
    assert os.path.exists(path)
    lib = ctypes.CDLL(path)
    names = _declared()
    assert {"hbsjd_create", "hbsjd_rollout", "hbsjd_round", "hbsjd_destroy"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(n for n in binding.EXPORTS) == sorted(n for n in names if n in binding.EXPORTS)
    for n in names:
        assert n in binding.EXPORTS, f"{n} is declared but not bound"


def test_binding_structs_match_header_layout():
    # sizes fixed by the header: 9 int32 + 2 float; 2 int32 + 2 float + 4 int32 + u64 + 2 int32; 8 int64 + 2 float
    assert ctypes.sizeof(binding.hbsjd_model_desc) == 44
    assert ctypes.sizeof(binding.hbsjd_params) == 48
    assert binding.hbsjd_params.seed.offset == 32
    assert ctypes.sizeof(binding.hbsjd_stats) == 72


def test_strerror_without_a_device():
    lib = binding.load()
    assert lib.hbsjd_strerror(0) == b"ok"
    assert lib.hbsjd_strerror(-1) == b"invalid argument"
    assert lib.hbsjd_strerror(-5) == b"bounded device wait gave up"
    # null arguments are rejected before any CUDA call
    assert lib.hbsjd_create(None, None, None, 0, 1, 1, None) == -1
    assert lib.hbsjd_round(None, None) == -1
    lib.hbsjd_destroy(None)
