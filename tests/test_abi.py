"""The C-ABI shared library builds for sm_100a, loads without a GPU and exports every symbol the
header declares (no compute call is made here)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib_path():
    from paper_2601_21109_b200 import build
    return build.build()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "cwl.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(cwl_[a-z_]+)\s*\(", text)))


def test_header_declares_the_three_calls():
    names = declared_functions()
    for must in ("cwl_score_tokens", "cwl_partition", "cwl_apply"):
        assert must in names


def test_library_exports_every_declared_symbol(lib_path):
    lib = ctypes.CDLL(lib_path)
    for name in declared_functions():
        assert hasattr(lib, name), name


def test_the_test_hook_exists_in_the_test_build_only(lib_path):
    from paper_2601_21109_b200 import build
    hooks = ctypes.CDLL(build.LIB_HOOKS)
    for name in ("cwl_debug_set", "cwl_trace_set", "cwl_probe_read", "cwl_probe_read_mix"):
        assert not hasattr(ctypes.CDLL(lib_path), name), name
        assert hasattr(hooks, name), name
    for name in declared_functions():                        # and everything else as well
        assert hasattr(hooks, name), name


def test_binding_covers_the_header(lib_path):
    from paper_2601_21109_b200 import binding
    assert sorted(binding.EXPORTS) == declared_functions()
    L = binding.lib()
    assert L.cwl_version() >= 100
    assert L.cwl_status_string(0) == b"ok"
    assert binding.cwl_partition_workspace_bytes(2048, 1) > 2048 * 8
    assert binding.cwl_apply_workspace_bytes(2048, 4096, 4096, 64) >= 2048 * 64 * 2


def test_struct_layouts_match_the_header(lib_path):
    from paper_2601_21109_b200 import binding
    # cwl_policy: int32 + 8 int32 + 8 float + 7 float + 4 int32 = 28 words
    assert ctypes.sizeof(binding.CPolicy) == 28 * 4
    assert ctypes.sizeof(binding.CChunkTable) == 6 * 8 + 8


def test_argument_errors_are_reported_without_a_device(lib_path):
    from paper_2601_21109_b200 import binding
    L = binding.lib()
    # NULL pointers and bad sizes are rejected before anything touches CUDA
    assert L.cwl_score_tokens(None, 8, 4, 8, None, None) == 1
    assert L.cwl_score_tokens(None, 8, 0, 8, None, None) == 0             # nothing to do
    pol = binding.make_policy([4, 8], [1.0, 1.0], [0.5], 4, 2, 0)     # max_len < min_len
    tab = binding.CChunkTable(8, 8, 8, 8, 8, 8, 4)
    assert L.cwl_partition(8, 8, 1, 16, ctypes.byref(pol), tab, 8, 1 << 20, None, None) == 1
    null_tab = binding.CChunkTable(None, None, None, None, None, None, 0)
    assert L.cwl_apply(16, 24, 16, 16, None, 0, None, 0, 4, 24, 16, 0, null_tab, 0, 16, 16, None, 0, None, None) == 3
