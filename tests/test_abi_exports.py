"""The C-ABI library builds without a GPU, loads, and exports every function include/d3.h declares.
No compute call is made here."""
import ctypes
import os
import re

from paper_2601_07568_b200 import binding
from paper_2601_07568_b200 import build as d3build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions(header="d3.h"):
    src = open(os.path.join(ROOT, "include", header)).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(d3_[a-z0-9_]+)\s*\(", src)))


def test_header_functions_are_exported_and_bound():
    lib_path = d3build.build()
    L = ctypes.CDLL(lib_path)
    names = declared_functions()
    assert len(names) >= 20
    missing = [n for n in names if not hasattr(L, n)]
    assert not missing, missing
    assert sorted(binding.EXPORTS) == names
    unbound = [n for n in names if not hasattr(binding, n)]
    assert not unbound, unbound
    # the measurement / test switches of include/d3_debug.h
    dbg = [n for n in declared_functions("d3_debug.h") if n not in ("d3_tuning", "d3_ctx")]
    assert sorted(binding.DEBUG_EXPORTS) == dbg
    assert not [n for n in dbg if not hasattr(L, n) or not hasattr(binding, n)]


def test_host_only_entry_points():
    L = binding.lib()
    assert binding.d3_version().startswith("d3-b200")
    assert L.d3_strerror(0) == b"ok"
    assert L.d3_strerror(binding.D3_ERR_DEVICE_TIMEOUT) == b"bounded device-side wait gave up"
    assert L.d3_strerror(-99) == b"unknown error"
    # null arguments are rejected before any CUDA call
    assert L.d3_create(None, None, None) == binding.D3_ERR_INVALID_ARG
    assert L.d3_prefill(None, None, None, 1, 1) == binding.D3_ERR_INVALID_ARG
    assert L.d3_generate(None, 32, ctypes.c_float(0.9), 1, None, None, None) == binding.D3_ERR_INVALID_ARG


def test_error_word_to_status_mapping():
    """Host side of the give-up path: the status a call returns for a device error word."""
    assert binding.d3_status_of_error_word(0) == binding.D3_OK
    assert binding.d3_status_of_error_word(1) == binding.D3_ERR_DEVICE_TIMEOUT
    for other in (2, 4, 8, 16, 2 | 4):
        assert binding.d3_status_of_error_word(other) == binding.D3_ERR_INVALID_ARG
    # the time-out bit wins over the others
    assert binding.d3_status_of_error_word(1 | 2 | 16) == binding.D3_ERR_DEVICE_TIMEOUT


def test_tuning_defaults_and_ranges():
    t = binding.d3_tuning_defaults()
    assert (t.ring_kb, t.ctas_per_sm, t.producers, t.tile_columns, t.attn_key_tiles) == (0, 0, 0, 0, 0)
    assert (t.cluster_k_split, t.row_tile_pairs, t.round_robin, t.column_strips, t.strip_stages, t.chain) == (-1, -1, 1, 0, 0, -1)
    assert ctypes.sizeof(binding.d3_tuning) == 16 * 4 and t.attention_tmem == -1 and t.cta_pairs == -1 and t.chain_clusters == 0 and t.chain_l2_ahead == -1 and t.weights_as_rows == -1
    assert binding.lib().d3_set_tuning(None, ctypes.byref(t)) == binding.D3_ERR_INVALID_ARG


def test_struct_layouts_match_header():
    # 8 int32 + 3 float + 7 int32 = 18 four-byte fields; 12 pointers; 6 int64 + 2 float
    assert ctypes.sizeof(binding.d3_config) == 18 * 4
    assert ctypes.sizeof(binding.d3_weights) == 12 * ctypes.sizeof(ctypes.c_void_p)
    assert ctypes.sizeof(binding.d3_stats) == 6 * 8 + 2 * 4
