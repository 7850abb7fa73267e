"""CPU-only checks of the C-ABI library: it loads, exports what gs.h declares, its host
function agrees with the oracle, and argument errors come back as status codes."""
import ctypes
import re
from pathlib import Path

import numpy as np
import pytest

from oracle import gs_oracle as O
from paper_2407_15452_b200 import binding as B
from tests.helpers import pack_alias, unpack_alias

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module")
def lib():
    from paper_2407_15452_b200.build import build_library
    build_library()
    return B.lib()


def test_library_exports_every_declared_symbol(lib):
    header = (ROOT / "include" / "gs.h").read_text()
    declared = set(re.findall(r"GS_API\s+[\w\s\*]+?\b(gs_\w+)\s*\(", header))
    assert len(declared) >= 12
    assert declared == set(B.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_struct_layouts_match_header():
    assert ctypes.sizeof(B.SgnsConfig) == 10 * 4 + 3 * 8 + 3 * 8 + 8 + 8 + 2 * 4 + 4 * 4 + 8 + 6 * 8
    assert ctypes.sizeof(B.EpochStats) == 8 + 5 * 8 + 4 * 4 + 8      # loss, 5 counters, 4 times, refused ids


@pytest.mark.parametrize("power", [0.75, 1.0, 0.0])
def test_host_alias_builder_matches_oracle_bit_for_bit(lib, power):
    rng = np.random.default_rng(3)
    w = rng.pareto(1.1, size=20000) + 0.01
    w[rng.integers(0, 20000, 500)] = 0.0
    table = B.gs_build_alias(w, power)
    thr, alias = O.build_alias(w, power)
    assert np.array_equal(table, pack_alias(thr, alias))
    t2, a2 = unpack_alias(table)
    assert np.array_equal(t2, thr) and np.array_equal(a2, alias)


def test_host_alias_builder_rejects_bad_input(lib):
    with pytest.raises(B.GsError) as e:
        B.gs_build_alias(np.zeros(5), 0.75)
    assert e.value.status == -1 and "positive" in str(e.value)
    with pytest.raises(B.GsError):
        B.gs_build_alias(np.array([1.0, -2.0]), 0.75)
    with pytest.raises(B.GsError):
        B.gs_build_alias(np.array([1.0, np.nan]), 0.75)


def test_host_keep_thresholds_match_oracle_bit_for_bit(lib):
    rng = np.random.default_rng(5)
    w = rng.pareto(1.1, size=30000) + 0.01
    w[rng.integers(0, 30000, 300)] = 0.0
    for t in (1e-3, 1e-5, 1e-7):
        got = B.gs_build_keep_thresholds(w, t)
        want = O.keep_thresholds(w, t)
        assert np.array_equal(got, want)
        assert (got == 0xFFFFFFFF).any() and (got != 0xFFFFFFFF).any()
    with pytest.raises(B.GsError):
        B.gs_build_keep_thresholds(np.zeros(4), 1e-3)
    with pytest.raises(B.GsError):
        B.gs_build_keep_thresholds(np.ones(4), 0.0)


def test_argument_errors_are_status_codes_without_touching_a_gpu(lib):
    h = ctypes.c_void_p(0)
    st = lib.gs_graph_load_csr(ctypes.c_int64(0), ctypes.c_int64(0), None, 0, None, 0, None,
                               ctypes.byref(h))
    assert st == -1 and not h.value and b"n_nodes" in lib.gs_last_error()
    st = lib.gs_graph_load_csr(ctypes.c_int64(4), ctypes.c_int64(1 << 31), ctypes.c_void_p(16), 0,
                               ctypes.c_void_p(16), 0, None, ctypes.byref(h))
    assert st == -1 and b"int32 offsets" in lib.gs_last_error()
    st = lib.gs_sgns_step(None, None, ctypes.c_int64(1), 128, None, ctypes.c_int64(0),
                          ctypes.c_int64(0), 4, 2, 1, None, ctypes.c_float(0.1), ctypes.c_uint64(0),
                          0, None, None, None, None, None)
    assert st == -1
    st = lib.gs_sgns_step(ctypes.c_void_p(256), ctypes.c_void_p(512), ctypes.c_int64(10), 100,
                          ctypes.c_void_p(16), ctypes.c_int64(1), ctypes.c_int64(0), 4, 2, 1,
                          ctypes.c_void_p(16), ctypes.c_float(0.1), ctypes.c_uint64(0), 0,
                          None, None, None, None, None)
    assert st == -6 and b"dim" in lib.gs_last_error()
    st = lib.gs_random_walks(None, None, ctypes.c_int64(1), ctypes.c_int64(0), 4,
                             ctypes.c_uint64(0), None, None, None)
    assert st == -1
    st = lib.gs_shuffled_starts(ctypes.c_int64(0), ctypes.c_uint64(1), ctypes.c_uint32(0),
                                ctypes.c_int64(0), ctypes.c_int64(4), ctypes.c_void_p(16), None)
    assert st == -1 and b"n_nodes" in lib.gs_last_error()
    st = lib.gs_subsample_walks(ctypes.c_void_p(16), ctypes.c_int64(2), ctypes.c_int64(0), 2000,
                                ctypes.c_void_p(16), ctypes.c_int64(5), ctypes.c_uint64(0),
                                ctypes.c_void_p(16), None, None)
    assert st == -6 and b"walk_len" in lib.gs_last_error()
    p16 = ctypes.c_void_p(256)
    st = lib.gs_sgns_step_adam(p16, p16, p16, p16, p16, p16, ctypes.c_int64(10), 128, p16,
                               ctypes.c_int64(1), ctypes.c_int64(0), 4, 2, 1, p16, ctypes.c_float(0.1),
                               ctypes.c_float(0.9), ctypes.c_float(0.999), ctypes.c_float(1e-8),
                               ctypes.c_int64(0), ctypes.c_uint64(0), 0, None, None, None)
    assert st == -1 and b"step" in lib.gs_last_error()
    assert lib.gs_tune_node2vec_group(3) == -1
    assert lib.gs_tune_node2vec_group(1) == 0
    assert lib.gs_tune_node2vec_group(0) == 0
    lib.gs_graph_free(None)
