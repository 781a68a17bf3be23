"""Host-side checks that need no GPU: the library loads, exports every declared symbol, and rejects
malformed circuits before touching a device."""
import os
import re

import numpy as np
import pytest

from paper_2502_01681_b200 import dg4

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "dg4.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dg4_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = dg4.load()
    names = _declared_symbols()
    assert len(names) >= 14
    for name in names:
        assert hasattr(lib, name), name
    assert set(names) == set(dg4.EXPORTS)


def test_status_strings():
    lib = dg4.load()
    seen = {lib.dg4_status_string(s).decode() for s in range(0, -9, -1)}
    assert len(seen) == 9 and "unknown status" not in seen
    assert lib.dg4_status_string(-99).decode() == "unknown status"


@pytest.mark.parametrize("row_ptr,col_idx,level,hops,chunk,status", [
    ([1, 1, 2], [0], [0, 1], 1, 0, dg4.DG4_ERR_NOT_SORTED),            # does not start at 0
    ([0, 0, 2, 1], [0, 0], [0, 1, 2], 1, 0, dg4.DG4_ERR_NOT_SORTED),   # decreasing
    ([0, 0, 0, 0, 3], [0, 1, 2], [0, 0, 0, 1], 1, 0, dg4.DG4_ERR_BAD_DEGREE),
    ([0, 0, 1], [0], [0, 0], 1, 0, dg4.DG4_ERR_BAD_LEVEL),             # level does not increase
    ([0, 0, 1], [1], [0, 1], 1, 0, dg4.DG4_ERR_BAD_LEVEL),             # self loop
    ([0, 0, 1], [5], [0, 1], 1, 0, dg4.DG4_ERR_BAD_LEVEL),             # source out of range
    ([0, 0, 1], [0], [-1, 1], 1, 0, dg4.DG4_ERR_BAD_LEVEL),
    ([0, 0, 1], [0], [0, 1], 9, 0, dg4.DG4_ERR_UNSUPPORTED),
    ([0, 0, 1], [0], [0, 1], 0, 0, dg4.DG4_ERR_UNSUPPORTED),
    ([0, 0, 1], [0], [0, 1], 1, 100, dg4.DG4_ERR_INVALID_ARG),         # chunk not a multiple of 1024
])
def test_graph_create_rejects_malformed_circuits(row_ptr, col_idx, level, hops, chunk, status):
    with pytest.raises(dg4.Dg4Error) as e:
        dg4.dg4_graph_create(np.array(row_ptr), np.array(col_idx), np.array(level), hops, chunk)
    assert e.value.status == status
    assert e.value.detail


def test_null_handles_are_rejected_not_dereferenced():
    lib = dg4.load()
    assert lib.dg4_graph_destroy(None) == dg4.DG4_OK
    assert lib.dg4_graph_info(None, None) == dg4.DG4_ERR_INVALID_ARG
    assert lib.dg4_graph_rebuild(None, None) == dg4.DG4_ERR_INVALID_ARG
    assert lib.dg4_layer_workspace_bytes(None, None) == 0
    assert not lib.dg4_graph_device_array(None, 0)
    d = dg4.desc(8, dg4.DG4_BF16, 0.25)
    import ctypes
    assert lib.dg4_sparse_attn_fwd(None, ctypes.byref(d), None, 128, None, 128, None, 128, None, 128, None) \
        == dg4.DG4_ERR_INVALID_ARG


def test_large_circuits_are_validated_in_parallel_and_the_lowest_bad_node_is_reported():
    n = 300_000                                    # above the size at which validation uses several threads
    row_ptr = np.arange(n + 1, dtype=np.int32) - 1
    row_ptr[0] = 0                                 # node 0 is a primary input, node v > 0 has fan-in v - 1
    col_idx = np.arange(n - 1, dtype=np.int32)
    level = np.arange(n, dtype=np.int32)
    level[200_000] = 5                             # level does not increase along edge 199999 -> 200000
    level[250_000] = -3                            # a later fault that must not be the one reported
    with pytest.raises(dg4.Dg4Error) as e:
        dg4.dg4_graph_create(row_ptr, col_idx, level, 2, 0)
    assert e.value.status == dg4.DG4_ERR_BAD_LEVEL and "200000" in e.value.detail
