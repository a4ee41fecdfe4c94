"""CPU checks of the boundary: the library loads and exports every symbol include/ps.h declares."""
import ctypes as C
import os
import re

from paper_2406_05546_b200 import ps

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "ps.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(?:int32_t|const char\*)\s+((?:ps_|workers_)\w+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound():
    lib = ps.load()
    names = _declared()
    assert len(names) >= 19
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(ps.EXPORTS) == names


def test_query_bytes_needs_no_gpu_and_checks_ranges():
    lib = ps.load()
    c = ps.Config()
    c.max_workers, c.max_batch, c.ring_depth, c.chain_len, c.replicate_every = 128, 128, 1, 1, 1
    c.queue_slots, c.dropout_p, c.external_store = 25600 + 128, 0.25, 1
    a, p = C.c_uint64(), C.c_uint64()
    assert lib.ps_query_bytes(C.byref(c), C.byref(a), C.byref(p)) == 0
    queue_bytes = (25600 + 128) * ps.P_PAD * 4
    assert queue_bytes < a.value < queue_bytes + 2 * 2**30      # config 5 fits one 180 GB GPU
    c.ring_depth = 17
    assert lib.ps_query_bytes(C.byref(c), C.byref(a), C.byref(p)) == -1
    assert b"ring_depth" in lib.ps_last_error(None)
    c.ring_depth, c.dropout_p = 9, 1.0
    assert lib.ps_query_bytes(C.byref(c), C.byref(a), C.byref(p)) == -1


def test_struct_sizes_match_header_layout():
    assert C.sizeof(ps.Config) == 88 and C.sizeof(ps.Snapshot) == 16
    assert C.sizeof(ps.ApplyResult) == 24 and C.sizeof(ps.Stats) == 72
    assert ps.P_PAD % 64 == 0 and ps.P_PAD >= ps.P


def test_no_cpu_fallback():
    import pytest
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(RuntimeError):
        ps.ParameterServer([0.0] * ps.P, 1, 1)
