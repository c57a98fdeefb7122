"""The C-ABI library loads, exports every symbol include/pe.h declares, and its host-only
checks return the documented codes.  No GPU work."""
import ctypes
import os
import re

import numpy as np
import pytest

from tests.conftest import ROOT


@pytest.fixture(scope="module")
def pe():
    from paper_2503_09357_b200.build import build_libpe
    build_libpe()
    from paper_2503_09357_b200 import binding
    return binding


def declared_functions():
    text = open(os.path.join(ROOT, "include", "pe.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(pe_[a-z_]+)\s*\(", text)))


def test_header_declares_the_boundary():
    names = declared_functions()
    for must in ("pe_graph_create", "pe_eval_batch", "pe_destroy"):
        assert must in names
    assert len(names) >= 8


def test_library_exports_every_declared_symbol(pe):
    lib = ctypes.CDLL(pe.LIB_PATH)
    for name in declared_functions():
        assert hasattr(lib, name), f"{name} is declared in pe.h but not exported"


def test_binding_has_the_same_names(pe):
    for name in declared_functions():
        assert hasattr(pe, name), f"binding lacks {name}"


def _desc(pe, **over):
    base = dict(num_ops=3, edge_src=np.array([0, 1]), edge_dst=np.array([1, 2]), dur=np.array([1, 2, 3]),
                num_devices=2, mem_delta=np.array([1, -1, 0]), comm=np.array([1, 1]))
    base.update(over)
    return pe.make_desc(**base)


def test_validate_codes(pe):
    ok = lambda **o: pe.pe_graph_validate(_desc(pe, **o)[0])
    assert ok() == pe.PE_OK
    assert ok(edge_src=np.array([0, 2]), edge_dst=np.array([2, 0])) == pe.PE_ERR_CYCLE
    assert ok(edge_src=np.array([0, 1]), edge_dst=np.array([1, 1])) == pe.PE_ERR_CYCLE          # self loop
    assert ok(edge_src=np.array([0, 3]), edge_dst=np.array([1, 2])) == pe.PE_ERR_RANGE           # endpoint >= V
    assert ok(dur=np.array([1, -2, 3])) == pe.PE_ERR_RANGE
    assert ok(comm=np.array([1, -1])) == pe.PE_ERR_RANGE
    assert ok(mem_weight=np.array([1, -1, 0])) == pe.PE_ERR_RANGE
    assert ok(link_class=np.array([[0, 1], [0, 0]])) == pe.PE_ERR_RANGE                          # class >= L
    assert ok(link_class=np.array([[0, 255], [0, 0]])) == pe.PE_OK                               # 0xFF = no channel
    assert ok(num_devices=0) == pe.PE_ERR_INVALID_ARG
    assert ok(num_devices=256) == pe.PE_ERR_INVALID_ARG
    assert ok(num_ops=0) == pe.PE_ERR_INVALID_ARG
    assert ok(num_link_classes=0) == pe.PE_ERR_INVALID_ARG
    assert ok(dur=None) == pe.PE_ERR_INVALID_ARG
    big = 2 ** 30
    assert ok(dur=np.array([big, big, 1])) == pe.PE_ERR_OVERFLOW
    assert ok(dur=np.array([big, 1, 1]), comm=np.array([big, 1])) == pe.PE_ERR_OVERFLOW
    assert ok(mem_delta=np.array([big, -big, 1])) == pe.PE_ERR_OVERFLOW
    assert ok(dur=np.array([big, big - 3, 1]), comm=np.array([0, 0])) == pe.PE_OK
    assert pe._lib.pe_graph_validate(None) == pe.PE_ERR_INVALID_ARG


def test_strerror_and_null_handles(pe):
    for code in range(-9, 1):
        assert "unknown" not in pe.pe_strerror(code)
    assert "unknown" in pe.pe_strerror(-99)
    assert pe.pe_destroy(None) == pe.PE_OK
    assert pe.pe_workspace_bytes(None, 10, 0) == 0
    assert pe.pe_eval_variant(None, 10, 0) == pe.PE_ERR_INVALID_ARG
    assert pe.pe_kernel_launches() >= 0
    o = pe.make_outputs()
    assert pe.pe_eval_batch(None, 1, 0, 0, 2, 0, o) == pe.PE_ERR_INVALID_ARG
