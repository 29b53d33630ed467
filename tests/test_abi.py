"""Host-side checks that need no GPU: the library loads, exports what include/detox.h declares, and
rejects bad arguments before launching anything."""
import ctypes
import os
import re

import numpy as np
import pytest

import paper_1907_12205_b200 as dx
from paper_1907_12205_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_1907_12205_b200 import build
    build.build()
    return dx.load()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "detox.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b((?:detox|agg)_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert set(names) == set(dx.EXPORTS)
    for n in names:
        assert getattr(lib, n) is not None


def test_status_strings(lib):
    assert dx.status_string(0) == "ok"
    assert "argument" in dx.status_string(1)
    assert dx.status_string(99) == "unknown status"


def test_workspace_sizes(lib):
    assert dx.detox_vote_workspace_bytes(45, 3) >= 15 * 16
    assert dx.detox_vote_workspace_bytes(45, 4) == 0
    assert dx.agg_multikrum_workspace_bytes(45, 1000) > 45 * 45 * 8
    assert dx.agg_multikrum_workspace_bytes(5000, 1000) == 0
    p = dx.Pipeline(45, 3, 1000, np.arange(45), dx.AGG_MEAN, [0, 5, 10, 15], np.arange(15), dx.AGG_MULTIKRUM, 1, 1)
    assert p.workspace_bytes() > 3 * 1024 * 4                   # the three set means (votes are not stored)
    q = dx.Pipeline(105, 3, 1000, np.arange(105), dx.AGG_NONE, None, None, dx.AGG_MULTIKRUM, 3, 30)
    assert q.workspace_bytes() > 35 * 1024 * 4                  # the 35 votes, stored for the Gram kernel
    q = dx.Pipeline(45, 3, 1000, np.arange(45), dx.AGG_NONE, None, None, dx.AGG_COORD_MEDIAN)
    assert 0 < q.workspace_bytes() < 15 * 1000 * 4              # votes are read through winner[]: no copy
    bad = dx.Pipeline(45, 3, 1000, np.arange(45), dx.AGG_NONE, None, None, dx.AGG_BULYAN, 4, 1)  # 15 < 4*4+3
    assert bad.workspace_bytes() == 0


def test_distance_workspace_covers_every_row_count_of_the_tensor_core_path(lib):
    """The workspace of the distance pass is planned on the host (slab slots of both operand splits, norms, row scales,
    centre choice).  For every row count of the tensor-core path and column counts from one stage to ResNet-50 size the
    plan must exist, hold at least the distance matrix and its slab partials, and grow with d."""
    for m in list(range(17, 257, 7)) + [32, 33, 64, 65, 128, 129, 256]:
        prev = 0
        for d in (64, 4097, 1_000_000, 11_173_962, 25_557_032):
            b = dx.agg_pairwise_sqdist_workspace_bytes(m, d)
            assert b >= m * m * 8 + m * 4, (m, d)
            assert b >= prev, (m, d)
            prev = b
        ncol = (m + 15) // 16 * 16
        # at least one fp32 partial of m x ncol per CTA at full width
        assert dx.agg_pairwise_sqdist_workspace_bytes(m, 25_557_032) >= 148 * m * ncol * 4
        assert dx.agg_multikrum_workspace_bytes(m, 11_173_962) >= dx.agg_pairwise_sqdist_workspace_bytes(m, 11_173_962)


def test_split_mode_switch_and_its_query(lib):
    assert dx.tc_split_mode() == dx.SPLIT_AUTO
    assert dx.tc_split_mode(dx.SPLIT_TF32) == dx.SPLIT_AUTO
    assert dx.tc_split_mode(7) == dx.SPLIT_TF32          # an unknown value only queries
    assert dx.tc_split_mode(dx.SPLIT_AUTO) == dx.SPLIT_TF32
    assert dx.tc_split_mode() == dx.SPLIT_AUTO


def test_bad_arguments_are_rejected_before_any_launch(lib):
    # Pointers are fake but never dereferenced: every call must fail in validation.
    fake = ctypes.c_void_p(0x1000)
    mem = np.arange(15, dtype=np.int32)
    ip = mem.ctypes.data_as(ctypes.POINTER(ctypes.c_int32))
    call = lib.detox_vote
    assert call(fake, 100, 15, 2, 100, ip, None, 0, fake, fake, 4096, None) == 1      # r even
    assert call(fake, 100, 15, 4, 100, ip, None, 0, fake, fake, 4096, None) == 1      # r does not divide n
    assert call(fake, 100, 15, 3, 0, ip, None, 0, fake, fake, 4096, None) == 1        # d < 1
    assert call(fake, 50, 15, 3, 100, ip, None, 0, fake, fake, 4096, None) == 1       # ld < d
    assert call(None, 100, 15, 3, 100, ip, None, 0, fake, fake, 4096, None) == 1      # null X
    assert call(fake, 100, 15, 3, 100, ip, None, 0, fake, None, 0, None) == 3         # no workspace
    assert call(fake, 100, 15, 3, 100, ip, None, 0, fake, ctypes.c_void_p(0x1010), 4096, None) == 3  # misaligned
    dup = mem.copy(); dup[3] = 2
    assert call(fake, 100, 15, 3, 100, dup.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)), None, 0, fake, fake,
                4096, None) == 1                                                       # not a partition
    assert call(fake, 100, 17 * 3, 17, 100, ip, None, 0, fake, fake, 4096, None) == 2  # r beyond the limit
    so = np.array([0, 5, 5, 15], np.int32)
    sm = np.arange(15, dtype=np.int32)
    assert lib.detox_hier_mean(fake, 100, 15, 100, so.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)),
                               sm.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)), 3, fake, 100, None) == 1  # empty set
    assert lib.agg_bulyan(fake, 100, 10, 100, 2, fake, None, fake, 1 << 30, None) == 1  # 10 < 4*2+3
    assert lib.agg_multikrum(fake, 100, 10, 100, 1, 11, fake, None, None, fake, 1 << 30, None) == 1  # m_sel > m
    assert lib.agg_coord_median(fake, 100, 2000, 100, fake, None, 0, None) == 2       # m beyond the limit


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", "/nonexistent/libdetox.so")
    with pytest.raises(ImportError):
        binding.load()
