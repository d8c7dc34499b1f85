"""CPU-only checks of the C-ABI library: it loads, exports every symbol the header declares, and
its host-only logic (layout, argument validation, workspace sizes) behaves.  No kernel is launched."""
import ctypes as C
import os
import re

import numpy as np
import pytest

import oracle
import paper_2106_11257_b200 as btard
from paper_2106_11257_b200 import build as btard_build
from paper_2106_11257_b200.binding import CclipArgs, VerifyArgs

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    btard_build.build()


def test_every_declared_symbol_is_exported():
    text = open(os.path.join(ROOT, "include", "btard.h")).read()
    declared = sorted(set(re.findall(r"BTARD_API\s+[\w\s\*]+?\b(btard_\w+)\s*\(", text)))
    assert declared, "no declarations found"
    assert sorted(btard.EXPORTS) == declared
    lib = btard.lib()
    for name in declared:
        assert getattr(lib, name) is not None


@pytest.mark.parametrize("d,P", [(0, 1), (1, 1), (10, 3), (5, 8), (1024, 1), (11173962, 16),
                                 (17683968, 64), (1 << 28, 64), (1000003, 7)])
@pytest.mark.parametrize("mode", [btard.SPLIT_PAPER, btard.SPLIT_CEIL_PAD])
@pytest.mark.parametrize("align", [4, 32])
def test_layout_is_bit_exact_against_the_oracle(d, P, mode, align):
    off, ln, stride = btard.partition_layout(d, P, mode, align)
    o_off, o_ln, o_stride = oracle.partition_layout(d, P, mode, align)
    assert np.array_equal(off, o_off) and np.array_equal(ln, o_ln)
    assert stride == max(o_stride, align)      # the library never returns a zero-length row


def test_layout_rejects_bad_arguments():
    for args in [(-1, 4, 0, 32), (10, 0, 0, 32), (10, 4, 2, 32), (10, 4, 0, 6), (10, 4, 0, 0)]:
        with pytest.raises(btard.BtardError):
            btard.partition_layout(*args)


def test_workspace_queries_and_validation_without_a_gpu():
    assert btard.centered_clip_workspace(16, 16, 698400) > 0
    assert btard.verify_projections_workspace(16, 16, 698400, 8) > 0
    assert btard.centered_clip_workspace(0, 16, 698400) == 0
    assert btard.centered_clip_workspace(btard.lib() and 257, 16, 698400) == 0
    assert btard.aggregate_host_scratch(16, 16, 698400, 1) > 16 * 16 * 698400 * 4
    lib = btard.lib()
    ln = np.array([8], dtype=np.int64)
    tau = np.array([1.0], dtype=np.float64)
    a = CclipArgs(n_peers=4, n_partitions=1, row_stride=8, part_len=ln.ctypes.data, tau=tau.ctypes.data,
                  max_iters=1)
    assert lib.btard_centered_clip(C.byref(a)) == -1            # NULL device pointers
    a.row_stride = 6
    assert lib.btard_centered_clip(C.byref(a)) == -2            # stride not a multiple of 4
    a.row_stride = 8
    tau[0] = -1.0
    assert lib.btard_centered_clip(C.byref(a)) == -1
    tau[0] = np.nan
    assert lib.btard_centered_clip(C.byref(a)) == -1
    tau[0] = 1.0
    a.n_peers = 1000
    assert lib.btard_centered_clip(C.byref(a)) == -5
    v = VerifyArgs(n_peers=4, n_partitions=1, row_stride=8, part_len=ln.ctypes.data,
                   tau=tau.ctypes.data, n_z=1)
    assert lib.btard_verify_projections(C.byref(v)) == -1
    assert lib.btard_centered_clip(None) == -1


def test_generator_layout_matches_the_library():
    import workloads
    for cfg in (1, 2, 3, 4, 5):
        w = workloads.make_workload(cfg, data=False)
        _, ln, stride = btard.partition_layout(w.d, w.P, btard.SPLIT_CEIL_PAD, 32)
        assert np.array_equal(ln, w.part_len) and stride == w.row_stride
