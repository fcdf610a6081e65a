"""The shared library loads without a GPU and exports every symbol include/ocs.h declares."""
import os
import re

import paper_1901_09504_b200 as ocs
from paper_1901_09504_b200 import build as ocs_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "ocs.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ocs_[a-z_0-9]+)\s*\(", text)))


def test_library_builds_loads_and_exports_all_declared_symbols():
    ocs_build.build()
    L = ocs.lib()
    names = _declared()
    assert len(names) >= 12
    for n in names:
        assert hasattr(L, n), n
    assert sorted(ocs.EXPORTS) == names
    assert b"sm_100a" in L.ocs_version()


def test_host_only_entry_points():
    assert ocs.ocs_num_splits(650, 0.02) == 13
    assert ocs.ocs_num_splits(25088, 0.1) == 2509
    assert ocs.ocs_num_splits(64, 0.0) == 0
    L = ocs.lib()
    assert L.ocs_split_workspace_bytes(4096, 25088, 1, 2509) > 8 * 25088
    assert L.ocs_quantize_workspace_bytes(2048, 128) >= 8 * 2048 + 8 * 128
    # a K split exchanges its partial sums through shared memory: the layer needs no global scratch
    assert L.ocs_qlinear_workspace_bytes(128, 4096, 25088, 2509) == 256
    assert L.ocs_qlinear_workspace_bytes(4096, 4096, 512, 0) == 256
    assert L.ocs_selftest_force_gemm_plan(96, 1) == 1 and L.ocs_selftest_force_gemm_plan(0, 0) == 0
