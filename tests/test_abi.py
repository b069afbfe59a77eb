"""The C-ABI library builds, loads without a GPU and exports every declared entry point."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_2608_04962_b200 import build as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def libpath():
    return B.build()


def _declared():
    text = open(os.path.join(ROOT, "include", "specroll.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(specroll_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(libpath):
    lib = ctypes.CDLL(libpath)
    names = _declared()
    assert {"specroll_propose", "specroll_tree_attn", "specroll_verify"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_binding_lists_the_same_entry_points():
    from paper_2608_04962_b200 import binding
    assert sorted(binding.EXPORTS) == _declared()


def test_host_only_entry_points(libpath):
    from paper_2608_04962_b200 import binding as S
    assert S.version() >= 100
    # node budget with the paper's setting C_peak = 512, N in [1, 10]
    assert [S.node_budget(512, b) for b in (256, 128, 64, 51, 1)] == [2, 4, 8, 10, 10]
    assert S.lib().specroll_strerror(1).decode().startswith("invalid")


def test_descriptor_validation_needs_no_device(libpath):
    from paper_2608_04962_b200 import binding as S
    assert S.propose_workspace_bytes(4, 8, 3, 2, 256, 1024) > 0
    assert S.propose_workspace_bytes(4, 8, 3, 2, 250, 1024) == 0      # d % 64 != 0
    assert S.propose_workspace_bytes(4, 65, 3, 2, 256, 1024) == 0     # too many nodes
    assert S.verify_workspace_bytes(4, 8, 3, 2, 1024) > 0
    assert S.verify_workspace_bytes(4, 8, 3, 2, 1001) == 0            # V % 8 != 0
    ip = np.array([0, 100, 300], np.int32)
    assert S.tree_attn_workspace_bytes(2, 8, 4, 2, 64, ip) > 0
    assert S.tree_attn_workspace_bytes(2, 8, 4, 3, 64, ip) == 0       # Hq % Hkv != 0
    assert S.tree_attn_workspace_bytes(2, 8, 4, 2, 96, ip) == 0       # head_dim
