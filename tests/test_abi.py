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


def test_attention_plan_is_host_only_and_consistent(libpath):
    """The planner (chunk length by simulated hand-out, cached per lengths) runs without a device."""
    from paper_2608_04962_b200 import binding as S
    from paper_2608_04962_b200 import inputs as I
    for name in ("qwen1.5b", "qwen7b", "sweep7b_B8"):
        w = I.WORKLOADS[name]
        L = I.kv_lengths(w)
        ip = np.zeros(w.B + 1, np.int32)
        np.cumsum(L, out=ip[1:])
        a = S.tree_attn_workspace_bytes(w.B, w.N, w.Hq, w.Hkv, w.D, ip)
        b = S.tree_attn_workspace_bytes(w.B, w.N, w.Hq, w.Hkv, w.D, ip)          # second time from the cache
        assert a == b and a > 0
        assert S.tree_attn_paged_workspace_bytes(w.B, w.N, w.Hq, w.Hkv, w.D, L.astype(np.int32)) == a
        first = S.tree_attn_launches(w.B, w.N, w.Hq, w.Hkv, w.D, ip)
        later = S.tree_attn_launches(w.B, w.N, w.Hq, w.Hkv, w.D, ip, flags=S.ATTN_REUSE_PLAN)
        assert first == later + 1 and later in (1, 2)                            # plan kernel only the first time
        # the scheduling hint about the cache changes nothing that is counted
        assert S.tree_attn_launches(w.B, w.N, w.Hq, w.Hkv, w.D, ip, flags=S.ATTN_REUSE_PLAN | S.ATTN_CACHE_SETTLED) == later
    # a changed length changes the plan's key: no stale answer
    ip2 = ip.copy()
    ip2[-1] += 4096
    assert S.tree_attn_workspace_bytes(w.B, w.N, w.Hq, w.Hkv, w.D, ip2) != 0
    assert S.tree_attn_launches(w.B, w.N, w.Hq, w.Hkv, w.D, ip, flags=64) == -1  # unknown flag
    assert S.verify_nucleus_workspace_bytes(4, 8, 3, 2, 1024) > 0


def test_cache_offsets_must_start_at_zero(libpath):
    """Token coordinates count from the base of Kc / Vc: an offset table that starts elsewhere is refused on the
    host, before anything is enqueued (no device needed)."""
    import ctypes as C
    from paper_2608_04962_b200 import binding as S
    desc = S.AttnDesc(2, 8, 4, 2, 64, 0.125, 0)
    ip = np.array([5, 100, 300], np.int32)
    parent = np.array([-1, 0, 0, 1, 1, 2, 3, 3], np.int32)
    null = C.c_void_p(0)
    rc = S.lib().specroll_tree_attn(C.byref(desc), null, null, null, null, ip.ctypes.data_as(C.c_void_p), null, null,
                                    parent.ctypes.data_as(C.c_void_p), null, null, null, C.c_size_t(0), null)
    assert rc == 1                                                                # SPECROLL_EINVAL
    assert S.tree_attn_launches(2, 8, 4, 2, 64, np.array([0, 100, 300], np.int32), flags=S.ATTN_NO_PDL) >= 1


def test_an_empty_batch_is_valid_and_needs_no_device(libpath):
    """B = 0: descriptor and topology are checked, nothing is enqueued, the (empty) arrays may be NULL."""
    import ctypes as C
    from paper_2608_04962_b200 import binding as S
    L, null = S.lib(), C.c_void_p(0)
    parent = np.array([-1, 0, 0, 1], np.int32)
    pp = parent.ctypes.data_as(C.c_void_p)
    pd = S.ProposeDesc(0, 4, 2, 2, 64, 64, 1.0, 1e-5, 1e-6, 0.0, 0)
    assert L.specroll_propose(C.byref(pd), *([null] * 9), pp, *([null] * 7), C.c_size_t(0), null) == 0
    assert L.specroll_tree_draw(C.c_int32(0), C.c_int32(4), C.c_int32(2), C.c_int32(2), C.c_float(1.0), pp,
                                *([null] * 8)) == 0
    vd = S.VerifyDesc(0, 4, 2, 2, 64, 1.0, 0)
    assert L.specroll_verify(C.byref(vd), null, pp, *([null] * 15), C.c_size_t(0), null) == 0
    ad = S.AttnDesc(0, 4, 4, 2, 64, 0.125, 0)
    ip = np.zeros(1, np.int32)
    assert L.specroll_tree_attn(C.byref(ad), null, null, null, null, ip.ctypes.data_as(C.c_void_p), null, null, pp, null,
                                null, null, C.c_size_t(0), null) == 0
    # a malformed tree is still refused
    bad = np.array([-1, 2, 0, 1], np.int32)
    assert L.specroll_verify(C.byref(vd), null, bad.ctypes.data_as(C.c_void_p), *([null] * 15), C.c_size_t(0), null) == 1
