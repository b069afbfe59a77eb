"""Thin Python binding of the C-ABI library ``libspecroll.so``.

Argument marshalling only: every function checks dtype / device / contiguity of torch
tensors, allocates outputs and the workspace with torch, and passes raw pointers to the
entry point of the same name.  No step of the method runs in Python.  The library is loaded
on first use and loading fails loudly when it has not been built: there is no fallback.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# SPECROLL_LIB selects another build of the same library (the debug build with index checks, libspecroll_check.so)
LIB_PATH = os.environ.get("SPECROLL_LIB") or os.path.join(_HERE, "libspecroll.so")
_lib = None

EXPORTS = ("specroll_version", "specroll_strerror", "specroll_node_budget", "specroll_check_status", "specroll_check_inject",
           "specroll_propose_workspace_bytes", "specroll_propose", "specroll_workspace_status",
           "specroll_tree_draw",
           "specroll_tree_attn_workspace_bytes", "specroll_tree_attn", "specroll_tree_attn_launches",
           "specroll_tree_attn_paged_workspace_bytes", "specroll_tree_attn_paged",
           "specroll_commit_path", "specroll_commit_path_layers", "specroll_gather_hidden",
           "specroll_verify_workspace_bytes", "specroll_verify", "specroll_verify_static",
           "specroll_verify_nucleus_workspace_bytes", "specroll_verify_nucleus",
           "specroll_reflex_feedback_workspace_bytes", "specroll_reflex_feedback", "specroll_reflex_feedback_ex",
           "specroll_reflex_sketch", "specroll_reflex_gate",
           "specroll_target_head_stats_workspace_bytes", "specroll_target_head_stats", "specroll_target_head_rows",
           "specroll_verify_want_ids", "specroll_verify_walk_sparse", "specroll_verify_terminal_rows")


PROPOSE_LEGACY_MMA = 1
REFLEX_PRE_HEAD = 2
ATTN_LEGACY_MMA = 1
ATTN_REUSE_PLAN = 2
ATTN_CACHE_SETTLED = 4
ATTN_NO_PDL = 8
VERIFY_LAZY_STATS = 1
FEEDBACK_SEVERITY = 1
PAGE_TOKENS = 128


class SpecrollError(RuntimeError):
    pass


class ProposeDesc(C.Structure):
    _fields_ = [("B", C.c_int32), ("N", C.c_int32), ("K", C.c_int32), ("k", C.c_int32),
                ("d", C.c_int32), ("V", C.c_int32), ("temperature", C.c_float),
                ("ln_eps", C.c_float), ("rms_eps", C.c_float), ("clip_c", C.c_float),
                ("flags", C.c_int32)]


class AttnDesc(C.Structure):
    _fields_ = [("B", C.c_int32), ("N", C.c_int32), ("Hq", C.c_int32), ("Hkv", C.c_int32),
                ("D", C.c_int32), ("scale", C.c_float), ("flags", C.c_int32)]


class VerifyDesc(C.Structure):
    _fields_ = [("B", C.c_int32), ("N", C.c_int32), ("K", C.c_int32), ("k", C.c_int32),
                ("V", C.c_int32), ("temperature", C.c_float), ("flags", C.c_int32)]


class FeedbackDesc(C.Structure):
    _fields_ = [("R", C.c_int32), ("k", C.c_int32), ("k_support", C.c_int32), ("d", C.c_int32), ("V", C.c_int32),
                ("temperature", C.c_float), ("eps", C.c_float), ("flags", C.c_int32), ("severity_min", C.c_float)]


class GateDesc(C.Structure):
    _fields_ = [("R", C.c_int32), ("S", C.c_int32), ("d", C.c_int32), ("rank", C.c_int32), ("H", C.c_int32),
                ("z_delta", C.c_float), ("mem_eps", C.c_float), ("flags", C.c_int32)]


def lib():
    """The loaded library.  Raises if it is missing: the CUDA path is the only path."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise SpecrollError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2608_04962_b200.build` "
                "(there is no CPU or PyTorch fallback)")
        l = C.CDLL(LIB_PATH)
        l.specroll_version.restype = C.c_int
        l.specroll_strerror.restype = C.c_char_p
        l.specroll_strerror.argtypes = [C.c_int]
        l.specroll_node_budget.restype = C.c_int32
        l.specroll_node_budget.argtypes = [C.c_int32] * 4
        for n in ("specroll_propose_workspace_bytes", "specroll_verify_workspace_bytes",
                  "specroll_tree_attn_workspace_bytes", "specroll_tree_attn_paged_workspace_bytes",
                  "specroll_verify_nucleus_workspace_bytes", "specroll_reflex_feedback_workspace_bytes",
                  "specroll_target_head_stats_workspace_bytes"):
            getattr(l, n).restype = C.c_size_t
        for n in ("specroll_propose", "specroll_workspace_status", "specroll_tree_draw", "specroll_tree_attn",
                  "specroll_verify", "specroll_verify_static", "specroll_tree_attn_paged", "specroll_commit_path",
                  "specroll_commit_path_layers", "specroll_gather_hidden", "specroll_verify_nucleus",
                  "specroll_tree_attn_launches", "specroll_reflex_feedback"):
            getattr(l, n).restype = C.c_int
        _lib = l
    return _lib


def _check(rc: int, what: str):
    if rc != 0:
        raise SpecrollError(f"{what}: {lib().specroll_strerror(rc).decode()} (code {rc})")


def _dev(t: Optional[torch.Tensor], dtype, name: str):
    if t is None:
        return None
    if not t.is_cuda:
        raise SpecrollError(f"{name} must be a CUDA tensor")
    if t.dtype != dtype:
        raise SpecrollError(f"{name} must have dtype {dtype}, got {t.dtype}")
    if not t.is_contiguous():
        raise SpecrollError(f"{name} must be contiguous")
    return C.c_void_p(t.data_ptr())


def _host_i32(a, name: str) -> np.ndarray:
    a = np.ascontiguousarray(np.asarray(a), dtype=np.int32)
    if a.ndim != 1:
        raise SpecrollError(f"{name} must be one-dimensional")
    return a


def _stream() -> C.c_void_p:
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


# Every device tensor this module allocates (outputs and workspaces) comes from this function.  The tests swap in
# an allocator that surrounds each tensor with guard bytes and checks them afterwards (set_allocator); by default
# it is torch.empty.
_empty = torch.empty


def set_allocator(fn=None):
    """Replaces the allocator of outputs and workspaces (signature of torch.empty); None restores torch.empty."""
    global _empty
    _empty = torch.empty if fn is None else fn


def alloc(*size, **kw) -> torch.Tensor:
    """torch.empty through the current allocator (for callers that keep outputs and workspaces of their own)."""
    return _empty(*size, **kw)


def _workspace(nbytes: int, device) -> torch.Tensor:
    return _empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)


def version() -> int:
    return int(lib().specroll_version())


def check_status(reset: bool = True):
    """specroll_check_status after a device synchronisation: (code, detail).  code is -1 for a normal build, 0 when
    the debug build's index checks found nothing, else SPECROLL_EINDEX with detail = the sequence it was found in."""
    torch.cuda.synchronize()
    detail = C.c_int32(0)
    rc = int(lib().specroll_check_status(C.byref(detail), C.c_int32(1 if reset else 0)))
    return rc, int(detail.value)


def workspace_status(workspace: torch.Tensor) -> int:
    """specroll_workspace_status: 0, or the error code a kernel left in this workspace (synchronises)."""
    return int(lib().specroll_workspace_status(C.c_void_p(workspace.data_ptr()), _stream()))


def node_budget(C_hw: int, B_active: int, N_min: int = 1, N_max: int = 10) -> int:
    return int(lib().specroll_node_budget(C_hw, B_active, N_min, N_max))


# ----------------------------------------------------------------------------------- propose


def propose_workspace_bytes(B, N, K, k, d, V, temperature=1.0, ln_eps=1e-5, rms_eps=1e-6,
                            clip_c=0.0, flags=0) -> int:
    desc = ProposeDesc(B, N, K, k, d, V, temperature, ln_eps, rms_eps, clip_c, flags)
    return int(lib().specroll_propose_workspace_bytes(C.byref(desc)))


def propose(h, anchor, A, bias, W, m, alpha, parent, u_draw, k, temperature=1.0, ln_eps=1e-5,
            rms_eps=1e-6, clip_c=0.0, ln_gamma=None, ln_beta=None, workspace=None,
            out: Optional[Dict[str, torch.Tensor]] = None, flags: int = 0,
            check_status: bool = False) -> Dict[str, torch.Tensor]:
    """specroll_propose.  Device tensors in, dict of device tensors out.
    ``check_status`` also calls specroll_workspace_status (synchronises the stream)."""
    parent = _host_i32(parent, "parent")
    B, d = h.shape
    K, V, N = A.shape[0], W.shape[0], parent.shape[0]
    if tuple(A.shape) != (K, d, d) or tuple(bias.shape) != (K, d) or W.shape[1] != d:
        raise SpecrollError("propose: inconsistent weight shapes")
    if tuple(u_draw.shape) != (B, N) or tuple(anchor.shape) != (B,):
        raise SpecrollError("propose: inconsistent u_draw / anchor shapes")
    if flags & REFLEX_PRE_HEAD:
        if m is not None and tuple(m.shape) != (B, d):
            raise SpecrollError("propose: with REFLEX_PRE_HEAD m must be [B,d]")
        if alpha is not None and tuple(alpha.shape) != (B,):
            raise SpecrollError("propose: with REFLEX_PRE_HEAD alpha must be [B]")
    else:
        if m is not None and tuple(m.shape) != (B, K, d):
            raise SpecrollError("propose: m must be [B,K,d]")
        if alpha is not None and tuple(alpha.shape) != (B, K):
            raise SpecrollError("propose: alpha must be [B,K]")
    desc = ProposeDesc(B, N, K, k, d, V, temperature, ln_eps, rms_eps, clip_c, flags)
    dev = h.device
    if out is None:
        out = {"cand_id": _empty((B, K, k), dtype=torch.int32, device=dev),
               "cand_logit": _empty((B, K, k), dtype=torch.float32, device=dev),
               "tree_tok": _empty((B, N), dtype=torch.int32, device=dev),
               "tree_cand": _empty((B, N), dtype=torch.uint8, device=dev),
               "slot_q": _empty((B, N), dtype=torch.float32, device=dev)}
    if workspace is None:
        workspace = _workspace(lib().specroll_propose_workspace_bytes(C.byref(desc)), dev)
    bf = torch.bfloat16
    rc = lib().specroll_propose(
        C.byref(desc), _dev(h, bf, "h"), _dev(anchor, torch.int32, "anchor"), _dev(A, bf, "A"),
        _dev(bias, bf, "bias"), _dev(ln_gamma, bf, "ln_gamma"), _dev(ln_beta, bf, "ln_beta"),
        _dev(W, bf, "W"), _dev(m, torch.float32, "m"), _dev(alpha, torch.float32, "alpha"),
        parent.ctypes.data_as(C.c_void_p), _dev(u_draw, torch.float32, "u_draw"),
        _dev(out["cand_id"], torch.int32, "cand_id"), _dev(out["cand_logit"], torch.float32, "cand_logit"),
        _dev(out["tree_tok"], torch.int32, "tree_tok"), _dev(out["tree_cand"], torch.uint8, "tree_cand"),
        _dev(out["slot_q"], torch.float32, "slot_q"), C.c_void_p(workspace.data_ptr()),
        C.c_size_t(workspace.numel()), _stream())
    _check(rc, "specroll_propose")
    if check_status:
        _check(lib().specroll_workspace_status(C.c_void_p(workspace.data_ptr()), _stream()), "specroll_workspace_status")
    return out


def tree_draw(parent, anchor, cand_id, cand_logit, u_draw, temperature=1.0) -> Dict[str, torch.Tensor]:
    """specroll_tree_draw."""
    parent = _host_i32(parent, "parent")
    B, K, k = cand_id.shape
    N = parent.shape[0]
    dev = cand_id.device
    out = {"tree_tok": _empty((B, N), dtype=torch.int32, device=dev),
           "tree_cand": _empty((B, N), dtype=torch.uint8, device=dev),
           "slot_q": _empty((B, N), dtype=torch.float32, device=dev)}
    rc = lib().specroll_tree_draw(
        C.c_int32(B), C.c_int32(N), C.c_int32(K), C.c_int32(k), C.c_float(temperature),
        parent.ctypes.data_as(C.c_void_p), _dev(anchor, torch.int32, "anchor"),
        _dev(cand_id, torch.int32, "cand_id"), _dev(cand_logit, torch.float32, "cand_logit"),
        _dev(u_draw, torch.float32, "u_draw"), _dev(out["tree_tok"], torch.int32, "tree_tok"),
        _dev(out["tree_cand"], torch.uint8, "tree_cand"), _dev(out["slot_q"], torch.float32, "slot_q"),
        _stream())
    _check(rc, "specroll_tree_draw")
    return out


# ----------------------------------------------------------------------------------- attention


def tree_attn_workspace_bytes(B, N, Hq, Hkv, D, kv_indptr_host, scale=None) -> int:
    ip = _host_i32(kv_indptr_host, "kv_indptr_host")
    desc = AttnDesc(B, N, Hq, Hkv, D, scale if scale is not None else 1.0 / float(np.sqrt(D)), 0)
    return int(lib().specroll_tree_attn_workspace_bytes(C.byref(desc), ip.ctypes.data_as(C.c_void_p)))


def tree_attn_launches(B, N, Hq, Hkv, D, kv_indptr_host, flags: int = 0) -> int:
    """Kernels one tree_attn call enqueues for these lengths (the plan decides whether a merge kernel runs)."""
    ip = _host_i32(kv_indptr_host, "kv_indptr_host")
    desc = AttnDesc(B, N, Hq, Hkv, D, 1.0 / float(np.sqrt(D)), flags)
    return int(lib().specroll_tree_attn_launches(C.byref(desc), ip.ctypes.data_as(C.c_void_p)))


def tree_attn(Q, Kc, Vc, kv_indptr_dev, kv_indptr_host, Kt, Vt, parent, scale=None, want_lse=False,
              workspace=None, out=None, lse=None, flags: int = 0, check_status: bool = False):
    """specroll_tree_attn.  Returns O (and lse when asked).
    ``check_status`` also calls specroll_workspace_status (synchronises the stream)."""
    parent = _host_i32(parent, "parent")
    ip = _host_i32(kv_indptr_host, "kv_indptr_host")
    B, N, Hq, D = Q.shape
    Hkv = Kt.shape[2]
    if ip.shape[0] != B + 1 or tuple(Kt.shape) != (B, N, Hkv, D) or tuple(Vt.shape) != (B, N, Hkv, D):
        raise SpecrollError("tree_attn: inconsistent shapes")
    if Kc.shape[0] != int(ip[-1]) or tuple(Kc.shape[1:]) != (Hkv, D) or Vc.shape != Kc.shape:
        raise SpecrollError("tree_attn: cache shape does not match kv_indptr")
    if scale is None:
        scale = 1.0 / float(np.sqrt(D))
    desc = AttnDesc(B, N, Hq, Hkv, D, scale, flags)
    dev = Q.device
    if out is None:
        out = _empty((B, N, Hq, D), dtype=torch.bfloat16, device=dev)
    if want_lse and lse is None:
        lse = _empty((B, N, Hq), dtype=torch.float32, device=dev)
    if workspace is None:
        workspace = _workspace(lib().specroll_tree_attn_workspace_bytes(
            C.byref(desc), ip.ctypes.data_as(C.c_void_p)), dev)
    bf = torch.bfloat16
    rc = lib().specroll_tree_attn(
        C.byref(desc), _dev(Q, bf, "Q"), _dev(Kc, bf, "Kc"), _dev(Vc, bf, "Vc"),
        _dev(kv_indptr_dev, torch.int32, "kv_indptr_dev"), ip.ctypes.data_as(C.c_void_p),
        _dev(Kt, bf, "Kt"), _dev(Vt, bf, "Vt"), parent.ctypes.data_as(C.c_void_p),
        _dev(out, bf, "O"), _dev(lse, torch.float32, "lse"), C.c_void_p(workspace.data_ptr()),
        C.c_size_t(workspace.numel()), _stream())
    _check(rc, "specroll_tree_attn")
    if check_status:
        _check(lib().specroll_workspace_status(C.c_void_p(workspace.data_ptr()), _stream()),
               "specroll_workspace_status")
    return (out, lse) if want_lse else out


def tree_attn_paged_workspace_bytes(B, N, Hq, Hkv, D, kv_len_host, scale=None) -> int:
    kl = _host_i32(kv_len_host, "kv_len_host")
    desc = AttnDesc(B, N, Hq, Hkv, D, scale if scale is not None else 1.0 / float(np.sqrt(D)), 0)
    return int(lib().specroll_tree_attn_paged_workspace_bytes(C.byref(desc), kl.ctypes.data_as(C.c_void_p)))


def tree_attn_paged(Q, Kp, Vp, page_table, page_indptr, kv_len_dev, kv_len_host, Kt, Vt, parent, scale=None,
                    want_lse=False, workspace=None, out=None, lse=None, flags: int = 0, check_status: bool = False):
    """specroll_tree_attn_paged.  Kp, Vp: [n_pages, 128, Hkv, D]; page_table, page_indptr, kv_len_dev: device
    int32; kv_len_host: host copy of the lengths.  Returns O (and lse when asked)."""
    parent = _host_i32(parent, "parent")
    kl = _host_i32(kv_len_host, "kv_len_host")
    B, N, Hq, D = Q.shape
    Hkv = Kt.shape[2]
    if kl.shape[0] != B or tuple(Kt.shape) != (B, N, Hkv, D) or tuple(Vt.shape) != (B, N, Hkv, D):
        raise SpecrollError("tree_attn_paged: inconsistent shapes")
    if tuple(Kp.shape[1:]) != (PAGE_TOKENS, Hkv, D) or Vp.shape != Kp.shape:
        raise SpecrollError("tree_attn_paged: page pool must be [n_pages, 128, Hkv, D]")
    if page_indptr.numel() != B + 1 or kv_len_dev.numel() != B:
        raise SpecrollError("tree_attn_paged: page_indptr / kv_len_dev sizes")
    if scale is None:
        scale = 1.0 / float(np.sqrt(D))
    desc = AttnDesc(B, N, Hq, Hkv, D, scale, flags)
    dev = Q.device
    if out is None:
        out = _empty((B, N, Hq, D), dtype=torch.bfloat16, device=dev)
    if want_lse and lse is None:
        lse = _empty((B, N, Hq), dtype=torch.float32, device=dev)
    if workspace is None:
        workspace = _workspace(lib().specroll_tree_attn_paged_workspace_bytes(
            C.byref(desc), kl.ctypes.data_as(C.c_void_p)), dev)
    bf = torch.bfloat16
    rc = lib().specroll_tree_attn_paged(
        C.byref(desc), _dev(Q, bf, "Q"), _dev(Kp, bf, "Kp"), _dev(Vp, bf, "Vp"), C.c_int64(Kp.shape[0]),
        _dev(page_table, torch.int32, "page_table"), _dev(page_indptr, torch.int32, "page_indptr"),
        _dev(kv_len_dev, torch.int32, "kv_len_dev"), kl.ctypes.data_as(C.c_void_p),
        _dev(Kt, bf, "Kt"), _dev(Vt, bf, "Vt"), parent.ctypes.data_as(C.c_void_p),
        _dev(out, bf, "O"), _dev(lse, torch.float32, "lse"), C.c_void_p(workspace.data_ptr()),
        C.c_size_t(workspace.numel()), _stream())
    _check(rc, "specroll_tree_attn_paged")
    if check_status:
        _check(lib().specroll_workspace_status(C.c_void_p(workspace.data_ptr()), _stream()),
               "specroll_workspace_status")
    return (out, lse) if want_lse else out


def commit_path(Kt, Vt, path_node, n_acc, Kp, Vp, page_table, page_indptr, kv_len, kv_len_out=None, status=None):
    """specroll_commit_path: appends the committed path's tree rows to one layer's paged cache (in place)."""
    B, N, Hkv, D = Kt.shape
    K = path_node.shape[1] - 1
    bf = torch.bfloat16
    rc = lib().specroll_commit_path(
        B, N, K, Hkv, D, _dev(Kt, bf, "Kt"), _dev(Vt, bf, "Vt"), _dev(path_node, torch.int32, "path_node"),
        _dev(n_acc, torch.int32, "n_acc"), _dev(Kp, bf, "Kp"), _dev(Vp, bf, "Vp"), C.c_int64(Kp.shape[0]),
        _dev(page_table, torch.int32, "page_table"), _dev(page_indptr, torch.int32, "page_indptr"),
        _dev(kv_len, torch.int32, "kv_len"), _dev(kv_len_out, torch.int32, "kv_len_out"),
        _dev(status, torch.int32, "status"), _stream())
    _check(rc, "specroll_commit_path")


def commit_path_layers(Kt, Vt, path_node, n_acc, Kp, Vp, page_table, page_indptr, kv_len, kv_len_out=None,
                       status=None):
    """specroll_commit_path_layers: Kt, Vt, Kp, Vp are lists with one tensor per layer."""
    n = len(Kt)
    if not (len(Vt) == len(Kp) == len(Vp) == n) or n == 0:
        raise SpecrollError("commit_path_layers: one tensor per layer in each list")
    B, N, Hkv, D = Kt[0].shape
    K = path_node.shape[1] - 1
    bf = torch.bfloat16
    arr = C.c_void_p * n
    ptrs = [arr(*[_dev(t, bf, name).value for t in ts]) for ts, name in ((Kt, "Kt"), (Vt, "Vt"), (Kp, "Kp"), (Vp, "Vp"))]
    for ts in (Kt, Vt):
        if any(tuple(t.shape) != (B, N, Hkv, D) for t in ts):
            raise SpecrollError("commit_path_layers: tree K/V shapes differ between layers")
    for ts in (Kp, Vp):
        if any(tuple(t.shape) != tuple(Kp[0].shape) for t in ts):
            raise SpecrollError("commit_path_layers: page pools differ between layers")
    rc = lib().specroll_commit_path_layers(
        B, N, K, Hkv, D, n, ptrs[0], ptrs[1], _dev(path_node, torch.int32, "path_node"),
        _dev(n_acc, torch.int32, "n_acc"), ptrs[2], ptrs[3], C.c_int64(Kp[0].shape[0]),
        _dev(page_table, torch.int32, "page_table"), _dev(page_indptr, torch.int32, "page_indptr"),
        _dev(kv_len, torch.int32, "kv_len"), _dev(kv_len_out, torch.int32, "kv_len_out"),
        _dev(status, torch.int32, "status"), _stream())
    _check(rc, "specroll_commit_path_layers")


def gather_hidden(hidden, term_node, out=None):
    """specroll_gather_hidden: hidden[B,N,d] bf16, term_node[B] -> h_next[B,d]."""
    B, N, d = hidden.shape
    if out is None:
        out = _empty((B, d), dtype=torch.bfloat16, device=hidden.device)
    rc = lib().specroll_gather_hidden(B, N, d, _dev(hidden, torch.bfloat16, "hidden"),
                                      _dev(term_node, torch.int32, "term_node"), _dev(out, torch.bfloat16, "h_next"),
                                      _stream())
    _check(rc, "specroll_gather_hidden")
    return out


# ----------------------------------------------------------------------------------- verify


def verify_workspace_bytes(B, N, K, k, V, temperature=1.0) -> int:
    desc = VerifyDesc(B, N, K, k, V, temperature, 0)
    return int(lib().specroll_verify_workspace_bytes(C.byref(desc)))


def verify_nucleus_workspace_bytes(B, N, K, k, V, temperature=1.0) -> int:
    desc = VerifyDesc(B, N, K, k, V, temperature, 0)
    return int(lib().specroll_verify_nucleus_workspace_bytes(C.byref(desc)))


def verify(logits, parent, tree_tok, tree_cand, cand_id, cand_logit, u_acc, u_fin, temperature=1.0,
           workspace=None, out: Optional[Dict[str, torch.Tensor]] = None, flags: int = 0) -> Dict[str, torch.Tensor]:
    """specroll_verify.  Device tensors in, dict of device tensors out."""
    parent = _host_i32(parent, "parent")
    B, N, V = logits.shape
    _, K, k = cand_id.shape
    if parent.shape[0] != N or tuple(tree_tok.shape) != (B, N) or tuple(u_acc.shape) != (B, N):
        raise SpecrollError("verify: inconsistent shapes")
    desc = VerifyDesc(B, N, K, k, V, temperature, flags)
    dev = logits.device
    i32, f32 = torch.int32, torch.float32
    if out is None:
        out = {"n_acc": _empty(B, dtype=i32, device=dev),
               "path_node": _empty((B, K + 1), dtype=i32, device=dev),
               "out_tok": _empty((B, K + 1), dtype=i32, device=dev),
               "term_node": _empty(B, dtype=i32, device=dev),
               "term_kind": _empty(B, dtype=i32, device=dev),
               "row_max": _empty((B, N), dtype=f32, device=dev),
               "row_sum": _empty((B, N), dtype=f32, device=dev),
               "min_margin": _empty(B, dtype=f32, device=dev)}
    if workspace is None:
        workspace = _workspace(lib().specroll_verify_workspace_bytes(C.byref(desc)), dev)
    rc = lib().specroll_verify(
        C.byref(desc), _dev(logits, torch.bfloat16, "logits"), parent.ctypes.data_as(C.c_void_p),
        _dev(tree_tok, i32, "tree_tok"), _dev(tree_cand, torch.uint8, "tree_cand"),
        _dev(cand_id, i32, "cand_id"), _dev(cand_logit, f32, "cand_logit"), _dev(u_acc, f32, "u_acc"),
        _dev(u_fin, f32, "u_fin"), _dev(out["n_acc"], i32, "n_acc"), _dev(out["path_node"], i32, "path_node"),
        _dev(out["out_tok"], i32, "out_tok"), _dev(out["term_node"], i32, "term_node"),
        _dev(out["term_kind"], i32, "term_kind"), _dev(out["row_max"], f32, "row_max"),
        _dev(out["row_sum"], f32, "row_sum"), _dev(out.get("min_margin"), f32, "min_margin"),
        C.c_void_p(workspace.data_ptr()), C.c_size_t(workspace.numel()), _stream())
    _check(rc, "specroll_verify")
    return out


def verify_fused(hidden, W, parent, tree_tok, tree_cand, cand_id, cand_logit, u_acc, u_fin, temperature=1.0):
    """Exact verification from the target's final hidden states, without the logits tensor: the projection with
    fused row statistics over all (sequence, node) rows (specroll_target_head_stats), the walk on the target logits
    of the candidate tokens (specroll_verify_walk_sparse), then the one row per sequence that the terminal draw
    needs (specroll_gather_hidden, specroll_target_head_rows, specroll_verify_terminal_rows).
    hidden [B, N, d] bf16, W [V, d] bf16; the other arguments as for ``verify``.  Returns the same dict."""
    parent = _host_i32(parent, "parent")
    B, N, d = hidden.shape
    V = W.shape[0]
    _, K, k = cand_id.shape
    desc = VerifyDesc(B, N, K, k, V, temperature, 0)
    dev = hidden.device
    i32, f32 = torch.int32, torch.float32
    want = _empty((B * N, k), dtype=i32, device=dev)
    rc = lib().specroll_verify_want_ids(C.byref(desc), parent.ctypes.data_as(C.c_void_p), _dev(cand_id, i32, "cand_id"),
                                        _dev(want, i32, "want_id"), _stream())
    _check(rc, "specroll_verify_want_ids")
    st = target_head_stats(hidden.reshape(B * N, d), W, want, temperature=temperature)
    out = {"n_acc": _empty(B, dtype=i32, device=dev), "path_node": _empty((B, K + 1), dtype=i32, device=dev),
           "out_tok": _empty((B, K + 1), dtype=i32, device=dev), "term_node": _empty(B, dtype=i32, device=dev),
           "term_kind": _empty(B, dtype=i32, device=dev), "row_max": st["row_max"].reshape(B, N),
           "row_sum": st["row_sum"].reshape(B, N), "min_margin": _empty(B, dtype=f32, device=dev)}
    ws = _workspace(lib().specroll_verify_workspace_bytes(C.byref(desc)), dev)
    rc = lib().specroll_verify_walk_sparse(
        C.byref(desc), _dev(st["want_logit"], torch.bfloat16, "cand_target"), _dev(st["row_max"], f32, "row_max"),
        _dev(st["row_sum"], f32, "row_sum"), parent.ctypes.data_as(C.c_void_p), _dev(tree_tok, i32, "tree_tok"),
        _dev(tree_cand, torch.uint8, "tree_cand"), _dev(cand_id, i32, "cand_id"), _dev(cand_logit, f32, "cand_logit"),
        _dev(u_acc, f32, "u_acc"), _dev(out["n_acc"], i32, "n_acc"), _dev(out["path_node"], i32, "path_node"),
        _dev(out["out_tok"], i32, "out_tok"), _dev(out["term_node"], i32, "term_node"),
        _dev(out["term_kind"], i32, "term_kind"), _dev(out["min_margin"], f32, "min_margin"),
        C.c_void_p(ws.data_ptr()), C.c_size_t(ws.numel()), _stream())
    _check(rc, "specroll_verify_walk_sparse")
    h_term = gather_hidden(hidden, out["term_node"])
    rows = target_head_rows(h_term, W)
    rc = lib().specroll_verify_terminal_rows(
        C.byref(desc), _dev(rows, torch.bfloat16, "term_logits"), _dev(st["row_max"], f32, "row_max"),
        _dev(out["n_acc"], i32, "n_acc"), _dev(out["term_node"], i32, "term_node"), _dev(u_fin, f32, "u_fin"),
        _dev(out["out_tok"], i32, "out_tok"), C.c_void_p(ws.data_ptr()), C.c_size_t(ws.numel()), _stream())
    _check(rc, "specroll_verify_terminal_rows")
    return out


def verify_nucleus(logits, parent, tree_tok, tree_cand, cand_id, cand_logit, u_acc, u_fin, top_p, temperature=1.0,
                   workspace=None, out: Optional[Dict[str, torch.Tensor]] = None,
                   flags: int = 0) -> Dict[str, torch.Tensor]:
    """specroll_verify_nucleus: verification against nucleus-truncated target distributions.
    The returned dict also holds nucleus_thr and nucleus_sum [B,N]."""
    parent = _host_i32(parent, "parent")
    B, N, V = logits.shape
    _, K, k = cand_id.shape
    if parent.shape[0] != N or tuple(tree_tok.shape) != (B, N) or tuple(u_acc.shape) != (B, N):
        raise SpecrollError("verify_nucleus: inconsistent shapes")
    desc = VerifyDesc(B, N, K, k, V, temperature, flags)
    dev = logits.device
    i32, f32 = torch.int32, torch.float32
    if out is None:
        out = {"n_acc": _empty(B, dtype=i32, device=dev),
               "path_node": _empty((B, K + 1), dtype=i32, device=dev),
               "out_tok": _empty((B, K + 1), dtype=i32, device=dev),
               "term_node": _empty(B, dtype=i32, device=dev),
               "term_kind": _empty(B, dtype=i32, device=dev),
               "row_max": _empty((B, N), dtype=f32, device=dev),
               "row_sum": _empty((B, N), dtype=f32, device=dev),
               "min_margin": _empty(B, dtype=f32, device=dev),
               "nucleus_thr": _empty((B, N), dtype=f32, device=dev),
               "nucleus_sum": _empty((B, N), dtype=f32, device=dev)}
    if workspace is None:
        workspace = _workspace(lib().specroll_verify_nucleus_workspace_bytes(C.byref(desc)), dev)
    rc = lib().specroll_verify_nucleus(
        C.byref(desc), C.c_float(top_p), _dev(logits, torch.bfloat16, "logits"), parent.ctypes.data_as(C.c_void_p),
        _dev(tree_tok, i32, "tree_tok"), _dev(tree_cand, torch.uint8, "tree_cand"),
        _dev(cand_id, i32, "cand_id"), _dev(cand_logit, f32, "cand_logit"), _dev(u_acc, f32, "u_acc"),
        _dev(u_fin, f32, "u_fin"), _dev(out["n_acc"], i32, "n_acc"), _dev(out["path_node"], i32, "path_node"),
        _dev(out["out_tok"], i32, "out_tok"), _dev(out["term_node"], i32, "term_node"),
        _dev(out["term_kind"], i32, "term_kind"), _dev(out["row_max"], f32, "row_max"),
        _dev(out["row_sum"], f32, "row_sum"), _dev(out.get("min_margin"), f32, "min_margin"),
        _dev(out.get("nucleus_thr"), f32, "nucleus_thr"), _dev(out.get("nucleus_sum"), f32, "nucleus_sum"),
        C.c_void_p(workspace.data_ptr()), C.c_size_t(workspace.numel()), _stream())
    _check(rc, "specroll_verify_nucleus")
    return out


def reflex_feedback_workspace_bytes(R, k, k_support, d, V, temperature=1.0, eps=1e-6) -> int:
    desc = FeedbackDesc(R, k, k_support, d, V, temperature, eps, 0, 0.0)
    return int(lib().specroll_reflex_feedback_workspace_bytes(C.byref(desc)))


def reflex_feedback(logits, rec_row, row_max, row_sum, cand_id, cand_logit, y_star, W, rho, rec_mem, m, k_support,
                    temperature=1.0, eps=1e-6, workspace=None, severity_min=None, want_e=False):
    """specroll_reflex_feedback(_ex): verifier feedback of R matured records, memory ``m`` updated in place.
    logits [rows, V] bf16 (any leading shape), row_max/row_sum [rows]; returns d_dist, d_cov, tv, severity [R]
    (and e [R, d] with ``want_e``).  With ``severity_min`` the update is weighted by the severity and
    observations below it are discarded."""
    V = logits.shape[-1]
    R, k = cand_id.shape
    d = W.shape[1]
    weighted = severity_min is not None
    desc = FeedbackDesc(R, k, k_support, d, V, temperature, eps, FEEDBACK_SEVERITY if weighted else 0,
                        float(severity_min) if weighted else 0.0)
    dev = logits.device
    f32, i32 = torch.float32, torch.int32
    out = {n: _empty(R, dtype=f32, device=dev) for n in ("d_dist", "d_cov", "tv", "severity")}
    if want_e:
        out["e"] = _empty((R, d), dtype=f32, device=dev)
    need = lib().specroll_reflex_feedback_workspace_bytes(C.byref(desc))
    if need == 0:
        raise SpecrollError("reflex_feedback: invalid descriptor")
    if workspace is None:
        workspace = _workspace(need, dev)
    rc = lib().specroll_reflex_feedback_ex(
        C.byref(desc), _dev(logits, torch.bfloat16, "logits"), _dev(rec_row, i32, "rec_row"),
        _dev(row_max, f32, "row_max"), _dev(row_sum, f32, "row_sum"), _dev(cand_id, i32, "cand_id"),
        _dev(cand_logit, f32, "cand_logit"), _dev(y_star, i32, "y_star"), _dev(W, torch.bfloat16, "W"),
        _dev(rho, f32, "rho"), _dev(rec_mem, i32, "rec_mem"), _dev(m, f32, "m"), _dev(out["d_dist"], f32, "d_dist"),
        _dev(out["d_cov"], f32, "d_cov"), _dev(out["tv"], f32, "tv"), _dev(out["severity"], f32, "severity"),
        _dev(out["e"], f32, "e") if want_e else None, C.c_void_p(workspace.data_ptr()),
        C.c_size_t(workspace.numel()), _stream())
    _check(rc, "specroll_reflex_feedback_ex")
    return out


def reflex_sketch(X, Pi, rows=None):
    """specroll_reflex_sketch: normalised random-projection sketches [R, rank] of the rows of X [*, d] fp32
    (``rows`` [R] i32 selects them; all rows in order when None) under the projection Pi [rank, d] fp32."""
    rank, d = Pi.shape
    R = X.shape[0] if rows is None else rows.shape[0]
    out = _empty((R, rank), dtype=torch.float32, device=X.device)
    rc = lib().specroll_reflex_sketch(C.c_int32(R), C.c_int32(d), C.c_int32(rank), _dev(X, torch.float32, "X"),
                                      _dev(rows, torch.int32, "rows") if rows is not None else None,
                                      _dev(Pi, torch.float32, "Pi"), _dev(out, torch.float32, "sketch"), _stream())
    _check(rc, "specroll_reflex_sketch")
    return out


def reflex_gate(s, xi, slot, keep, n, mean, M2, n_fb, m, horizon, n_align_min, n_fb_min, alpha_lo, alpha_hi,
                z_delta=0.60, mem_eps=1e-12):
    """specroll_reflex_gate: alignments of R matured records into the slots' online moments (n, mean, M2, n_fb
    updated in place), then the reliability score and the correction ratio of every slot.  Returns a [R],
    rel [S], alpha [S]."""
    R, rank = s.shape
    S, d = m.shape
    H = n_align_min.shape[0]
    dev = m.device
    f32, i32 = torch.float32, torch.int32
    desc = GateDesc(R, S, d, rank, H, z_delta, mem_eps, 0)
    out = {"a": _empty(max(R, 1), dtype=f32, device=dev)[:R], "rel": _empty(S, dtype=f32, device=dev),
           "alpha": _empty(S, dtype=f32, device=dev)}
    rc = lib().specroll_reflex_gate(
        C.byref(desc), _dev(s, f32, "s"), _dev(xi, f32, "xi"), _dev(slot, i32, "slot"),
        _dev(keep, torch.uint8, "keep") if keep is not None else None, _dev(n, i32, "n"), _dev(mean, f32, "mean"),
        _dev(M2, f32, "M2"), _dev(n_fb, i32, "n_fb"), _dev(m, f32, "m"), _dev(horizon, i32, "horizon"),
        _dev(n_align_min, i32, "n_align_min"), _dev(n_fb_min, i32, "n_fb_min"), _dev(alpha_lo, f32, "alpha_lo"),
        _dev(alpha_hi, f32, "alpha_hi"), _dev(out["a"], f32, "a"), _dev(out["rel"], f32, "rel"),
        _dev(out["alpha"], f32, "alpha"), _stream())
    _check(rc, "specroll_reflex_gate")
    return out


def target_head_stats(H, W, want_id=None, temperature=1.0, workspace=None):
    """specroll_target_head_stats: row_max, row_sum [R] and want_logit [R, kw] (bf16) of l = bf16(H W^T) without
    storing l.  H [R, d] bf16, W [V, d] bf16, want_id [R, kw] i32 or None."""
    R, d = H.shape
    V = W.shape[0]
    kw = 0 if want_id is None else want_id.shape[1]
    dev = H.device
    out = {"row_max": _empty(R, dtype=torch.float32, device=dev),
           "row_sum": _empty(R, dtype=torch.float32, device=dev),
           "want_logit": _empty((R, kw), dtype=torch.bfloat16, device=dev)}
    need = lib().specroll_target_head_stats_workspace_bytes(C.c_int32(R), C.c_int32(d), C.c_int32(V))
    if need == 0:
        raise SpecrollError("target_head_stats: invalid shape")
    if workspace is None:
        workspace = _workspace(need, dev)
    rc = lib().specroll_target_head_stats(
        C.c_int32(R), C.c_int32(d), C.c_int32(V), C.c_float(temperature), _dev(H, torch.bfloat16, "H"),
        _dev(W, torch.bfloat16, "W"), _dev(want_id, torch.int32, "want_id") if kw else None, C.c_int32(kw),
        _dev(out["row_max"], torch.float32, "row_max"), _dev(out["row_sum"], torch.float32, "row_sum"),
        _dev(out["want_logit"], torch.bfloat16, "want_logit") if kw else None, C.c_void_p(workspace.data_ptr()),
        C.c_size_t(workspace.numel()), _stream())
    _check(rc, "specroll_target_head_stats")
    return out


def target_head_rows(H, W, out=None):
    """specroll_target_head_rows: logits [R, V] bf16 = bf16(H W^T)."""
    R, d = H.shape
    V = W.shape[0]
    if out is None:
        out = _empty((R, V), dtype=torch.bfloat16, device=H.device)
    status = torch.zeros(1, dtype=torch.int32, device=H.device)
    rc = lib().specroll_target_head_rows(C.c_int32(R), C.c_int32(d), C.c_int32(V), _dev(H, torch.bfloat16, "H"),
                                         _dev(W, torch.bfloat16, "W"), _dev(out, torch.bfloat16, "logits"),
                                         _dev(status, torch.int32, "status"), _stream())
    _check(rc, "specroll_target_head_rows")
    return out


def verify_static(logits, parent, tree_tok, tree_cand, cand_id, cand_logit, u_acc, u_fin, temperature=1.0,
                  out: Dict[str, torch.Tensor] = None) -> Dict[str, torch.Tensor]:
    """specroll_verify_static: verification for hosts that cannot allocate a workspace.

    The scratch is a fixed array inside the library, so this wrapper passes none.  The output
    tensors must be supplied by a caller that truly cannot allocate (``out``); when ``out`` is
    omitted they are created here with torch for convenience, which is the only allocation on
    this path and is the caller's, not the library's.  Raises SpecrollError with the library's
    message when B or B*k exceed the entry point's fixed limits.
    """
    parent = _host_i32(parent, "parent")
    B, N, V = logits.shape
    _, K, k = cand_id.shape
    if parent.shape[0] != N or tuple(tree_tok.shape) != (B, N) or tuple(u_acc.shape) != (B, N):
        raise SpecrollError("verify_static: inconsistent shapes")
    desc = VerifyDesc(B, N, K, k, V, temperature, 0)
    dev = logits.device
    i32, f32 = torch.int32, torch.float32
    if out is None:
        out = {"n_acc": _empty(B, dtype=i32, device=dev),
               "path_node": _empty((B, K + 1), dtype=i32, device=dev),
               "out_tok": _empty((B, K + 1), dtype=i32, device=dev),
               "term_node": _empty(B, dtype=i32, device=dev),
               "term_kind": _empty(B, dtype=i32, device=dev),
               "row_max": _empty((B, N), dtype=f32, device=dev),
               "row_sum": _empty((B, N), dtype=f32, device=dev),
               "min_margin": _empty(B, dtype=f32, device=dev)}
    rc = lib().specroll_verify_static(
        C.byref(desc), _dev(logits, torch.bfloat16, "logits"), parent.ctypes.data_as(C.c_void_p),
        _dev(tree_tok, i32, "tree_tok"), _dev(tree_cand, torch.uint8, "tree_cand"),
        _dev(cand_id, i32, "cand_id"), _dev(cand_logit, f32, "cand_logit"), _dev(u_acc, f32, "u_acc"),
        _dev(u_fin, f32, "u_fin"), _dev(out["n_acc"], i32, "n_acc"), _dev(out["path_node"], i32, "path_node"),
        _dev(out["out_tok"], i32, "out_tok"), _dev(out["term_node"], i32, "term_node"),
        _dev(out["term_kind"], i32, "term_kind"), _dev(out["row_max"], f32, "row_max"),
        _dev(out["row_sum"], f32, "row_sum"), _dev(out.get("min_margin"), f32, "min_margin"), _stream())
    _check(rc, "specroll_verify_static")
    return out


# ----------------------------------------------------------------------------------- helpers


def bf16_tensor(bits: np.ndarray, device="cuda") -> torch.Tensor:
    """uint16 bf16 bit patterns (host numpy) -> bf16 tensor on the device."""
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16))
    return t.view(torch.bfloat16).to(device)


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    """bf16 tensor -> uint16 bit patterns on the host."""
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
