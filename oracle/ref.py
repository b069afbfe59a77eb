"""ctypes front-end of the CPU oracle (``specroll_ref.c``).

TEST INFRASTRUCTURE, NOT PRODUCT CODE: only the tests, the smoke check and the
benchmark's CPU-baseline leg import this module.  It never touches the CUDA library.
All arrays are host numpy arrays; bf16 tensors are uint16 bit patterns.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "specroll_ref.c")
_LIB = os.path.join(_HERE, "libspecroll_ref.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP across independent rows only)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.specroll_ref_num_threads.restype = C.c_int
    return _lib


def num_threads() -> int:
    return int(lib().specroll_ref_num_threads())


def _p(a: Optional[np.ndarray]):
    if a is None:
        return None
    assert a.flags["C_CONTIGUOUS"], "oracle arrays must be contiguous"
    return a.ctypes.data_as(C.c_void_p)


def _chk(rc: int, what: str):
    if rc != 0:
        raise ValueError(f"oracle {what}: invalid arguments (code {rc})")


def _as(a, dt):
    return None if a is None else np.ascontiguousarray(a, dtype=dt)


def round_bf16(x: np.ndarray) -> np.ndarray:
    x = _as(x, np.float64)
    out = np.empty(x.shape, np.uint16)
    lib().specroll_ref_round_bf16(C.c_int64(x.size), _p(x), _p(out))
    return out


def heads(h, A, bias, m=None, alpha=None, gamma=None, beta=None, ln_eps=1e-5, rms_eps=1e-6,
          clip_c=0.0):
    """Returns dict(xhat bf16, z fp64 (uncorrected), zc fp64 (corrected), zt bf16), all [B,K,d]."""
    h, A, bias = _as(h, np.uint16), _as(A, np.uint16), _as(bias, np.uint16)
    B, d = h.shape
    K = A.shape[0]
    assert A.shape == (K, d, d) and bias.shape == (K, d)
    m, alpha = _as(m, np.float32), _as(alpha, np.float32)
    gamma, beta = _as(gamma, np.uint16), _as(beta, np.uint16)
    xhat = np.empty((B, K, d), np.uint16)
    z = np.empty((B, K, d), np.float64)
    zc = np.empty((B, K, d), np.float64)
    zt = np.empty((B, K, d), np.uint16)
    rc = lib().specroll_ref_heads(B, K, d, C.c_double(ln_eps), C.c_double(rms_eps),
                                  C.c_double(clip_c), _p(h), _p(A), _p(bias), _p(gamma), _p(beta),
                                  _p(m), _p(alpha), _p(xhat), _p(z), _p(zc), _p(zt))
    _chk(rc, "heads")
    return {"xhat": xhat, "z": z, "zc": zc, "zt": zt}


def prehead(h, m, alpha, rms_eps=1e-6, clip_c=0.0):
    """The correction applied to the last hidden state (secondary form).  h [B,d] bf16 bits, m [B,d] fp32,
    alpha [B] fp32.  Returns dict(hc fp64 unrounded, ht bf16 bits)."""
    h = _as(h, np.uint16)
    m, alpha = _as(m, np.float32), _as(alpha, np.float32)
    B, d = h.shape
    hc = np.empty((B, d), np.float64)
    ht = np.empty((B, d), np.uint16)
    _chk(lib().specroll_ref_prehead(B, d, C.c_double(rms_eps), C.c_double(clip_c), _p(h), _p(m), _p(alpha), _p(hc),
                                    _p(ht)), "prehead")
    return {"hc": hc, "ht": ht}


def lm_logits(zt, W):
    zt, W = _as(zt, np.uint16), _as(W, np.uint16)
    zt2 = zt.reshape(-1, zt.shape[-1])
    M, d = zt2.shape
    V = W.shape[0]
    out = np.empty((M, V), np.float64)
    _chk(lib().specroll_ref_lm_logits(M, V, d, _p(zt2), _p(W), _p(out)), "lm_logits")
    return out


def topk(logits, k):
    logits = _as(logits, np.float64)
    M, V = logits.shape
    cid = np.empty((M, k), np.int32)
    cl = np.empty((M, k), np.float32)
    _chk(lib().specroll_ref_topk(M, V, k, _p(logits), _p(cid), _p(cl)), "topk")
    return cid, cl


def lm_topk(zt, W, k):
    zt, W = _as(zt, np.uint16), _as(W, np.uint16)
    zt2 = zt.reshape(-1, zt.shape[-1])
    M, d = zt2.shape
    V = W.shape[0]
    cid = np.empty((M, k), np.int32)
    cl = np.empty((M, k), np.float32)
    _chk(lib().specroll_ref_lm_topk(M, V, d, k, _p(zt2), _p(W), _p(cid), _p(cl)), "lm_topk")
    return cid, cl


def tree_draw(parent, anchor, cand_id, cand_logit, u_draw, temperature=1.0):
    parent, anchor = _as(parent, np.int32), _as(anchor, np.int32)
    cand_id, cand_logit = _as(cand_id, np.int32), _as(cand_logit, np.float32)
    u_draw = _as(u_draw, np.float32)
    B, K, k = cand_id.shape
    N = parent.shape[0]
    assert u_draw.shape == (B, N) and anchor.shape == (B,)
    tok = np.empty((B, N), np.int32)
    tc = np.empty((B, N), np.uint8)
    sq = np.empty((B, N), np.float64)
    rc = lib().specroll_ref_tree_draw(B, N, K, k, C.c_double(float(np.float32(temperature))), _p(parent), _p(anchor),
                                      _p(cand_id), _p(cand_logit), _p(u_draw), _p(tok), _p(tc),
                                      _p(sq))
    _chk(rc, "tree_draw")
    return {"tree_tok": tok, "tree_cand": tc, "slot_q": sq}


def propose(h, anchor, A, bias, W, m, alpha, parent, u_draw, k, temperature=1.0, ln_eps=1e-5,
            rms_eps=1e-6, clip_c=0.0, gamma=None, beta=None, pre_head=False):
    """pre_head: m [B,d] and alpha [B] correct the hidden state before the heads (no correction after them)."""
    if pre_head:
        h = prehead(h, m, alpha, rms_eps=rms_eps, clip_c=clip_c)["ht"]
        m, alpha = None, None
    h, A, bias, W = (_as(x, np.uint16) for x in (h, A, bias, W))
    anchor, parent = _as(anchor, np.int32), _as(parent, np.int32)
    m, alpha, u_draw = _as(m, np.float32), _as(alpha, np.float32), _as(u_draw, np.float32)
    gamma, beta = _as(gamma, np.uint16), _as(beta, np.uint16)
    B, d = h.shape
    K, V, N = A.shape[0], W.shape[0], parent.shape[0]
    cid = np.empty((B, K, k), np.int32)
    cl = np.empty((B, K, k), np.float32)
    tok = np.empty((B, N), np.int32)
    tc = np.empty((B, N), np.uint8)
    sq = np.empty((B, N), np.float64)
    rc = lib().specroll_ref_propose(B, N, K, k, d, V, C.c_double(float(np.float32(temperature))), C.c_double(ln_eps),
                                    C.c_double(rms_eps), C.c_double(clip_c), _p(h), _p(anchor),
                                    _p(A), _p(bias), _p(gamma), _p(beta), _p(W), _p(m), _p(alpha),
                                    _p(parent), _p(u_draw), _p(cid), _p(cl), _p(tok), _p(tc), _p(sq))
    _chk(rc, "propose")
    return {"cand_id": cid, "cand_logit": cl, "tree_tok": tok, "tree_cand": tc, "slot_q": sq}


def tree_attn(Q, Kc, Vc, kv_indptr, Kt, Vt, parent, scale=None, want_lse=False):
    Q, Kc, Vc, Kt, Vt = (_as(x, np.uint16) for x in (Q, Kc, Vc, Kt, Vt))
    kv_indptr, parent = _as(kv_indptr, np.int32), _as(parent, np.int32)
    B, N, Hq, D = Q.shape
    Hkv = Kt.shape[2]
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    O64 = np.empty((B, N, Hq, D), np.float64)
    Obf = np.empty((B, N, Hq, D), np.uint16)
    lse = np.empty((B, N, Hq), np.float64) if want_lse else None
    rc = lib().specroll_ref_tree_attn(B, N, Hq, Hkv, D, C.c_double(scale), _p(Q), _p(Kc), _p(Vc),
                                      _p(kv_indptr), _p(Kt), _p(Vt), _p(parent), _p(O64), _p(Obf),
                                      _p(lse))
    _chk(rc, "tree_attn")
    out = {"O64": O64, "Obf": Obf}
    if want_lse:
        out["lse"] = lse
    return out


def verify(logits, parent, tree_tok, tree_cand, cand_id, cand_logit, u_acc, u_fin,
           temperature=1.0, top_p=None):
    if top_p is not None:
        return _verify_nucleus(logits, parent, tree_tok, tree_cand, cand_id, cand_logit, u_acc, u_fin,
                               temperature, top_p)
    logits = _as(logits, np.uint16)
    parent, tree_tok = _as(parent, np.int32), _as(tree_tok, np.int32)
    tree_cand, cand_id = _as(tree_cand, np.uint8), _as(cand_id, np.int32)
    cand_logit, u_acc, u_fin = (_as(x, np.float32) for x in (cand_logit, u_acc, u_fin))
    B, N, V = logits.shape
    _, K, k = cand_id.shape
    n_acc = np.empty(B, np.int32)
    path = np.empty((B, K + 1), np.int32)
    out_tok = np.empty((B, K + 1), np.int32)
    term_node = np.empty(B, np.int32)
    term_kind = np.empty(B, np.int32)
    row_max = np.empty((B, N), np.float64)
    row_sum = np.empty((B, N), np.float64)
    mm = np.empty(B, np.float64)
    fm = np.empty(B, np.float64)
    rc = lib().specroll_ref_verify(B, N, K, k, V, C.c_double(float(np.float32(temperature))), _p(logits), _p(parent),
                                   _p(tree_tok), _p(tree_cand), _p(cand_id), _p(cand_logit),
                                   _p(u_acc), _p(u_fin), _p(n_acc), _p(path), _p(out_tok),
                                   _p(term_node), _p(term_kind), _p(row_max), _p(row_sum), _p(mm),
                                   _p(fm))
    _chk(rc, "verify")
    return {"n_acc": n_acc, "path_node": path, "out_tok": out_tok, "term_node": term_node,
            "term_kind": term_kind, "row_max": row_max, "row_sum": row_sum, "min_margin": mm,
            "fin_margin": fm}


def _verify_nucleus(logits, parent, tree_tok, tree_cand, cand_id, cand_logit, u_acc, u_fin, temperature, top_p):
    logits = _as(logits, np.uint16)
    parent, tree_tok = _as(parent, np.int32), _as(tree_tok, np.int32)
    tree_cand, cand_id = _as(tree_cand, np.uint8), _as(cand_id, np.int32)
    cand_logit, u_acc, u_fin = (_as(x, np.float32) for x in (cand_logit, u_acc, u_fin))
    B, N, V = logits.shape
    _, K, k = cand_id.shape
    n_acc = np.empty(B, np.int32)
    path = np.empty((B, K + 1), np.int32)
    out_tok = np.empty((B, K + 1), np.int32)
    term_node = np.empty(B, np.int32)
    term_kind = np.empty(B, np.int32)
    row_max = np.empty((B, N), np.float64)
    row_sum = np.empty((B, N), np.float64)
    mm = np.empty(B, np.float64)
    fm = np.empty(B, np.float64)
    thr = np.full((B, N), np.nan)
    ksum = np.full((B, N), np.nan)
    nm = np.empty(B, np.float64)
    rc = lib().specroll_ref_verify_nucleus(
        B, N, K, k, V, C.c_double(float(np.float32(temperature))), C.c_double(float(np.float32(top_p))), _p(logits),
        _p(parent), _p(tree_tok), _p(tree_cand), _p(cand_id), _p(cand_logit), _p(u_acc), _p(u_fin), _p(n_acc),
        _p(path), _p(out_tok), _p(term_node), _p(term_kind), _p(row_max), _p(row_sum), _p(mm), _p(fm), _p(thr),
        _p(ksum), _p(nm))
    _chk(rc, "verify_nucleus")
    return {"n_acc": n_acc, "path_node": path, "out_tok": out_tok, "term_node": term_node,
            "term_kind": term_kind, "row_max": row_max, "row_sum": row_sum, "min_margin": mm,
            "fin_margin": fm, "nucleus_thr": thr, "nucleus_sum": ksum, "nucleus_margin": nm}


def node_budget(C_hw, B_active, N_min=1, N_max=10) -> int:
    f = lib().specroll_ref_node_budget
    f.restype = C.c_int32
    return int(f(C.c_int32(C_hw), C.c_int32(B_active), C.c_int32(N_min), C.c_int32(N_max)))


# ----------------------------------------------------------------------------------- between two steps
# The paper names "accepted-path KV extraction" among the contents of generation time and gives no formula; the
# page layout is the library's.  These are written out as plain loops over tokens: a paged cache is read token
# by token through the table, and a committed path is appended token by token.

PAGE_TOKENS = 128


def paged_to_contiguous(Kp, Vp, page_table, page_indptr, kv_len):
    """The cache that a page table describes, as the contiguous ragged arrays of ``tree_attn``:
    token t of sequence b lives in pool page page_table[page_indptr[b] + t // 128] at row t % 128."""
    Kp, Vp = _as(Kp, np.uint16), _as(Vp, np.uint16)
    page_table, page_indptr, kv_len = (_as(x, np.int32) for x in (page_table, page_indptr, kv_len))
    B = kv_len.shape[0]
    indptr = np.zeros(B + 1, np.int32)
    np.cumsum(kv_len, out=indptr[1:])
    Kc = np.zeros((int(indptr[-1]),) + Kp.shape[2:], np.uint16)
    Vc = np.zeros_like(Kc)
    for b in range(B):
        for t in range(int(kv_len[b])):
            page = int(page_table[page_indptr[b] + t // PAGE_TOKENS])
            Kc[indptr[b] + t] = Kp[page, t % PAGE_TOKENS]
            Vc[indptr[b] + t] = Vp[page, t % PAGE_TOKENS]
    return Kc, Vc, indptr


def tree_attn_paged(Q, Kp, Vp, page_table, page_indptr, kv_len, Kt, Vt, parent, scale=None, want_lse=False):
    """Tree attention over a paged cache = tree attention over the cache the table describes."""
    Kc, Vc, indptr = paged_to_contiguous(Kp, Vp, page_table, page_indptr, kv_len)
    return tree_attn(Q, Kc, Vc, indptr, Kt, Vt, parent, scale=scale, want_lse=want_lse)


def commit_path(Kt, Vt, path_node, n_acc, Kp, Vp, page_table, page_indptr, kv_len):
    """Appends tree rows path_node[b, 0..n_acc[b]] of every sequence to its paged cache.  Returns new copies
    (Kp, Vp, kv_len); a token that does not fit the sequence's own pages is dropped and reported in ``overflow``."""
    Kt, Vt, Kp, Vp = (_as(x, np.uint16) for x in (Kt, Vt, Kp, Vp))
    path_node, n_acc, page_table, page_indptr, kv_len = (
        _as(x, np.int32) for x in (path_node, n_acc, page_table, page_indptr, kv_len))
    Kp, Vp, new_len = Kp.copy(), Vp.copy(), kv_len.copy()
    overflow = False
    for b in range(kv_len.shape[0]):
        own = int(page_indptr[b + 1] - page_indptr[b])
        for i in range(int(n_acc[b]) + 1):
            pos = int(kv_len[b]) + i
            if pos // PAGE_TOKENS >= own:
                overflow = True
                continue
            page = int(page_table[page_indptr[b] + pos // PAGE_TOKENS])
            Kp[page, pos % PAGE_TOKENS] = Kt[b, path_node[b, i]]
            Vp[page, pos % PAGE_TOKENS] = Vt[b, path_node[b, i]]
        new_len[b] = kv_len[b] + n_acc[b] + 1
    return {"Kp": Kp, "Vp": Vp, "kv_len": new_len, "overflow": overflow}


def gather_hidden(hidden, term_node):
    hidden, term_node = _as(hidden, np.uint16), _as(term_node, np.int32)
    return np.stack([hidden[b, term_node[b]] for b in range(hidden.shape[0])])


# ----------------------------------------------------------------------------------- verifier feedback
def reflex_feedback(logits_rows, W, cand_id, cand_logit, y_star, m, rho, k_support, temperature=1.0, eps=1e-6,
                    severity=False, severity_min=0.03):
    """Verifier-derived feedback of matured proposals and the memory update (Sec. 3.3 / 3.4: Eq. "support",
    "distdir", "covdir", the RMS normalisation, Eq. "unified-feedback", Eq. "ema"; the magnitudes d_dist and
    d_cov from Eq. "acceptance-gap-decomposition").  One record per row, written out step by step in fp64:

      p = softmax(logits / T) over the vocabulary; q = softmax(cand_logit / T) on the k candidates C, zero elsewhere
      S = C  u  Top_kS(p)  u  {y*}                (ties of Top by (logit desc, id asc))
      p_S, q_S = p, q renormalised on S           (q lives on C, a subset of S, so q_S = q)
      r_dist = sum_{v in S} (p_S(v) - q_S(v)) W_v
      C* = Top_k(p),  O = C* \\ C,  b* = weakest candidate (last of the list, which is sorted by logit)
      r_cov = sum_{y in O} p_S(y) (W_y - W_b*)
      d_dist = p(C) TV(p_C, q_C),  d_cov = p(C*) - p(C)
      rbar = r / (RMS(r) + eps);  g = d_dist rbar_dist + d_cov rbar_cov;  e = (d_dist + d_cov) g / (RMS(g) + eps)
      m <- rho m + (1 - rho) e

    With ``severity`` (App. "Implementation details", paragraph "Verifier-derived feedback"): the observation's
    severity  w = clip(0.3 TV(p_S, q_S) + 0.7 p_out, 0, 1),  p_out = 1 - p(C) the target mass outside the
    candidates, weights it,  m <- rho m + (1 - rho) w e,  and an observation with w < severity_min is discarded
    (the memory row keeps its value).  w and TV(p_S, q_S) are returned either way.

    logits_rows [R,V] and W [V,d] are bf16 bit patterns; m [R,d], rho [R] floats.  Returns the new memory and the
    intermediate quantities."""
    logits_rows, W = _as(logits_rows, np.uint16), _as(W, np.uint16)
    cand_id, y_star = _as(cand_id, np.int32), _as(y_star, np.int32)
    cand_logit = np.asarray(cand_logit, np.float32).astype(np.float64)
    m = np.asarray(m, np.float64)
    rho = np.asarray(rho, np.float64)
    R, V = logits_rows.shape
    k = cand_id.shape[1]
    d = W.shape[1]
    T = float(np.float32(temperature))
    if k_support < k:
        raise ValueError("the support budget must cover the target's top-k (k_support >= k)")
    Wf = (W.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    out = {"m": np.empty((R, d)), "e": np.empty((R, d)), "d_dist": np.empty(R), "d_cov": np.empty(R),
           "tv": np.empty(R), "p_C": np.empty(R), "support": [], "tv_S": np.empty(R), "w": np.empty(R),
           "kept": np.ones(R, bool)}
    rms = lambda v: np.sqrt(np.mean(v * v))
    for r in range(R):
        l = (logits_rows[r].astype(np.uint32) << 16).view(np.float32).astype(np.float64)
        p = np.exp((l - l.max()) / T)
        p /= p.sum()
        C = [int(c) for c in cand_id[r]]
        q_c = np.exp((cand_logit[r] - cand_logit[r].max()) / T)
        q_c /= q_c.sum()
        order = np.lexsort((np.arange(V), -l))            # by (logit desc, id asc)
        top_s = [int(v) for v in order[:k_support]]
        S = []
        for v in C + top_s + [int(y_star[r])]:
            if v not in S:
                S.append(v)
        pS = {v: p[v] for v in S}
        tot = sum(pS.values())
        pS = {v: x / tot for v, x in pS.items()}
        qS = {v: 0.0 for v in S}
        for j, c in enumerate(C):
            qS[c] += q_c[j]
        r_dist = np.zeros(d)
        for v in S:
            r_dist += (pS[v] - qS[v]) * Wf[v]
        c_star = [int(v) for v in order[:k]]
        O = [v for v in c_star if v not in C]
        b_star = C[-1]
        r_cov = np.zeros(d)
        for y in O:
            r_cov += pS[y] * (Wf[y] - Wf[b_star])
        pC = sum(p[c] for c in C)
        tv = 0.5 * sum(abs(p[c] / pC - q_c[j]) for j, c in enumerate(C))
        d_dist = pC * tv
        d_cov = sum(p[v] for v in c_star) - pC
        g = d_dist * r_dist / (rms(r_dist) + eps) + d_cov * r_cov / (rms(r_cov) + eps)
        e = (d_dist + d_cov) * g / (rms(g) + eps)
        tv_S = 0.5 * sum(abs(pS[v] - qS[v]) for v in S)
        w = min(1.0, max(0.0, 0.3 * tv_S + 0.7 * (1.0 - pC)))
        out["tv_S"][r], out["w"][r] = tv_S, w
        if not severity:
            out["m"][r] = rho[r] * m[r] + (1.0 - rho[r]) * e
        elif w < severity_min:
            out["m"][r] = m[r]
            out["kept"][r] = False
        else:
            out["m"][r] = rho[r] * m[r] + (1.0 - rho[r]) * w * e
        out["e"][r] = e
        out["d_dist"][r], out["d_cov"][r], out["tv"][r], out["p_C"][r] = d_dist, d_cov, tv, pC
        out["support"].append(S)
    return out


def reflex_sketch(X, Pi):
    """Normalised random-projection sketch (Sec. 3.4 "Reliability from delayed alignment"; App. "Implementation
    details": rank 24, seed 29): sketch(x) = Pi x / ||Pi x||_2, the zero vector when Pi x = 0.  X [R,d], Pi [rank,d]
    (the projection's entries are an input: both sides are given the same matrix)."""
    X, Pi = np.asarray(X, np.float64), np.asarray(Pi, np.float64)
    out = np.zeros((X.shape[0], Pi.shape[0]))
    for r in range(X.shape[0]):
        y = np.array([float(np.dot(Pi[i], X[r])) for i in range(Pi.shape[0])])
        nrm = np.sqrt(np.sum(y * y))
        if nrm > 0.0:
            out[r] = y / nrm
    return out


def reflex_gate(s, xi, slot, keep, n, mean, M2, n_fb, m, horizon, n_align_min, n_fb_min, alpha_lo, alpha_hi,
                z_delta=0.60, mem_eps=1e-12):
    """Reliability score and gate of every (trajectory, horizon) slot (Sec. 3.4 Eq. "reliability-score" and the
    indicator of Eq. "reflex-correction"; App. "Implementation details": exact online sample moments, minimum
    counts per horizon, correction interval per horizon).

    Records r = 0..R-1 are taken in order; a kept record of slot j = slot[r] contributes its realised alignment
    a_r = cos(s_r, xi_r) (0 when either sketch is the zero vector) to the slot's running count, mean and sum of
    squared deviations (Welford's recurrences, which give the exact sample mean and variance), and counts as one
    feedback observation.  Then, per slot with horizon h:
        Rel = mean - z_delta * sqrt(M2 / (n - 1)) / sqrt(n)          (n >= 2; otherwise not eligible)
        open = n >= n_align_min[h]  and  n_fb >= n_fb_min[h]  and  Rel > 0  and  RMS(m_slot) > mem_eps
        alpha = alpha_lo[h] + (alpha_hi[h] - alpha_lo[h]) * min(Rel, 1)   if open, else 0
    (the paper places the ratio in [alpha_lo, alpha_hi] for an eligible score without giving the map; the linear one
    in the score is this implementation's reading).  Returns a [R] (nan for records not kept) and the updated
    state, Rel [S] (-inf when n < 2) and alpha [S]."""
    s, xi = np.asarray(s, np.float64), np.asarray(xi, np.float64)
    n, n_fb = np.array(n, np.int64), np.array(n_fb, np.int64)
    mean, M2 = np.array(mean, np.float64), np.array(M2, np.float64)
    m = np.asarray(m, np.float64)
    R, S = s.shape[0], n.shape[0]
    a = np.full(R, np.nan)
    for r in range(R):
        if keep is not None and not keep[r]:
            continue
        j = int(slot[r])
        ns, nx = np.sqrt(np.sum(s[r] ** 2)), np.sqrt(np.sum(xi[r] ** 2))
        a[r] = float(np.dot(s[r], xi[r]) / (ns * nx)) if ns > 0.0 and nx > 0.0 else 0.0
        n[j] += 1
        delta = a[r] - mean[j]
        mean[j] += delta / n[j]
        M2[j] += delta * (a[r] - mean[j])
        n_fb[j] += 1
    rel = np.full(S, -np.inf)
    alpha = np.zeros(S)
    for j in range(S):
        h = int(horizon[j])
        if n[j] >= 2:
            rel[j] = mean[j] - z_delta * np.sqrt(M2[j] / (n[j] - 1)) / np.sqrt(n[j])
        rms = np.sqrt(np.mean(m[j] ** 2))
        if n[j] >= n_align_min[h] and n_fb[j] >= n_fb_min[h] and rel[j] > 0.0 and rms > mem_eps:
            alpha[j] = alpha_lo[h] + (alpha_hi[h] - alpha_lo[h]) * min(rel[j], 1.0)
    return {"a": a, "n": n, "mean": mean, "M2": M2, "n_fb": n_fb, "rel": rel, "alpha": alpha}


def target_head(H, W, temperature=1.0, want_id=None):
    """The target's vocabulary projection followed by what the verification takes from it (Sec. 3.2, App. B.2):
    l = bf16(H W^T) with H [R,d], W [V,d] bf16 bit patterns (products and sums in fp64, one rounding to bf16, as a
    projection that stores bf16 logits does), row_max = max_v l, row_sum = sum_v exp((l - row_max)/T), and the logits
    at want_id [R,kw].  Returns the logits as bf16 bit patterns too."""
    H, W = _as(H, np.uint16), _as(W, np.uint16)
    Hf = (H.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    Wf = (W.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    T = float(np.float32(temperature))
    l64 = Hf @ Wf.T
    bits = round_bf16(l64)
    l = (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    row_max = l.max(-1)
    row_sum = np.exp((l - row_max[:, None]) / T).sum(-1)
    out = {"logits": bits, "row_max": row_max, "row_sum": row_sum}
    if want_id is not None:
        out["want_logit"] = np.take_along_axis(bits, np.asarray(want_id, np.int64), -1)
    return out

