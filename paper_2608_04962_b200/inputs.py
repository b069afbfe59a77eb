"""Seeded synthetic inputs for the SpecRoll per-step hot path.

This module serves both the CUDA path and the CPU oracle.  It holds no arithmetic of
the method itself: only random draws, storage-format conversion (fp32 <-> bf16 bit
patterns) and the workload shapes.  All host arrays are numpy; bf16 tensors are carried
as ``uint16`` bit patterns.

Workload shapes stand in for the paper's 1.5B-14B rollout workloads (the paper's
datasets and checkpoints are not used): Gaussian weights/activations, log-normal
KV-cache lengths, a best-first sparse tree topology shared by the batch, and target
logits with one boosted "mode" token per node so that the realised accepted length is in
the range the paper's tables report.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Dict, List, Optional, Tuple

import numpy as np

# ----------------------------------------------------------------------------------
# storage-format helpers (bf16 carried as uint16 bit patterns)
# ----------------------------------------------------------------------------------


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (nearest, ties to even); returns the uint16 bit patterns."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = (u + np.uint32(0x7FFF) + lsb) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns (uint16) to fp32 exactly."""
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def rng(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(seed))


def uniforms24(seed: int, shape) -> np.ndarray:
    """float32 uniforms in [0, 1) carrying 24 random bits."""
    return rng(seed).random(size=shape, dtype=np.float32)


# ----------------------------------------------------------------------------------
# workload configurations
# ----------------------------------------------------------------------------------


@dataclass(frozen=True)
class Workload:
    name: str
    cfg_id: int               # enters the seeds: seed = 1000 * cfg_id + stream
    B: int                    # sequences
    N: int                    # tree nodes per sequence (root = node 0 = anchor)
    K: int                    # future-token heads
    k: int                    # per-head top-k (candidate support size)
    d: int                    # hidden size
    V: int                    # vocabulary
    Hq: int
    Hkv: int
    D: int
    kv_kind: str              # "uniform" | "lognormal"
    kv_a: int                 # uniform: low ; lognormal: median
    kv_b: int                 # uniform: high; lognormal: max
    layers: int               # attention layers per step (public depth of the named model)
    temperature: float = 1.0
    clip_c: float = 0.0
    alpha_heads: Tuple[float, ...] = ()
    fixed_parent: Optional[Tuple[int, ...]] = None

    @property
    def G(self) -> int:
        return self.Hq // self.Hkv


# seed streams
S_UNIFORM, S_WEIGHT, S_ACT, S_KV, S_LEN, S_LOGIT, S_REFLEX = range(7)

_PAPER_ALPHA = (0.025, 0.010, 0.006, 0.004, 0.003)  # upper ends of the paper's intervals, extended

WORKLOADS: Dict[str, Workload] = {
    "tiny": Workload("tiny", 1, B=4, N=8, K=3, k=2, d=256, V=1024, Hq=4, Hkv=2, D=64,
                     kv_kind="uniform", kv_a=64, kv_b=256, layers=2, clip_c=0.1,
                     alpha_heads=(0.1, 0.1, 0.1),
                     fixed_parent=(-1, 0, 0, 1, 1, 2, 3, 3)),
    "qwen1.5b": Workload("qwen1.5b", 2, B=256, N=16, K=4, k=8, d=1536, V=151936, Hq=12, Hkv=2,
                         D=128, kv_kind="lognormal", kv_a=1500, kv_b=8192, layers=28,
                         alpha_heads=_PAPER_ALPHA[:4]),
    "qwen7b": Workload("qwen7b", 3, B=128, N=32, K=4, k=8, d=3584, V=152064, Hq=28, Hkv=4,
                       D=128, kv_kind="lognormal", kv_a=3000, kv_b=16384, layers=28,
                       alpha_heads=_PAPER_ALPHA[:4]),
    "qwen14b": Workload("qwen14b", 4, B=64, N=48, K=5, k=8, d=5120, V=152064, Hq=40, Hkv=8,
                        D=128, kv_kind="lognormal", kv_a=4000, kv_b=16384, layers=48,
                        alpha_heads=_PAPER_ALPHA[:5]),
}

# concurrency-aware sweep on the 7B shape: (B, N, KV median)
SWEEP_POINTS = ((256, 8, 2000), (128, 16, 2760), (64, 24, 3800),
                (32, 32, 5250), (16, 48, 7250), (8, 64, 10000))
for _i, (_B, _N, _med) in enumerate(SWEEP_POINTS):
    WORKLOADS[f"sweep7b_B{_B}"] = replace(WORKLOADS["qwen7b"], name=f"sweep7b_B{_B}",
                                          cfg_id=50 + _i, B=_B, N=_N, kv_a=_med)


def scaled(w: Workload, **kw) -> Workload:
    """A reduced copy of a workload (same seeds stream id) for parity tests."""
    return replace(w, **kw)


# ----------------------------------------------------------------------------------
# tree topology (shared by all sequences of a call)
# ----------------------------------------------------------------------------------


def best_first_topology(N: int, K: int, k: int) -> np.ndarray:
    """Parent array of an N-node sparse tree, depth <= K, fan-out <= k.

    Root has score 1; the rank-r child of u has score score(u) * 0.6 * 0.5**r.  Nodes are
    taken in order of decreasing score (ties: shallower, then lower parent, then lower
    rank) and renumbered breadth-first, so parent[n] < n.
    """
    assert N >= 1
    # node records: (score, depth, parent_tmp_id, rank)
    nodes = [(1.0, 0, -1, 0)]
    n_children = [0]
    while len(nodes) < N:
        best = None
        for u, (su, du, _, _) in enumerate(nodes):
            r = n_children[u]
            if du >= K or r >= k:
                continue
            cand = (-(su * 0.6 * 0.5 ** r), du + 1, u, r)
            if best is None or cand < best:
                best = cand
        if best is None:
            raise ValueError(f"cannot place {N} nodes with depth<={K}, fan-out<={k}")
        negs, dep, u, r = best
        nodes.append((-negs, dep, u, r))
        n_children.append(0)
        n_children[u] += 1
    # breadth-first renumbering (stable in (depth, parent's new id, rank))
    order = [0]
    new_id = {0: 0}
    head = 0
    while head < len(order):
        u = order[head]
        head += 1
        kids = sorted((i for i, nd in enumerate(nodes) if nd[2] == u), key=lambda i: nodes[i][3])
        for c in kids:
            new_id[c] = len(order)
            order.append(c)
    parent = np.full(N, -1, dtype=np.int32)
    for old, nd in enumerate(nodes):
        if old != 0:
            parent[new_id[old]] = new_id[nd[2]]
    assert all(parent[n] < n for n in range(1, N))
    return parent


def paper_540_topology() -> np.ndarray:
    """N=10: root -> 5 children; 4 depth-2 nodes placed 2/1/1 under the first three."""
    return np.array([-1, 0, 0, 0, 0, 0, 1, 1, 2, 3], dtype=np.int32)


def topology(w: Workload) -> np.ndarray:
    if w.fixed_parent is not None and len(w.fixed_parent) == w.N:
        return np.array(w.fixed_parent, dtype=np.int32)
    return best_first_topology(w.N, w.K, w.k)


def node_depths(parent: np.ndarray) -> np.ndarray:
    dep = np.zeros(len(parent), dtype=np.int32)
    for n in range(1, len(parent)):
        dep[n] = dep[parent[n]] + 1
    return dep


# ----------------------------------------------------------------------------------
# per-entry-point inputs
# ----------------------------------------------------------------------------------


def kv_lengths(w: Workload) -> np.ndarray:
    g = rng(1000 * w.cfg_id + S_LEN)
    if w.kv_kind == "uniform":
        return g.integers(w.kv_a, w.kv_b + 1, size=w.B).astype(np.int32)
    z = g.standard_normal(w.B)
    L = np.rint(np.clip(w.kv_a * np.exp(0.7 * z), 64, w.kv_b))
    return L.astype(np.int32)


def _normal_bf16(g: np.random.Generator, shape, std: float) -> np.ndarray:
    x = g.standard_normal(size=shape, dtype=np.float32)
    if std != 1.0:
        x *= np.float32(std)
    return f32_to_bf16_bits(x)


def propose_inputs(w: Workload, peaked: bool = False) -> dict:
    """Inputs of the proposal step.  ``peaked`` draws h ~ N(0,1) (well-separated top-k)."""
    gw = rng(1000 * w.cfg_id + S_WEIGHT)
    ga = rng(1000 * w.cfg_id + S_ACT)
    gr = rng(1000 * w.cfg_id + S_REFLEX)
    out = {}
    out["A"] = _normal_bf16(gw, (w.K, w.d, w.d), 0.02)       # row = output unit
    out["bias"] = _normal_bf16(gw, (w.K, w.d), 0.02)
    out["W"] = _normal_bf16(gw, (w.V, w.d), 0.02)            # row = token
    out["h"] = _normal_bf16(ga, (w.B, w.d), 1.0 if peaked else 0.02)
    out["anchor"] = ga.integers(0, w.V, size=w.B).astype(np.int32)
    out["m"] = gr.standard_normal(size=(w.B, w.K, w.d), dtype=np.float32)
    on = gr.random(size=(w.B, w.K)) < 0.5
    ah = np.zeros(w.K, dtype=np.float32)
    n_a = min(w.K, len(w.alpha_heads))
    ah[:n_a] = w.alpha_heads[:n_a]
    alpha = on.astype(np.float32) * ah[None, :]
    if w.clip_c > 0:
        # a quarter of the active pairs exceed the clip so that it binds
        big = gr.random(size=(w.B, w.K)) < 0.25
        alpha = np.where(big & on, np.float32(2.0 * w.clip_c), alpha).astype(np.float32)
    else:
        gr.random(size=(w.B, w.K))
    out["alpha"] = alpha
    out["parent"] = topology(w)
    out["u_draw"] = uniforms24(1000 * w.cfg_id + S_UNIFORM, (w.B, w.N))
    return out


def attn_inputs(w: Workload, layer: int = 0) -> dict:
    g = rng(1000 * w.cfg_id + S_KV + 100 * layer)
    L = kv_lengths(w)
    indptr = np.zeros(w.B + 1, dtype=np.int32)
    np.cumsum(L, out=indptr[1:])
    T = int(indptr[-1])
    out = {"kv_indptr": indptr, "parent": topology(w)}
    out["Q"] = _normal_bf16(g, (w.B, w.N, w.Hq, w.D), 1.0)
    out["Kc"] = _normal_bf16(g, (T, w.Hkv, w.D), 1.0)
    out["Vc"] = _normal_bf16(g, (T, w.Hkv, w.D), 1.0)
    out["Kt"] = _normal_bf16(g, (w.B, w.N, w.Hkv, w.D), 1.0)
    out["Vt"] = _normal_bf16(g, (w.B, w.N, w.Hkv, w.D), 1.0)
    return out


def target_logits(w: Workload, parent: np.ndarray, tree_tok: np.ndarray, flat: bool = False,
                  boost: float = 14.0) -> np.ndarray:
    """Target logits [B, N, V] as bf16 bits.

    Background N(0,1); per node a mode token gets +boost: the node's first child token
    w.p. 0.45, its second child w.p. 0.15, else a uniformly random token.  ``flat``
    instead draws N(0, 0.03^2) with no mode (exercises tiny acceptance ratios).
    """
    g = rng(1000 * w.cfg_id + S_LOGIT)
    B, N, V = w.B, w.N, w.V
    x = g.standard_normal(size=(B, N, V), dtype=np.float32)
    if flat:
        x *= np.float32(0.03)
        return f32_to_bf16_bits(x)
    kids: List[List[int]] = [[] for _ in range(N)]
    for n in range(1, N):
        kids[int(parent[n])].append(n)
    pick = g.random(size=(B, N))
    rnd_tok = g.integers(0, V, size=(B, N))
    for n in range(N):
        mode = rnd_tok[:, n].copy()
        if len(kids[n]) >= 1:
            sel = pick[:, n] < 0.45
            mode[sel] = tree_tok[sel, kids[n][0]]
        if len(kids[n]) >= 2:
            sel = (pick[:, n] >= 0.45) & (pick[:, n] < 0.60)
            mode[sel] = tree_tok[sel, kids[n][1]]
        x[np.arange(B), n, mode] += np.float32(boost)
    return f32_to_bf16_bits(x)


def verify_uniforms(w: Workload) -> Tuple[np.ndarray, np.ndarray]:
    g = rng(1000 * w.cfg_id + S_UNIFORM + 500)
    u_acc = g.random(size=(w.B, w.N), dtype=np.float32)
    u_fin = g.random(size=(w.B,), dtype=np.float32)
    return u_acc, u_fin


def synthetic_candidates(w: Workload) -> Tuple[np.ndarray, np.ndarray]:
    """Stand-in candidate lists for verification-only runs: per (sequence, head) k distinct
    token ids with logits sorted in descending order (gaps of a peaked head distribution)."""
    g = rng(1000 * w.cfg_id + S_ACT + 700)
    ids = np.empty((w.B, w.K, w.k), dtype=np.int32)
    for b in range(w.B):
        for hd in range(w.K):
            ids[b, hd] = g.choice(w.V, size=w.k, replace=False)
    lg = -np.sort(-(g.standard_normal(size=(w.B, w.K, w.k), dtype=np.float32) * np.float32(1.5)), axis=-1)
    return ids, np.ascontiguousarray(lg, dtype=np.float32)


def paged_cache(Kc, Vc, kv_indptr, spare_tokens: int, seed: int):
    """Scatters a contiguous ragged cache into a pool of 128-token pages in a seeded random page order.

    Every sequence gets room for ``spare_tokens`` more tokens; the pool has a few unused pages and unused rows
    hold a bit pattern that is not zero, so that a kernel reading beyond a sequence's length would be noticed.
    Returns Kp, Vp [n_pages, 128, Hkv, D] (uint16 bit patterns), page_table, page_indptr, kv_len (int32)."""
    PAGE = 128
    kv_indptr = np.asarray(kv_indptr, np.int64)
    B = kv_indptr.shape[0] - 1
    kv_len = (kv_indptr[1:] - kv_indptr[:-1]).astype(np.int32)
    own = (kv_len.astype(np.int64) + spare_tokens + PAGE - 1) // PAGE
    page_indptr = np.zeros(B + 1, np.int32)
    np.cumsum(own, out=page_indptr[1:])
    n_pages = int(page_indptr[-1]) + 3
    g = rng(seed)
    page_table = g.permutation(n_pages)[: int(page_indptr[-1])].astype(np.int32)
    Kp = np.full((n_pages, PAGE) + Kc.shape[1:], 0x7F00, np.uint16)   # bf16 2^127: poisons any sum it enters
    Vp = np.full((n_pages, PAGE) + Vc.shape[1:], 0x7F00, np.uint16)
    for b in range(B):
        for i in range(int((kv_len[b] + PAGE - 1) // PAGE)):
            lo = int(kv_indptr[b]) + i * PAGE
            hi = min(int(kv_indptr[b + 1]), lo + PAGE)
            page = int(page_table[page_indptr[b] + i])
            Kp[page, : hi - lo] = Kc[lo:hi]
            Vp[page, : hi - lo] = Vc[lo:hi]
    return Kp, Vp, page_table, page_indptr, kv_len

