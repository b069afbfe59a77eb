"""Pins for the oracle's nucleus-truncated verification.

The kept set is pinned by a hand-worked table, by brute force over all top sets of a small vocabulary, and by
what the rule implies (tie groups stay whole, the kept mass brackets top_p); the walk by the statistical fact it
must reproduce: the emitted tokens are exact samples of the *truncated* target distribution."""
import itertools

import numpy as np

from oracle import ref
from paper_2608_04962_b200 import inputs as I

N_TRIALS = 400_000


def _bits(x):
    return I.f32_to_bf16_bits(np.asarray(x, np.float32))


def _root_only(logits_row, top_p, T=1.0, u_fin=0.5):
    """Verification of a lone root: nothing to accept, the token is drawn from the (truncated) root distribution."""
    V = logits_row.shape[0]
    lg = _bits(logits_row)[None, None, :]
    parent = np.array([-1], np.int32)
    cid = np.zeros((1, 1, 1), np.int32)
    cl = np.zeros((1, 1, 1), np.float32)
    return ref.verify(lg, parent, np.zeros((1, 1), np.int32), np.full((1, 1), 255, np.uint8), cid, cl,
                      np.zeros((1, 1), np.float32), np.array([u_fin], np.float32), temperature=T, top_p=top_p)


def test_hand_worked_table_with_a_tie_at_the_cut():
    # probabilities 1/2, 1/4, 1/8, 1/8 (logits are exact in bf16; T = 1/ln 2 makes p = 2^l / sum)
    row = np.array([0.0, -1.0, -2.0, -2.0])
    T = 1.0 / np.log(2.0)
    o = _root_only(row, 0.70, T)                       # 1/2 + 1/4 = 0.75 >= 0.70: two tokens
    assert np.isclose(o["nucleus_thr"][0, 0], -1.0) and np.isclose(o["nucleus_sum"][0, 0], 1.5, rtol=1e-6)
    assert np.isclose(o["nucleus_margin"][0], 0.05, atol=1e-6)      # 0.75 - 0.70
    o = _root_only(row, 0.80, T)                       # needs the third token, whose twin comes along: all four
    assert np.isclose(o["nucleus_thr"][0, 0], -2.0) and np.isclose(o["nucleus_sum"][0, 0], 2.0, rtol=1e-6)
    assert np.isclose(o["nucleus_margin"][0], 0.05, atol=1e-6)      # 0.80 - 0.75
    o = _root_only(row, 0.40, T)                       # the largest token alone
    assert np.isclose(o["nucleus_thr"][0, 0], 0.0) and np.isclose(o["nucleus_sum"][0, 0], 1.0, rtol=1e-6)


def test_kept_set_against_brute_force_over_all_top_sets():
    g = I.rng(7)
    for trial in range(30):
        V = 7
        row = _bits(np.round(g.standard_normal(V) * 2) / 2).astype(np.uint16)      # coarse values: ties are common
        vals = I.bf16_bits_to_f32(row).astype(np.float64)
        p = np.exp(vals - vals.max())
        p /= p.sum()
        top_p = float(np.float32(g.uniform(0.05, 0.99)))
        # brute force: among all sets that are closed under "at least as probable as a member", the smallest
        # one whose mass reaches top_p
        best = None
        for r in range(1, V + 1):
            for S in itertools.combinations(range(V), r):
                lo = min(p[list(S)])
                if any(p[v] >= lo and v not in S for v in range(V)):
                    continue
                if p[list(S)].sum() >= top_p and (best is None or len(S) < len(best)):
                    best = S
            if best is not None:
                break
        o = _root_only(vals, top_p)
        kept = vals >= o["nucleus_thr"][0, 0] - 1e-9
        assert set(np.nonzero(kept)[0]) == set(best), (trial, vals, top_p)
        assert np.isclose(o["nucleus_sum"][0, 0] / o["row_sum"][0, 0], p[list(best)].sum(), rtol=1e-9)


def test_disabled_and_degenerate_thresholds():
    w = I.WORKLOADS["tiny"]
    x = I.propose_inputs(w, peaked=True)
    d = ref.propose(x["h"], x["anchor"], x["A"], x["bias"], x["W"], x["m"], x["alpha"], x["parent"], x["u_draw"],
                    k=w.k, clip_c=w.clip_c)
    lg = I.target_logits(w, x["parent"], d["tree_tok"])
    u_acc, u_fin = I.verify_uniforms(w)
    args = (lg, x["parent"], d["tree_tok"], d["tree_cand"], d["cand_id"], d["cand_logit"], u_acc, u_fin)
    base = ref.verify(*args)
    off = ref.verify(*args, top_p=1.0)
    for key in ("n_acc", "path_node", "out_tok", "term_node", "term_kind"):
        assert np.array_equal(base[key], off[key])
    # a vanishing threshold keeps the most probable tie group only: every emitted non-accepted token is an argmax
    tiny = ref.verify(*args, top_p=1e-6)
    vals = I.bf16_bits_to_f32(lg)
    for b in range(w.B):
        node, tok = tiny["term_node"][b], tiny["out_tok"][b, tiny["n_acc"][b]]
        assert vals[b, node, tok] == vals[b, node].max()


def test_emitted_tokens_follow_the_truncated_target():
    # root with two children; its first child has two children.  Vocabulary 8, k = 4.
    parent = np.array([-1, 0, 0, 1, 1], np.int32)
    g = I.rng(31)
    p = g.dirichlet(np.full(8, 0.7), size=5)
    p = np.maximum(p, 1e-3)
    p /= p.sum(-1, keepdims=True)
    node_logits = np.log(p)
    # heads that resemble their targets, so that candidates fall inside the nucleus and get accepted
    head = np.stack([node_logits[0], node_logits[1]]) + 0.7 * g.standard_normal((2, 8))
    order = np.argsort(-head, axis=-1)[:, :4]
    cand_id, cand_logit = order.astype(np.int32), np.take_along_axis(head, order, -1).astype(np.float32)
    top_p = 0.8
    n = N_TRIALS
    lg = np.broadcast_to(_bits(node_logits)[None], (n, 5, 8)).copy()
    cid = np.broadcast_to(cand_id[None], (n, 2, 4)).copy()
    cl = np.broadcast_to(cand_logit[None], (n, 2, 4)).copy()
    u = I.uniforms24(77, (3, n, 5))
    draw = ref.tree_draw(parent, np.zeros(n, np.int32), cid, cl, u[0])
    out = ref.verify(lg, parent, draw["tree_tok"], draw["tree_cand"], cid, cl, u[1], u[2][:, 0].copy(), top_p=top_p)
    # the truncated tables, computed here from the definition (sort, cut, renormalise; no ties in these tables)
    P = np.exp(I.bf16_bits_to_f32(_bits(node_logits)).astype(np.float64))
    P /= P.sum(-1, keepdims=True)
    Pt = np.zeros_like(P)
    for i in range(5):
        idx = np.argsort(-P[i])
        cut = int(np.searchsorted(np.cumsum(P[i][idx]), top_p)) + 1
        Pt[i, idx[:cut]] = P[i, idx[:cut]]
        Pt[i] /= Pt[i].sum()
    assert (Pt == 0).any()                                    # the cut removes something

    def within(freq, q, m):
        return np.abs(freq - q) < 4.5 * np.sqrt(np.maximum(q * (1 - q), 1e-12) / m) + 1e-9

    first = np.bincount(out["out_tok"][:, 0], minlength=8) / n
    assert within(first, Pt[0], n).all(), (first, Pt[0])
    assert (first[Pt[0] == 0] == 0).all()                     # a token outside the nucleus is never emitted
    for c in (1, 2):
        sel = (out["n_acc"] >= 1) & (out["path_node"][:, 1] == c)
        m = int(sel.sum())
        assert m > 2000, (c, m)
        f2 = np.bincount(out["out_tok"][sel, 1], minlength=8) / m
        assert within(f2, Pt[c], m).all(), (c, f2, Pt[c])
