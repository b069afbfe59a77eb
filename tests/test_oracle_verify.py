"""Pins for the exact-verification oracle (no GPU).

The node-wise accept/resample walk is an algorithm, so it is pinned by what the paper
proves about it and by what it prints: the emitted token follows the target
distribution (10^6 seeded trials on a vocabulary of 8), the first-slot acceptance equals
1 - TV(p, q), the worked example's 3/5 and 13/30, the sandwich bound, hand-traced cases,
and library routines for the softmax statistics and the inverse-CDF draw.
"""
import os
from fractions import Fraction

import numpy as np
from scipy.special import logsumexp, softmax

from oracle import ref
from paper_2608_04962_b200 import inputs as I

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "acceptance_worked_example.txt")
N_TRIALS = 1_000_000


def _bits(x):
    return I.f32_to_bf16_bits(np.asarray(x, np.float32))


def _f64(bits):
    return I.bf16_bits_to_f32(bits).astype(np.float64)


def _golden():
    out = {}
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        name, *vals = line.split()
        out[name] = [Fraction(v) for v in vals]
    return out


def _run(parent, node_logits, cand_id, cand_logit, n_trials, seed, T=1.0):
    """Draw the tree with the oracle's proposal law, then verify; same tables for all trials."""
    N, V = node_logits.shape
    K, k = cand_id.shape
    cid = np.broadcast_to(cand_id[None].astype(np.int32), (n_trials, K, k)).copy()
    cl = np.broadcast_to(cand_logit[None].astype(np.float32), (n_trials, K, k)).copy()
    lg = np.broadcast_to(_bits(node_logits)[None], (n_trials, N, V)).copy()
    u = I.uniforms24(seed, (3, n_trials, N))
    draw = ref.tree_draw(parent, np.zeros(n_trials, np.int32), cid, cl, u[0], temperature=T)
    out = ref.verify(lg, parent, draw["tree_tok"], draw["tree_cand"], cid, cl, u[1], u[2][:, 0].copy(),
                     temperature=T)
    out.update(draw)
    return out


def _within(freq, p, n, sig=4.5):
    return np.abs(freq - p) < sig * np.sqrt(np.maximum(p * (1 - p), 1e-12) / n) + 1e-9


def test_worked_example_numbers_are_consistent():
    g = _golden()
    p = g["p"]
    C = [int(c) - 1 for c in g["C"]]
    for q_name, a_name in (("q_C", "A1_q_C"), ("q_C'", "A1_q_C'")):
        q = dict(zip(C, g[q_name]))
        assert sum(min(p[v], q.get(v, Fraction(0))) for v in range(3)) == g[a_name][0]
    assert [p[c] / sum(p[c] for c in C) for c in C] == g["p_C"]


def test_worked_example_first_slot_acceptance_three_fifths_and_thirteen_thirtieths():
    g = _golden()
    p = np.array([float(v) for v in g["p"]])
    C = np.array([int(c) - 1 for c in g["C"]])
    parent = np.array([-1, 0], np.int32)
    node_logits = np.log(np.stack([p, p]))
    p_b = softmax(_f64(_bits(node_logits[0])))            # target after bf16 storage of the logits
    assert np.abs(p_b - p).max() < 2.5e-3
    for q_name, a_name, seed in (("q_C", "A1_q_C", 1), ("q_C'", "A1_q_C'", 2)):
        q = np.array([float(v) for v in g[q_name]])
        out = _run(parent, node_logits, C[None, :], np.log(q)[None, :], N_TRIALS, seed)
        acc = np.mean(out["n_acc"] == 1)
        a_exact = float(g[a_name][0])
        a_bf16 = np.minimum(p_b[C], q).sum()                # same identity at the stored logits
        assert abs(a_bf16 - a_exact) < 2.5e-3
        assert _within(acc, a_bf16, N_TRIALS), (acc, a_bf16, a_exact)
        assert abs(acc - a_exact) < 4e-3


def test_hand_traced_single_node():
    # p = (1/2, 2/5, 1/10) (up to bf16 storage), C = {0, 2} with q = (5/6, 1/6), two slots.
    # Slot 1 draws token 0 when u_draw < 5/6: ratio = (1/2)/(5/6) = 3/5.
    # Rejected -> residual [p - q]_+ = (0, 2/5, 0) -> (0, 1, 0); slot 2 is token 2 with q = 1:
    # ratio 0 -> rejected; fallback is token 1 whatever u_fin is.
    p = np.array([0.5, 0.4, 0.1])
    parent = np.array([-1, 0, 0], np.int32)
    lg = np.broadcast_to(_bits(np.log(p))[None, None], (4, 3, 3)).copy()
    cid = np.broadcast_to(np.array([[[0, 2]]], np.int32), (4, 1, 2)).copy()
    cl = np.broadcast_to(np.log(np.array([[[5 / 6, 1 / 6]]], np.float32)), (4, 1, 2)).copy()
    u_draw = np.array([[0, 0.1, 0.0]] * 4, np.float32)
    d = ref.tree_draw(parent, np.full(4, 7, np.int32), cid, cl, u_draw)
    assert d["tree_tok"].tolist() == [[7, 0, 2]] * 4
    np.testing.assert_allclose(d["slot_q"], [[1, 5 / 6, 1.0]] * 4, rtol=1e-6)
    u_acc = np.array([[0, 0.55, 0.5], [0, 0.65, 0.0], [0, 0.65, 0.999], [0, 0.59, 0.5]], np.float32)
    u_fin = np.array([0.3, 0.0, 0.99999, 0.7], np.float32)
    o = ref.verify(lg, parent, d["tree_tok"], d["tree_cand"], cid, cl, u_acc, u_fin)
    assert o["n_acc"].tolist() == [1, 0, 0, 1]
    assert o["term_kind"].tolist() == [1, 0, 0, 1]            # bonus after an accepted leaf, else fallback
    assert o["term_node"].tolist() == [1, 0, 0, 1]
    assert o["out_tok"][1].tolist() == [1, -1] and o["out_tok"][2].tolist() == [1, -1]
    assert o["path_node"].tolist() == [[0, 1], [0, -1], [0, -1], [0, 1]]
    # bonus tokens come from p of the leaf by inverse CDF in token order: 0.3 -> 0, 0.7 -> 1
    assert o["out_tok"][0].tolist() == [0, 0] and o["out_tok"][3].tolist() == [0, 1]
    np.testing.assert_allclose(o["min_margin"][0], abs(0.55 - 0.6), atol=2e-3)
    np.testing.assert_allclose(o["min_margin"][1], 0.0, atol=1e-12)   # slot 2: |0 - 0|


def test_hand_traced_second_slot_accepts_from_the_residual():
    # p = (0.2, 0.3, 0.5), C = {0, 2}, q1 = (0.8, 0.2).  Slot 1 = token 0: ratio 0.25.
    # Rejected -> [p - q1]_+ = (0, 0.3, 0.3) -> r = (0, 1/2, 1/2).  Slot 2 = token 2, q2 = 1:
    # ratio 1/2.  Accept iff u < 1/2.
    p = np.array([0.2, 0.3, 0.5])
    parent = np.array([-1, 0, 0], np.int32)
    lg = np.broadcast_to(_bits(np.log(p))[None, None], (2, 3, 3)).copy()
    cid = np.broadcast_to(np.array([[[0, 2]]], np.int32), (2, 1, 2)).copy()
    cl = np.broadcast_to(np.log(np.array([[[0.8, 0.2]]], np.float32)), (2, 1, 2)).copy()
    d = ref.tree_draw(parent, np.zeros(2, np.int32), cid, cl, np.zeros((2, 3), np.float32))
    u_acc = np.array([[0, 0.3, 0.45], [0, 0.3, 0.55]], np.float32)
    o = ref.verify(lg, parent, d["tree_tok"], d["tree_cand"], cid, cl, u_acc, np.array([0.9, 0.9], np.float32))
    assert o["n_acc"].tolist() == [1, 0]
    assert o["path_node"].tolist() == [[0, 2], [0, -1]]
    assert o["out_tok"][0, 0] == 2
    # second rejection: [r - q2]_+ = (0, 1/2, 0) -> token 1
    assert o["out_tok"][1].tolist() == [1, -1]
    np.testing.assert_allclose(o["min_margin"], [0.05, 0.05], atol=3e-3)


def _vocab8_tables(seed):
    g = I.rng(seed)
    p = g.dirichlet(np.full(8, 0.5), size=5)                 # one target table per node
    p = np.maximum(p, 1e-4)
    p /= p.sum(-1, keepdims=True)
    head = g.standard_normal((2, 8))                           # two heads' logits over the vocab
    k = 4
    order = np.argsort(-head, axis=-1)[:, :k]
    return np.log(p), order.astype(np.int32), np.take_along_axis(head, order, -1).astype(np.float32)


def test_million_trials_marginal_joint_first_slot_and_sandwich():
    # root with two children; its first child has two children (depth 2)
    parent = np.array([-1, 0, 0, 1, 1], np.int32)
    node_logits, cand_id, cand_logit = _vocab8_tables(2024)
    out = _run(parent, node_logits, cand_id, cand_logit, N_TRIALS, seed=99)
    P = softmax(_f64(_bits(node_logits)), axis=-1)
    # (1) one-node correction: the first emitted token follows p_root
    first = out["out_tok"][:, 0]
    freq = np.bincount(first, minlength=8) / N_TRIALS
    assert _within(freq, P[0], N_TRIALS).all(), (freq, P[0])
    # (2) first-slot acceptance = sum_v min(p, q_{u,1}) = 1 - TV(p, q_{u,1})
    q1 = np.zeros(8)
    q1[cand_id[0]] = softmax(cand_logit[0].astype(np.float64))
    a1 = np.mean((out["n_acc"] >= 1) & (out["path_node"][:, 1] == 1))
    assert _within(a1, 1 - 0.5 * np.abs(P[0] - q1).sum(), N_TRIALS)
    # (3) sandwich  p(C) * Omega_C <= Pr(some candidate accepted) <= p(C)
    C = cand_id[0]
    pC = P[0][C].sum()
    omega = np.minimum(P[0][C] / pC, q1[C]).sum()
    a_any = np.mean(out["n_acc"] >= 1)
    tol = 4.5 * np.sqrt(0.25 / N_TRIALS)
    assert pC * omega - tol <= a_any <= pC + tol
    # (4) exact continuation: given the committed first token came from node c, the next
    #     emitted token follows p_c (whether it was accepted below c or resampled there)
    for c in (1, 2):
        sel = (out["n_acc"] >= 1) & (out["path_node"][:, 1] == c)
        n = int(sel.sum())
        assert n > 2000
        f2 = np.bincount(out["out_tok"][sel, 1], minlength=8) / n
        assert _within(f2, P[c], n).all(), (c, f2, P[c])
    # (5) joint of the first two committed tokens on the accepted branch a -> b
    sel = out["n_acc"] >= 1
    a_tok, b_tok = out["out_tok"][sel, 0], out["out_tok"][sel, 1]
    node = out["path_node"][sel, 1]
    for a in np.unique(a_tok)[:3]:
        for c in (1, 2):
            s2 = (a_tok == a) & (node == c)
            if s2.sum() < 5000:
                continue
            f = np.bincount(b_tok[s2], minlength=8) / s2.sum()
            assert _within(f, P[c], int(s2.sum())).all()
    # accepted length bookkeeping
    assert (out["n_acc"] <= 2).all()
    assert ((out["term_kind"] == 1) == np.isin(out["term_node"], [2, 3, 4])).all()


def test_temperature_other_than_one_marginal_first_slot_and_continuation():
    # Same tree and tables at T = 0.7 and T = 1.3.  The target of every node is softmax(l / T), and the
    # proposal of the draw is the head softmax at the same T (App. B.1 Eq. "nodep" / "slotq"), so
    # the emitted tokens must follow softmax(l / T) and the first-slot acceptance must be
    # 1 - TV(softmax(l / T), q_{u,1}) (App. B.2 Eq. "nodeaccept").  A temperature applied to only one
    # of the two, or applied as a product instead of a quotient, fails every assertion below.
    parent = np.array([-1, 0, 0, 1, 1], np.int32)
    node_logits, cand_id, cand_logit = _vocab8_tables(77)
    node_logits = node_logits * 0.5 + 0.3                      # not normalised: log-probabilities would hide a slip at T = 1 only
    n = 400_000
    for T, seed in ((0.7, 5), (1.3, 6)):
        out = _run(parent, node_logits, cand_id, cand_logit, n, seed=seed, T=T)
        T32 = np.float64(np.float32(T))
        P = softmax(_f64(_bits(node_logits)) / T32, axis=-1)
        P1 = softmax(_f64(_bits(node_logits)), axis=-1)
        assert np.abs(P[0] - P1[0]).max() > 0.02               # the two temperatures are told apart by the test
        freq = np.bincount(out["out_tok"][:, 0], minlength=8) / n
        assert _within(freq, P[0], n).all(), (T, freq, P[0])
        assert not _within(freq, P1[0], n).all()
        q1 = np.zeros(8)
        q1[cand_id[0]] = softmax(cand_logit[0].astype(np.float64) / T32)
        a1 = np.mean((out["n_acc"] >= 1) & (out["path_node"][:, 1] == 1))
        assert _within(a1, 1 - 0.5 * np.abs(P[0] - q1).sum(), n), (T, a1)
        # slot_q recorded by the draw is the head softmax at T over what the earlier sibling left
        first = out["tree_cand"][:, 1].astype(int)
        np.testing.assert_allclose(out["slot_q"][:, 1], q1[cand_id[0]][first], rtol=1e-5)
        for c in (1, 2):
            sel = (out["n_acc"] >= 1) & (out["path_node"][:, 1] == c)
            m = int(sel.sum())
            assert m > 2000
            f2 = np.bincount(out["out_tok"][sel, 1], minlength=8) / m
            assert _within(f2, P[c], m).all(), (T, c, f2, P[c])


def test_single_candidate_closed_form():
    # k = 1: q is a point mass on y, so y is accepted w.p. p(y) and the fallback is p off y.
    g = I.rng(5)
    p = g.dirichlet(np.ones(8))
    parent = np.array([-1, 0], np.int32)
    n = 400000
    out = _run(parent, np.log(np.stack([p, p])), np.array([[3]]), np.array([[0.7]]), n, seed=17)
    P = softmax(_f64(_bits(np.log(p))))
    assert (out["tree_tok"][:, 1] == 3).all()
    assert _within(np.mean(out["n_acc"] == 1), P[3], n)
    rej = out["n_acc"] == 0
    f = np.bincount(out["out_tok"][rej, 0], minlength=8) / rej.sum()
    want = P.copy()
    want[3] = 0
    want /= want.sum()
    assert f[3] == 0 and _within(f, want, int(rej.sum())).all()


def test_row_statistics_against_scipy_and_temperature():
    w = I.scaled(I.WORKLOADS["tiny"], B=3, V=500)
    x = I.propose_inputs(w)
    tok = I.rng(1).integers(0, w.V, (w.B, w.N)).astype(np.int32)
    lg = I.target_logits(w, x["parent"], tok)
    T = 0.8
    cid = np.tile(np.arange(w.k, dtype=np.int32), (w.B, w.K, 1))
    cl = np.zeros((w.B, w.K, w.k), np.float32)
    d = ref.tree_draw(x["parent"], x["anchor"], cid, cl, x["u_draw"], temperature=T)
    u_acc, u_fin = I.verify_uniforms(w)
    o = ref.verify(lg, x["parent"], d["tree_tok"], d["tree_cand"], cid, cl, u_acc, u_fin, temperature=T)
    L = _f64(lg)
    np.testing.assert_array_equal(o["row_max"], L.max(-1))
    T32 = np.float64(np.float32(T))                          # the interface carries T as fp32
    np.testing.assert_allclose(np.log(o["row_sum"]) + o["row_max"] / T32, logsumexp(L / T32, axis=-1),
                               rtol=1e-12)


def test_terminal_draw_against_cumsum_searchsorted():
    # lone root (N = 1): the emitted token is a plain inverse-CDF sample of softmax(logits / T)
    B, V = 2000, 64
    g = I.rng(3)
    lg = _bits(g.standard_normal((B, 1, V)) * 2)
    u_fin = I.uniforms24(8, (B,))
    parent = np.array([-1], np.int32)
    o = ref.verify(lg, parent, np.zeros((B, 1), np.int32), np.full((B, 1), 255, np.uint8),
                   np.zeros((B, 1, 1), np.int32), np.zeros((B, 1, 1), np.float32),
                   np.zeros((B, 1), np.float32), u_fin)
    P = softmax(_f64(lg)[:, 0], axis=-1)
    cum = np.cumsum(P, -1)
    want = np.array([np.searchsorted(cum[b], np.float64(u_fin[b]) * cum[b, -1], side="right") for b in range(B)])
    safe = o["fin_margin"] > 1e-9
    assert safe.mean() > 0.99
    assert np.array_equal(o["out_tok"][safe, 0], np.minimum(want, V - 1)[safe])
    assert (o["n_acc"] == 0).all() and (o["term_kind"] == 0).all()


def test_deeper_walk_on_the_tiny_topology_is_self_consistent():
    w = I.WORKLOADS["tiny"]
    x = I.propose_inputs(w, peaked=True)
    pr = ref.propose(x["h"], x["anchor"], x["A"], x["bias"], x["W"], x["m"], x["alpha"], x["parent"],
                     x["u_draw"], k=w.k, clip_c=w.clip_c)
    lg = I.target_logits(w, x["parent"], pr["tree_tok"])
    u_acc, u_fin = I.verify_uniforms(w)
    o = ref.verify(lg, x["parent"], pr["tree_tok"], pr["tree_cand"], pr["cand_id"], pr["cand_logit"],
                   u_acc, u_fin)
    for b in range(w.B):
        n = o["n_acc"][b]
        path = o["path_node"][b]
        assert path[0] == 0 and (path[n + 1:] == -1).all()
        for i in range(1, n + 1):
            assert x["parent"][path[i]] == path[i - 1]
            assert o["out_tok"][b, i - 1] == pr["tree_tok"][b, path[i]]
        assert o["term_node"][b] == path[n]
        assert 0 <= o["out_tok"][b, n] < w.V
