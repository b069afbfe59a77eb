"""GPU parity: specroll_verify_nucleus against the CPU oracle on identical seeded inputs.

The kept set is decided by comparing a cumulative mass with top_p * S; the GPU adds the masses in fp32 and the
oracle in fp64, so a sequence may differ when the oracle's own margin at that decision is tiny (reported as
nucleus_margin); everything else must match like the plain verification."""
import numpy as np
import pytest
import torch

from oracle import ref
from paper_2608_04962_b200 import binding as S
from paper_2608_04962_b200 import inputs as I
from tests.util import dev, dev_bf16, host

pytestmark = pytest.mark.gpu

NEAR_TIE = 1e-4
NUC_EDGE = 1e-5        # |cumulative mass - top_p| below this may move the cut (counted)


def run_both(w, parent, logits, d, cid, cl, u_acc, u_fin, top_p):
    o = ref.verify(logits, parent, d["tree_tok"], d["tree_cand"], cid, cl, u_acc, u_fin, temperature=w.temperature,
                   top_p=top_p)
    g = S.verify_nucleus(dev_bf16(logits), parent, dev(d["tree_tok"]), dev(d["tree_cand"]), dev(cid), dev(cl),
                         dev(u_acc), dev(u_fin), top_p, temperature=w.temperature)
    torch.cuda.synchronize()
    return o, {k: host(v) for k, v in g.items()}


def check(w, o, g):
    B = w.B
    assert np.array_equal(g["row_max"].astype(np.float64), o["row_max"])
    assert np.abs(g["row_sum"] / o["row_sum"] - 1).max() < 2e-5
    # thresholds and kept sums on the nodes the oracle visited
    vis = np.isfinite(o["nucleus_thr"])
    edge = o["nucleus_margin"] < NUC_EDGE
    thr_ok = np.abs(g["nucleus_thr"][vis] - o["nucleus_thr"][vis]) <= 1e-5 * np.maximum(1.0, np.abs(o["nucleus_thr"][vis]))
    rows_b = np.nonzero(vis)[0]
    assert (thr_ok | edge[rows_b]).all()
    sum_ok = np.abs(g["nucleus_sum"][vis] / o["nucleus_sum"][vis] - 1) < 2e-5
    assert (sum_ok | edge[rows_b]).all()
    same = (g["n_acc"] == o["n_acc"]) & (g["path_node"] == o["path_node"]).all(1) & \
           (g["out_tok"] == o["out_tok"]).all(1) & (g["term_node"] == o["term_node"]) & \
           (g["term_kind"] == o["term_kind"])
    bad = np.flatnonzero(~same)
    for b in bad:
        assert o["min_margin"][b] < NEAR_TIE or o["fin_margin"][b] < 1e-6 or edge[b], \
            (b, o["min_margin"][b], o["fin_margin"][b], o["nucleus_margin"][b])
    assert len(bad) <= max(1, int(1e-3 * B))
    return len(bad)


@pytest.mark.parametrize("top_p", [0.95, 0.5])
def test_tiny_config(top_p):
    w = I.WORKLOADS["tiny"]
    x = I.propose_inputs(w, peaked=True)
    pr = ref.propose(x["h"], x["anchor"], x["A"], x["bias"], x["W"], x["m"], x["alpha"], x["parent"],
                     x["u_draw"], k=w.k, clip_c=w.clip_c)
    u_acc, u_fin = I.verify_uniforms(w)
    for flat in (False, True):
        lg = I.target_logits(w, x["parent"], pr["tree_tok"], flat=flat)
        o, g = run_both(w, x["parent"], lg, pr, pr["cand_id"], pr["cand_logit"], u_acc, u_fin, top_p)
        check(w, o, g)


@pytest.mark.parametrize("name,B,V,T,top_p", [("qwen1.5b", 24, 151936, 1.0, 0.95), ("qwen7b", 12, 152064, 0.7, 0.9),
                                              ("qwen1.5b", 300, 4104, 1.3, 0.95)])
def test_reduced_batches_of_the_large_configs(name, B, V, T, top_p):
    w = I.scaled(I.WORKLOADS[name], B=B, V=V, temperature=T)
    parent = I.topology(w)
    cid, cl = I.synthetic_candidates(w)
    d = ref.tree_draw(parent, np.zeros(w.B, np.int32), cid, cl, I.uniforms24(77, (w.B, w.N)), temperature=T)
    lg = I.target_logits(w, parent, d["tree_tok"])
    u_acc, u_fin = I.verify_uniforms(w)
    o, g = run_both(w, parent, lg, d, cid, cl, u_acc, u_fin, top_p)
    check(w, o, g)
    # the cut does remove tokens, and every emitted terminal token is inside its node's nucleus
    vals = I.bf16_bits_to_f32(lg)
    for b in range(w.B):
        node, tok = g["term_node"][b], g["out_tok"][b, g["n_acc"][b]]
        assert vals[b, node, tok] >= g["nucleus_thr"][b, node]
    assert (g["nucleus_sum"] < g["row_sum"] * 0.9999).any()


def test_many_sequences_small_vocab():
    w = I.scaled(I.WORKLOADS["tiny"], B=20000, V=64, K=3, k=4, N=8)
    parent = I.topology(w)
    cid, cl = I.synthetic_candidates(w)
    d = ref.tree_draw(parent, np.zeros(w.B, np.int32), cid, cl, I.uniforms24(5, (w.B, w.N)))
    lg = I.target_logits(w, parent, d["tree_tok"], boost=3.0)
    u_acc, u_fin = I.verify_uniforms(w)
    o, g = run_both(w, parent, lg, d, cid, cl, u_acc, u_fin, 0.9)
    assert check(w, o, g) / w.B < 1e-3


def test_threshold_of_one_is_the_plain_verification():
    w = I.scaled(I.WORKLOADS["tiny"], B=64, V=2048)
    parent = I.topology(w)
    cid, cl = I.synthetic_candidates(w)
    d = ref.tree_draw(parent, np.zeros(w.B, np.int32), cid, cl, I.uniforms24(6, (w.B, w.N)))
    lg = I.target_logits(w, parent, d["tree_tok"], boost=5.0)
    u_acc, u_fin = I.verify_uniforms(w)
    args = (dev_bf16(lg), parent, dev(d["tree_tok"]), dev(d["tree_cand"]), dev(cid), dev(cl), dev(u_acc), dev(u_fin))
    a = S.verify(*args)
    b = S.verify_nucleus(*args, 1.0)
    for key in ("n_acc", "path_node", "out_tok", "term_node", "term_kind"):
        assert torch.equal(a[key], b[key])
    with pytest.raises(S.SpecrollError):
        S.verify_nucleus(*args, 0.0)
