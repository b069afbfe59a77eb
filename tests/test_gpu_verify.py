"""GPU parity: specroll_verify against the CPU oracle on identical seeded inputs."""
import numpy as np
import pytest
import torch

from oracle import ref
from paper_2608_04962_b200 import binding as S
from paper_2608_04962_b200 import inputs as I
from tests.util import dev, dev_bf16, host

pytestmark = pytest.mark.gpu

NEAR_TIE = 1e-4        # |u - ratio| below this may flip the decision (counted)
P_RTOL = 1e-3          # relative tolerance on normalised probabilities


def run_both(w, parent, logits, tree_tok, tree_cand, cand_id, cand_logit, u_acc, u_fin):
    o = ref.verify(logits, parent, tree_tok, tree_cand, cand_id, cand_logit, u_acc, u_fin,
                   temperature=w.temperature)
    g = S.verify(dev_bf16(logits), parent, dev(tree_tok), dev(tree_cand), dev(cand_id), dev(cand_logit),
                 dev(u_acc), dev(u_fin), temperature=w.temperature)
    torch.cuda.synchronize()
    return o, {k: host(v) for k, v in g.items()}


def check(w, o, g, logits):
    B = w.B
    # softmax statistics: max is exact (a bf16 value), the normaliser to 1e-3 relative
    assert np.array_equal(g["row_max"].astype(np.float64), o["row_max"])
    np.testing.assert_allclose(g["row_sum"], o["row_sum"], rtol=P_RTOL)
    assert np.abs(g["row_sum"] / o["row_sum"] - 1).max() < 2e-5   # what bit-exact acceptance needs
    same = (g["n_acc"] == o["n_acc"]) & (g["path_node"] == o["path_node"]).all(1) & \
           (g["out_tok"] == o["out_tok"]).all(1) & (g["term_node"] == o["term_node"]) & \
           (g["term_kind"] == o["term_kind"])
    bad = np.flatnonzero(~same)
    near = 0
    for b in bad:
        walk_same = g["n_acc"][b] == o["n_acc"][b] and (g["path_node"][b] == o["path_node"][b]).all()
        if not walk_same:
            assert o["min_margin"][b] < NEAR_TIE, (b, o["min_margin"][b], g["n_acc"][b], o["n_acc"][b])
        else:
            # only the terminal inverse-CDF draw differs: neighbouring token at a bracket edge
            n = o["n_acc"][b]
            assert (g["out_tok"][b, :n] == o["out_tok"][b, :n]).all()
            assert o["fin_margin"][b] < 1e-6, (b, o["fin_margin"][b])
        near += 1
    assert near <= max(1, int(1e-3 * B)) and near / max(B, 1) < (1e-3 if B >= 1000 else 1.0), (near, B)
    ok = np.isfinite(o["min_margin"])
    mm_ok = np.abs(g["min_margin"][ok] - o["min_margin"][ok]) <= 1e-3 * np.maximum(1.0, o["min_margin"][ok])
    assert mm_ok[same[ok]].all()
    return len(bad)


def test_tiny_config_with_oracle_proposals():
    w = I.WORKLOADS["tiny"]
    x = I.propose_inputs(w, peaked=True)
    pr = ref.propose(x["h"], x["anchor"], x["A"], x["bias"], x["W"], x["m"], x["alpha"], x["parent"],
                     x["u_draw"], k=w.k, clip_c=w.clip_c)
    u_acc, u_fin = I.verify_uniforms(w)
    for flat in (False, True):
        lg = I.target_logits(w, x["parent"], pr["tree_tok"], flat=flat)
        o, g = run_both(w, x["parent"], lg, pr["tree_tok"], pr["tree_cand"], pr["cand_id"], pr["cand_logit"],
                        u_acc, u_fin)
        check(w, o, g, lg)


@pytest.mark.parametrize("name,B,V,T", [("qwen1.5b", 48, 151936, 1.0), ("qwen7b", 24, 152064, 0.7),
                                        ("qwen14b", 12, 152064, 1.0), ("qwen1.5b", 300, 4104, 1.3)])
def test_reduced_batches_of_the_large_configs(name, B, V, T):
    w = I.scaled(I.WORKLOADS[name], B=B, V=V, temperature=T)
    parent = I.topology(w)
    cid, cl = I.synthetic_candidates(w)
    u_draw = I.uniforms24(77, (w.B, w.N))
    d = ref.tree_draw(parent, np.zeros(w.B, np.int32), cid, cl, u_draw, temperature=T)
    lg = I.target_logits(w, parent, d["tree_tok"])
    u_acc, u_fin = I.verify_uniforms(w)
    o, g = run_both(w, parent, lg, d["tree_tok"], d["tree_cand"], cid, cl, u_acc, u_fin)
    check(w, o, g, lg)
    assert o["n_acc"].max() >= 1          # the workload does accept something
    # accepted-length statistics of the two sides agree
    assert abs(g["n_acc"].mean() - o["n_acc"].mean()) < 0.05


def test_many_sequences_small_vocab_mismatch_budget():
    # 20000 sequences: the 0.1 % budget on near-tie decisions is measurable here
    w = I.scaled(I.WORKLOADS["tiny"], B=20000, V=64, K=3, k=4, N=8)
    parent = I.topology(w)
    cid, cl = I.synthetic_candidates(w)
    d = ref.tree_draw(parent, np.zeros(w.B, np.int32), cid, cl, I.uniforms24(5, (w.B, w.N)))
    lg = I.target_logits(w, parent, d["tree_tok"], boost=3.0)
    u_acc, u_fin = I.verify_uniforms(w)
    o, g = run_both(w, parent, lg, d["tree_tok"], d["tree_cand"], cid, cl, u_acc, u_fin)
    n_bad = check(w, o, g, lg)
    assert n_bad / w.B < 1e-3
    near = np.mean(o["min_margin"] < NEAR_TIE)
    assert near < 1e-3 * 8                 # near ties are rare in the workload itself


def test_lone_root_and_chain_and_star_topologies():
    for parent in ([-1], [-1, 0, 1, 2], [-1, 0, 0, 0, 0]):
        N = len(parent)
        w = I.scaled(I.WORKLOADS["tiny"], B=16, N=N, V=512, K=3, k=4, fixed_parent=tuple(parent))
        parent = np.array(parent, np.int32)
        cid, cl = I.synthetic_candidates(w)
        d = ref.tree_draw(parent, np.zeros(w.B, np.int32), cid, cl, I.uniforms24(9, (w.B, N)))
        lg = I.target_logits(w, parent, d["tree_tok"], boost=6.0)
        u_acc, u_fin = I.verify_uniforms(w)
        o, g = run_both(w, parent, lg, d["tree_tok"], d["tree_cand"], cid, cl, u_acc, u_fin)
        check(w, o, g, lg)


@pytest.mark.parametrize("V", [8, 1032, 8200, 40008])
def test_terminal_draw_alone_over_ragged_vocabularies(V):
    """A lone root: the step is the terminal draw from the root's softmax.  Nearly flat logits spread the drawn tokens
    over the whole vocabulary, so every eighth of the row (the unit the draw narrows down to first) is hit, with
    vocabulary sizes that leave the eighths empty, partial or ragged; u_fin is stratified and includes 0."""
    B = 640
    w = I.scaled(I.WORKLOADS["tiny"], B=B, N=1, V=V, K=3, k=4, fixed_parent=(-1,))
    parent = np.array([-1], np.int32)
    cid, cl = I.synthetic_candidates(w)
    d = ref.tree_draw(parent, np.zeros(B, np.int32), cid, cl, I.uniforms24(3, (B, 1)))
    lg = I.target_logits(w, parent, d["tree_tok"], flat=True)
    u_acc, _ = I.verify_uniforms(w)
    u_fin = ((np.arange(B) + 0.5) / B).astype(np.float32)
    u_fin[0] = 0.0
    u_fin[-1] = np.float32(1.0 - 1e-4)
    o, g = run_both(w, parent, lg, d["tree_tok"], d["tree_cand"], cid, cl, u_acc, u_fin)
    check(w, o, g, lg)
    assert (g["n_acc"] == 0).all() and (g["term_kind"] == 0).all()
    tok = g["out_tok"][:, 0]
    assert tok.min() >= 0 and tok.max() < V
    if V >= 8200:
        assert len(set((tok.astype(np.int64) * 8 // V).tolist())) == 8


def test_wide_lists_wide_stars_and_underflowing_proposals():
    # the node routine's fast form holds a candidate and a child per lane: more than 32 of either, and slot
    # proposals whose weights underflow against a drawn candidate's logit, take the sequential form
    cases = []
    w = I.scaled(I.WORKLOADS["tiny"], B=24, N=16, V=2048, K=3, k=40)                       # k > 32
    cases.append((w, I.topology(w), None))
    star = [-1] + [0] * 39                                                                   # 39 children > 32
    w = I.scaled(I.WORKLOADS["tiny"], B=24, N=40, V=2048, K=2, k=48, fixed_parent=tuple(star))
    cases.append((w, np.array(star, np.int32), None))
    w = I.scaled(I.WORKLOADS["tiny"], B=24, N=12, V=1024, K=3, k=8)                        # gaps of 2000 between candidates
    cases.append((w, I.topology(w), 2000.0))
    for w, parent, gap in cases:
        cid, cl = I.synthetic_candidates(w)
        if gap is not None:
            cl = (-gap * np.arange(w.k, dtype=np.float32))[None, None, :].repeat(w.B, 0).repeat(w.K, 1).copy()
        d = ref.tree_draw(parent, np.zeros(w.B, np.int32), cid, cl, I.uniforms24(13, (w.B, w.N)))
        lg = I.target_logits(w, parent, d["tree_tok"], boost=5.0)
        u_acc, u_fin = I.verify_uniforms(w)
        o, g = run_both(w, parent, lg, d["tree_tok"], d["tree_cand"], cid, cl, u_acc, u_fin)
        check(w, o, g, lg)
        if gap is not None:
            # a later sibling's proposal is a point mass on the best remaining candidate
            assert (d["tree_cand"][:, 1:] < w.k).all()


def test_bad_arguments_are_refused_without_touching_the_device():
    w = I.scaled(I.WORKLOADS["tiny"], B=2)
    parent = I.topology(w)
    cid, cl = I.synthetic_candidates(w)
    lg = dev_bf16(np.zeros((w.B, w.N, w.V), np.uint16))
    args = (dev(np.zeros((w.B, w.N), np.int32)), dev(np.zeros((w.B, w.N), np.uint8)), dev(cid), dev(cl),
            dev(np.zeros((w.B, w.N), np.float32)), dev(np.zeros(w.B, np.float32)))
    bad_parent = parent.copy()
    bad_parent[3] = 5                      # not topological
    with pytest.raises(S.SpecrollError):
        S.verify(lg, bad_parent, *args)
    with pytest.raises(S.SpecrollError):
        S.verify(lg, parent, *args, temperature=0.0)
    with pytest.raises(S.SpecrollError):
        S.verify(lg, parent, *args, workspace=torch.empty(256, dtype=torch.uint8, device="cuda")[:16])


@pytest.mark.parametrize("name,B,V,T", [("qwen1.5b", 32, 151936, 1.0), ("qwen7b", 16, 8200, 0.7)])
def test_lazy_row_statistics_give_the_same_walk(name, B, V, T):
    # statistics of the visited rows only: same tokens as the full pass; row_max / row_sum written where visited
    w = I.scaled(I.WORKLOADS[name], B=B, V=V, temperature=T)
    parent = I.topology(w)
    cid, cl = I.synthetic_candidates(w)
    d = ref.tree_draw(parent, np.zeros(w.B, np.int32), cid, cl, I.uniforms24(78, (w.B, w.N)), temperature=T)
    lg = I.target_logits(w, parent, d["tree_tok"])
    u_acc, u_fin = I.verify_uniforms(w)
    o = ref.verify(lg, parent, d["tree_tok"], d["tree_cand"], cid, cl, u_acc, u_fin, temperature=T)
    args = (dev_bf16(lg), parent, dev(d["tree_tok"]), dev(d["tree_cand"]), dev(cid), dev(cl), dev(u_acc), dev(u_fin))
    out = {"n_acc": torch.empty(B, dtype=torch.int32, device="cuda"),
           "path_node": torch.empty((B, w.K + 1), dtype=torch.int32, device="cuda"),
           "out_tok": torch.empty((B, w.K + 1), dtype=torch.int32, device="cuda"),
           "term_node": torch.empty(B, dtype=torch.int32, device="cuda"),
           "term_kind": torch.empty(B, dtype=torch.int32, device="cuda"),
           "row_max": torch.full((B, w.N), -7.0, device="cuda"), "row_sum": torch.full((B, w.N), -7.0, device="cuda"),
           "min_margin": torch.empty(B, device="cuda")}
    g = {k: host(v) for k, v in S.verify(*args, temperature=T, out=out, flags=S.VERIFY_LAZY_STATS).items()}
    full = {k: host(v) for k, v in S.verify(*args, temperature=T).items()}
    for key in ("n_acc", "path_node", "out_tok", "term_node", "term_kind"):
        assert np.array_equal(g[key], full[key]), key               # the two GPU variants agree exactly
    visited = np.zeros((B, w.N), bool)
    for b in range(B):
        visited[b, g["path_node"][b, : g["n_acc"][b] + 1]] = True
        visited[b, g["term_node"][b]] = True
    assert np.array_equal(g["row_max"][visited].astype(np.float64), o["row_max"][visited])
    assert np.abs(g["row_sum"][visited] / o["row_sum"][visited] - 1).max() < 2e-5
    assert (g["row_max"][~visited] == -7.0).all() and (g["row_sum"][~visited] == -7.0).all()
    assert visited.sum() < 0.5 * visited.size                        # it does read fewer rows
    same = (g["n_acc"] == o["n_acc"]) & (g["out_tok"] == o["out_tok"]).all(1)
    assert (same | (o["min_margin"] < NEAR_TIE) | (o["fin_margin"] < 1e-6)).all()

