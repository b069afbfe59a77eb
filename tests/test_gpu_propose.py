"""GPU parity: specroll_propose / specroll_tree_draw against the CPU oracle."""
import numpy as np
import pytest
import torch

from oracle import ref
from paper_2608_04962_b200 import binding as S
from paper_2608_04962_b200 import inputs as I
from tests.util import dev, dev_bf16, host

pytestmark = pytest.mark.gpu

TIE = 1e-3             # top-k sets may differ only among logits within this distance of the k-th
# Reported candidate logits: a probability is proportional to exp(logit), so 1e-3 relative on the
# probability is 1e-3 absolute on the logit.  fp32 accumulation alone gives ~1e-7; the rest of the
# allowance covers a corrected state element that rounds to the neighbouring bf16 value because the
# GPU holds it in fp32 and the oracle in fp64 (one such flip moves a logit by ulp * |W| ~ 2e-4).
LOGIT_ATOL = 1e-3


def gpu_propose(w, x, **kw):
    g = S.propose(dev_bf16(x["h"]), dev(x["anchor"]), dev_bf16(x["A"]), dev_bf16(x["bias"]), dev_bf16(x["W"]),
                  dev(x["m"]) if x.get("m") is not None else None,
                  dev(x["alpha"]) if x.get("alpha") is not None else None,
                  x["parent"], dev(x["u_draw"]), k=w.k, temperature=w.temperature, clip_c=w.clip_c,
                  check_status=True, **kw)
    torch.cuda.synchronize()
    return {k: host(v) for k, v in g.items()}


def check_candidates(w, x, g, logit_atol, **okw):
    """Top-k sets against the oracle's full logits, tie-aware; returns rows whose lists are identical."""
    hd = ref.heads(x["h"], x["A"], x["bias"], m=x.get("m"), alpha=x.get("alpha"), clip_c=w.clip_c, **okw)
    full = ref.lm_logits(hd["zt"], x["W"])                      # [B*K, V] fp64
    oid, ol = ref.topk(full, w.k)
    gid = g["cand_id"].reshape(-1, w.k)
    gl = g["cand_logit"].reshape(-1, w.k).astype(np.float64)
    kth = ol[:, -1].astype(np.float64)
    rows = np.arange(full.shape[0])[:, None]
    assert (gid >= 0).all() and (gid < w.V).all()
    assert (np.sort(gid, 1)[:, 1:] != np.sort(gid, 1)[:, :-1]).all()          # distinct
    picked = full[rows, gid]
    assert (picked >= kth[:, None] - TIE).all()                               # nothing clearly outside
    must = full > (kth[:, None] + TIE)                                        # clearly inside
    got = np.zeros_like(must)
    got[rows, gid] = True
    assert (got | ~must).all()
    np.testing.assert_allclose(gl, picked, atol=logit_atol, rtol=0)           # reported logits
    assert (np.diff(gl, axis=1) <= 0).all()                                   # sorted descending
    same = (gid == oid).all(1)
    return same.reshape(w.B, w.K), oid.reshape(w.B, w.K, w.k), ol.reshape(w.B, w.K, w.k)


def check_tree(w, x, g, same, T=1.0, oid=None, ol=None):
    """The drawn tree.  (a) Where a sequence's candidate lists equal the oracle's id for id, the oracle's draw
    from ITS OWN lists must give the GPU's tokens (the lists' logits differ in their last bits, fp64 against
    fp32, so a draw decided within rounding of its uniform may differ: at most 2 % of the sequences).
    (b) The oracle's draw from the GPU's lists isolates the draw step: exact tokens expected."""
    if oid is not None:
        rows = np.flatnonzero(same.all(axis=1))
        if rows.size:
            d0 = ref.tree_draw(x["parent"], x["anchor"][rows], oid[rows], ol[rows].astype(np.float32),
                               x["u_draw"][rows], temperature=T)
            eq = (g["tree_tok"][rows] == d0["tree_tok"]).all(axis=1)
            assert eq.mean() >= 0.98, (eq.mean(), rows.size)
    d = ref.tree_draw(x["parent"], x["anchor"], g["cand_id"], g["cand_logit"], x["u_draw"], temperature=T)
    assert np.array_equal(g["tree_tok"], d["tree_tok"])
    assert np.array_equal(g["tree_cand"], d["tree_cand"])
    np.testing.assert_allclose(g["slot_q"], d["slot_q"], rtol=1e-5)
    assert (g["tree_tok"][:, 0] == x["anchor"]).all()


@pytest.mark.parametrize("peaked", [False, True])
def test_tiny_config(peaked):
    w = I.WORKLOADS["tiny"]
    x = I.propose_inputs(w, peaked=peaked)
    g = gpu_propose(w, x)
    same, oid, ol = check_candidates(w, x, g, logit_atol=LOGIT_ATOL)
    check_tree(w, x, g, same, oid=oid, ol=ol)
    if peaked:
        assert same.mean() > 0.9


@pytest.mark.parametrize("B,K,k,d,V,N", [(37, 4, 8, 512, 3000, 16), (130, 2, 8, 256, 1288, 9),
                                         (9, 5, 16, 320, 2056, 24), (64, 4, 8, 1536, 8192, 16),
                                         (300, 2, 8, 192, 1288, 9), (100, 3, 8, 448, 2048, 12)])
def test_ragged_shapes(B, K, k, d, V, N):
    # rows, hidden size and vocabulary not multiples of the 128-wide tiles; k above the fast-path size;
    # batches on either side of the head kernel's 64 / 128 / 256-sequence blocks, and one above 256
    w = I.scaled(I.WORKLOADS["qwen1.5b"], B=B, K=K, k=k, d=d, V=V, N=N, alpha_heads=(0.025, 0.01, 0.006, 0.004, 0.003)[:K])
    x = I.propose_inputs(w, peaked=True)
    g = gpu_propose(w, x)
    same, oid, ol = check_candidates(w, x, g, logit_atol=LOGIT_ATOL)
    check_tree(w, x, g, same, oid=oid, ol=ol)
    assert same.mean() > 0.9


def test_legacy_projection_kernel_agrees():
    # the mma.sync projection (flag) and the tcgen05 one must both match the oracle
    w = I.scaled(I.WORKLOADS["qwen1.5b"], B=40, K=4, k=8, d=512, V=5000, N=16)
    x = I.propose_inputs(w, peaked=True)
    for flags in (0, 1):
        g = gpu_propose(w, x, flags=flags)
        same, _, _ = check_candidates(w, x, g, logit_atol=LOGIT_ATOL)
        assert same.mean() > 0.9


def test_reflex_abstain_clip_and_affine_layernorm():
    w = I.scaled(I.WORKLOADS["tiny"], B=16, V=2048)
    x = I.propose_inputs(w, peaked=True)
    # (a) no memory at all
    x0 = dict(x, m=None, alpha=None)
    g0 = gpu_propose(w, x0)
    check_candidates(w, x0, g0, logit_atol=LOGIT_ATOL)
    # (b) strong correction so that the clip binds everywhere and changes the candidates
    x1 = dict(x, alpha=np.full((w.B, w.K), 0.5, np.float32))
    g1 = gpu_propose(w, x1)
    check_candidates(w, x1, g1, logit_atol=LOGIT_ATOL)
    assert (g1["cand_id"] != g0["cand_id"]).any()
    # (c) per-head LayerNorm affine
    gg = I.rng(31)
    gam = I.f32_to_bf16_bits(gg.uniform(0.5, 1.5, (w.K, w.d)).astype(np.float32))
    bet = I.f32_to_bf16_bits((0.1 * gg.standard_normal((w.K, w.d))).astype(np.float32))
    g2 = gpu_propose(w, x, ln_gamma=dev_bf16(gam), ln_beta=dev_bf16(bet))
    check_candidates(w, x, g2, logit_atol=LOGIT_ATOL, gamma=gam, beta=bet)


def test_correction_before_the_heads():
    # secondary form of the bounded correction: one memory row and ratio per sequence, applied to h; the heads
    # then run on the corrected state (the oracle's own pins fix that composition on the CPU)
    w = I.scaled(I.WORKLOADS["qwen1.5b"], B=70, K=4, k=8, d=640, V=4104, N=16)
    x = I.propose_inputs(w, peaked=True)
    gg = I.rng(77)
    m = gg.standard_normal((w.B, w.d)).astype(np.float32)
    alpha = gg.uniform(0.02, 0.3, w.B).astype(np.float32)
    alpha[::5] = 0.0                                          # some sequences abstain
    for clip_c in (0.0, 0.05):                                # unclipped; clip binding for the larger ratios
        wc = I.scaled(w, clip_c=clip_c)
        ht = ref.prehead(x["h"], m, alpha, clip_c=clip_c)["ht"]
        assert (ht[::5] == x["h"][::5]).all() and (ht[1] != x["h"][1]).any()
        g = gpu_propose(wc, dict(x, m=m, alpha=alpha), flags=S.REFLEX_PRE_HEAD)
        xo = dict(x, h=ht, m=None, alpha=None)
        same, oid, ol = check_candidates(wc, xo, g, logit_atol=LOGIT_ATOL)
        check_tree(wc, xo, g, same, oid=oid, ol=ol)
        assert same.mean() > 0.9
    # every ratio zero, or no memory at all: bit for bit the uncorrected proposal
    g_plain = gpu_propose(w, dict(x, m=None, alpha=None))
    for mm, aa in ((m, np.zeros(w.B, np.float32)), (None, None)):
        g0 = gpu_propose(w, dict(x, m=mm, alpha=aa), flags=S.REFLEX_PRE_HEAD)
        for key in ("cand_id", "cand_logit", "tree_tok", "tree_cand", "slot_q"):
            assert np.array_equal(g0[key], g_plain[key]), key
    # the per-head shapes of the default form are refused under the flag
    with pytest.raises(S.SpecrollError):
        gpu_propose(w, x, flags=S.REFLEX_PRE_HEAD)


def test_tree_draw_alone_matches_exactly():
    for name in ("qwen1.5b", "qwen7b", "qwen14b"):
        w = I.scaled(I.WORKLOADS[name], B=200)
        parent = I.topology(w)
        cid, cl = I.synthetic_candidates(w)
        u = I.uniforms24(3, (w.B, w.N))
        anchor = np.arange(w.B, dtype=np.int32)
        for T in (1.0, 0.6):
            o = ref.tree_draw(parent, anchor, cid, cl, u, temperature=T)
            g = S.tree_draw(parent, dev(anchor), dev(cid), dev(cl), dev(u), temperature=T)
            assert np.array_equal(host(g["tree_tok"]), o["tree_tok"])
            assert np.array_equal(host(g["tree_cand"]), o["tree_cand"])
            np.testing.assert_allclose(host(g["slot_q"]), o["slot_q"], rtol=1e-6)
    # the paper's nominal (5,4,0) allocation
    parent = I.paper_540_topology()
    w = I.scaled(I.WORKLOADS["tiny"], B=50, N=10, K=3, k=8, V=4096)
    cid, cl = I.synthetic_candidates(w)
    u = I.uniforms24(4, (w.B, 10))
    o = ref.tree_draw(parent, np.zeros(w.B, np.int32), cid, cl, u)
    g = S.tree_draw(parent, dev(np.zeros(w.B, np.int32)), dev(cid), dev(cl), dev(u))
    assert np.array_equal(host(g["tree_tok"]), o["tree_tok"])


def test_tree_draw_with_a_candidate_that_dwarfs_the_rest():
    # One candidate of every head leads the others by more than 745 T, so that once it has been drawn the weights
    # of the rest underflow against it and the draw has to renormalise over what is left (App. B.1 Eq. "slotq":
    # q_{u,j} is a softmax over the remaining candidates only).  Two parents of the same depth draw from the same
    # head: the second parent's first child must still see the leading candidate.
    parent = np.array([-1, 0, 0, 1, 1, 1, 2, 2, 2], np.int32)
    B, K, k = 64, 2, 4
    g = I.rng(77)
    cid = np.tile(np.arange(K * k, dtype=np.int32).reshape(1, K, k), (B, 1, 1))
    cl = np.sort(g.standard_normal((B, K, k)).astype(np.float32), axis=-1)[..., ::-1].copy()
    cl[..., 0] += 900.0
    u = I.uniforms24(9, (B, parent.shape[0]))
    anchor = np.zeros(B, np.int32)
    for T in (1.0, 0.7):
        o = ref.tree_draw(parent, anchor, cid, cl, u, temperature=T)
        d = S.tree_draw(parent, dev(anchor), dev(cid), dev(cl), dev(u), temperature=T)
        assert (o["tree_cand"][:, [1, 3, 6]] == 0).all()          # every first child takes the leading candidate
        assert np.array_equal(host(d["tree_tok"]), o["tree_tok"])
        assert np.array_equal(host(d["tree_cand"]), o["tree_cand"])
        np.testing.assert_allclose(host(d["slot_q"]), o["slot_q"], rtol=1e-6)


def test_bad_arguments():
    w = I.scaled(I.WORKLOADS["tiny"], B=2)
    x = I.propose_inputs(w)
    bad = dict(x, parent=np.array([-1, 0, 0, 0, 1, 2, 3, 3], np.int32))   # three children > k = 2
    with pytest.raises(S.SpecrollError):
        gpu_propose(w, bad)
