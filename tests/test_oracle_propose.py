"""Pins for the proposal half of the CPU oracle (no GPU).

Each test compares the oracle with something other than itself: a library routine on a
special case, a closed form, or the sampling law the paper states.
"""
import itertools

import numpy as np
import pytest
import torch

from oracle import ref
from paper_2608_04962_b200 import inputs as I


def _f64(bits):
    return I.bf16_bits_to_f32(bits).astype(np.float64)


def test_bf16_rounding_matches_torch_and_handles_fp64_midpoints():
    g = I.rng(7)
    x = g.standard_normal(20000).astype(np.float32) * np.float32(3.0)
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = ref.round_bf16(x.astype(np.float64))
    assert np.array_equal(got, want)
    assert np.array_equal(I.f32_to_bf16_bits(x), want)
    # 1 + 2^-8 is a bf16 midpoint between 1.0 and 1.0078125.  Nudged in fp64 below fp32
    # resolution it must go to the side the exact value is on, and the tie goes to even.
    mid = 1.0 + 2.0 ** -8
    got = ref.round_bf16(np.array([mid, mid + 1e-12, mid - 1e-12, -mid - 1e-12]))
    assert list(got) == [0x3F80, 0x3F81, 0x3F80, 0xBF81]


def test_layernorm_against_torch_and_moments():
    w = I.scaled(I.WORKLOADS["tiny"], B=6, d=192, K=2)
    x = I.propose_inputs(w, peaked=True)                     # h ~ N(0,1): eps is negligible
    out = ref.heads(x["h"], x["A"], x["bias"])
    xh = _f64(out["xhat"])                                   # [B,K,d]
    hv = torch.from_numpy(_f64(x["h"]))
    want = torch.nn.functional.layer_norm(hv, (192,), eps=1e-5).numpy()
    for hd in range(2):
        # bf16 storage: relative 2^-9 per element
        np.testing.assert_allclose(xh[:, hd], want, rtol=2.0 ** -8, atol=1e-6)
    assert np.abs(xh.mean(-1)).max() < 2e-3
    np.testing.assert_allclose(xh.var(-1), 1.0, atol=5e-3)


def test_layernorm_affine():
    g = I.rng(11)
    B, K, d = 3, 2, 64
    h = I.f32_to_bf16_bits(g.standard_normal((B, d)).astype(np.float32))
    A = I.f32_to_bf16_bits(np.zeros((K, d, d), np.float32))
    bias = I.f32_to_bf16_bits(np.zeros((K, d), np.float32))
    gam = I.f32_to_bf16_bits(g.uniform(0.5, 1.5, (K, d)).astype(np.float32))
    bet = I.f32_to_bf16_bits(g.standard_normal((K, d)).astype(np.float32))
    out = ref.heads(h, A, bias, gamma=gam, beta=bet)
    hv = torch.from_numpy(_f64(h))
    for hd in range(K):
        want = torch.nn.functional.layer_norm(hv, (d,), torch.from_numpy(_f64(gam[hd])),
                                              torch.from_numpy(_f64(bet[hd])), eps=1e-5).numpy()
        np.testing.assert_allclose(_f64(out["xhat"][:, hd]), want, rtol=2.0 ** -8, atol=1e-6)


def test_head_mlp_against_numpy_matmul_and_torch_silu():
    w = I.scaled(I.WORKLOADS["tiny"], B=5)
    x = I.propose_inputs(w, peaked=True)
    out = ref.heads(x["h"], x["A"], x["bias"])
    xh = _f64(out["xhat"])
    A, bias, h = _f64(x["A"]), _f64(x["bias"]), _f64(x["h"])
    for hd in range(w.K):
        y = xh[:, hd] @ A[hd].T + bias[hd]                      # row = output unit
        want = h + torch.nn.functional.silu(torch.from_numpy(y)).numpy()
        np.testing.assert_allclose(out["z"][:, hd], want, rtol=1e-12, atol=1e-13)
    # a transposed weight matrix must not pass
    y_t = xh[:, 0] @ A[0] + bias[0]
    assert np.abs(out["z"][:, 0] - (h + y_t / (1 + np.exp(-y_t)))).max() > 1e-3


def test_reflex_abstains_exactly_and_has_closed_form_norm():
    w = I.scaled(I.WORKLOADS["tiny"], B=8)
    x = I.propose_inputs(w)
    base = ref.heads(x["h"], x["A"], x["bias"])
    # alpha = 0 everywhere, or no memory: bit-identical to the uncorrected state
    for kw in ({"m": x["m"], "alpha": np.zeros_like(x["alpha"])}, {"m": None, "alpha": None}):
        o = ref.heads(x["h"], x["A"], x["bias"], **kw)
        assert np.array_equal(o["zc"], base["z"])
        assert np.array_equal(o["zt"], ref.round_bf16(base["z"]))
    eps = 1e-6
    alpha = np.full((w.B, w.K), 0.02, np.float32)
    o = ref.heads(x["h"], x["A"], x["bias"], m=x["m"], alpha=alpha, rms_eps=eps)
    dz = o["zc"] - o["z"]
    m = x["m"].astype(np.float64)
    rms_m = np.sqrt((m ** 2).mean(-1))
    want = np.float64(np.float32(0.02)) * np.linalg.norm(o["z"], axis=-1) * rms_m / (rms_m + eps)
    np.testing.assert_allclose(np.linalg.norm(dz, axis=-1), want, rtol=1e-12)
    cos = (dz * m).sum(-1) / (np.linalg.norm(dz, axis=-1) * np.linalg.norm(m, axis=-1))
    np.testing.assert_allclose(cos, 1.0, rtol=1e-12)
    # negative alpha points the other way
    o2 = ref.heads(x["h"], x["A"], x["bias"], m=x["m"], alpha=-alpha)
    np.testing.assert_allclose(o2["zc"] - o2["z"], -dz, rtol=1e-9, atol=1e-15)


def test_reflex_clip_binds_only_above_threshold():
    w = I.scaled(I.WORKLOADS["tiny"], B=8)
    x = I.propose_inputs(w)
    alpha = np.where(np.arange(w.B)[:, None] % 2 == 0, 0.05, 0.3).astype(np.float32) * np.ones((1, w.K), np.float32)
    o = ref.heads(x["h"], x["A"], x["bias"], m=x["m"], alpha=alpha, clip_c=0.1)
    rel = np.linalg.norm(o["zc"] - o["z"], axis=-1) / np.linalg.norm(o["z"], axis=-1)
    np.testing.assert_allclose(rel[1::2], 0.1, rtol=1e-12)           # clipped
    np.testing.assert_allclose(rel[0::2], 0.05, rtol=1e-5)           # untouched (eps shifts 1e-6)
    assert (rel[0::2] < 0.05).all()


def test_correction_before_the_heads_closed_form_abstention_clip_and_composition():
    # the secondary form: one memory row and one ratio per sequence, applied to the last hidden state
    w = I.scaled(I.WORKLOADS["tiny"], B=8)
    x = I.propose_inputs(w, peaked=True)
    hf = _f64(x["h"])
    m1 = x["m"][:, 0, :].copy()
    eps = 1e-6
    # abstention: bit-identical hidden state
    for kw in ({"m": m1, "alpha": np.zeros(w.B, np.float32)}, {"m": None, "alpha": None}):
        o = ref.prehead(x["h"], kw["m"], kw["alpha"])
        assert np.array_equal(o["ht"], x["h"]) and np.array_equal(o["hc"], hf)
    # closed form of the step: |dh| = alpha |h| RMS(m) / (RMS(m) + eps), parallel to m
    alpha = np.full(w.B, 0.03, np.float32)
    o = ref.prehead(x["h"], m1, alpha, rms_eps=eps)
    dh = o["hc"] - hf
    mm = m1.astype(np.float64)
    rms_m = np.sqrt((mm ** 2).mean(-1))
    want = np.float64(np.float32(0.03)) * np.linalg.norm(hf, axis=-1) * rms_m / (rms_m + eps)
    np.testing.assert_allclose(np.linalg.norm(dh, axis=-1), want, rtol=1e-12)
    np.testing.assert_allclose((dh * mm).sum(-1) / (np.linalg.norm(dh, axis=-1) * np.linalg.norm(mm, axis=-1)), 1.0, rtol=1e-12)
    assert np.array_equal(o["ht"], ref.round_bf16(o["hc"]))
    # the clip binds exactly at clip_c |h| and only above it
    alpha2 = np.where(np.arange(w.B) % 2 == 0, 0.05, 0.3).astype(np.float32)
    o2 = ref.prehead(x["h"], m1, alpha2, clip_c=0.1)
    rel = np.linalg.norm(o2["hc"] - hf, axis=-1) / np.linalg.norm(hf, axis=-1)
    np.testing.assert_allclose(rel[1::2], 0.1, rtol=1e-12)
    assert (rel[0::2] < 0.05).all() and (rel[0::2] > 0.0499).all()
    # the proposal in this form = the ordinary proposal, without memory, run on the corrected hidden state
    a = ref.propose(x["h"], x["anchor"], x["A"], x["bias"], x["W"], m1, alpha, x["parent"], x["u_draw"], k=w.k,
                    pre_head=True)
    b = ref.propose(o["ht"], x["anchor"], x["A"], x["bias"], x["W"], None, None, x["parent"], x["u_draw"], k=w.k)
    for key in a:
        assert np.array_equal(a[key], b[key]), key
    # and it is not the per-head form: with the same memory for every head the two give different states
    mk = np.repeat(m1[:, None, :], w.K, axis=1)
    ak = np.repeat(alpha[:, None], w.K, axis=1)
    post = ref.heads(x["h"], x["A"], x["bias"], m=mk, alpha=ak)["zc"]
    pre = ref.heads(o["ht"], x["A"], x["bias"])["zc"]
    assert np.abs(post - pre).max() > 1e-4


def test_projection_against_numpy_and_topk_against_argsort():
    w = I.scaled(I.WORKLOADS["tiny"], B=3, V=777)
    x = I.propose_inputs(w, peaked=True)
    zt = ref.heads(x["h"], x["A"], x["bias"])["zt"]
    lg = ref.lm_logits(zt, x["W"])
    want = _f64(zt).reshape(-1, w.d) @ _f64(x["W"]).T
    np.testing.assert_allclose(lg, want, rtol=1e-11, atol=1e-13)
    k = 5
    cid, cl = ref.topk(lg, k)
    order = np.lexsort((np.arange(w.V)[None, :].repeat(lg.shape[0], 0), -lg), axis=-1)[:, :k]
    assert np.array_equal(cid, order.astype(np.int32))
    assert np.array_equal(cl, np.take_along_axis(lg, order, -1).astype(np.float32))
    cid2, cl2 = ref.lm_topk(zt, x["W"], k)
    assert np.array_equal(cid, cid2) and np.array_equal(cl, cl2)


def test_topk_tie_order_is_lowest_index_first():
    lg = np.array([[1.0, 3.0, 3.0, 0.0, 3.0, 2.0]])
    cid, cl = ref.topk(lg, 4)
    assert cid.tolist() == [[1, 2, 4, 5]]
    assert cl.tolist() == [[3.0, 3.0, 3.0, 2.0]]


def test_tree_draw_follows_the_without_replacement_law():
    # root with 3 children drawn from a 4-candidate support: the ordered list (y1,y2,y3) has
    # probability prod_j w[y_j] / (sum of the weights still available), w = softmax weights.
    n_trials = 400000
    parent = np.array([-1, 0, 0, 0], np.int32)
    logit = np.array([1.0, 0.25, -0.5, 0.0], np.float32)          # sorted order not required by the law
    T = 0.7
    cand_id = np.tile(np.array([[[11, 5, 42, 7]]], np.int32), (n_trials, 1, 1))
    cand_logit = np.tile(logit[None, None, :], (n_trials, 1, 1))
    u = I.uniforms24(123, (n_trials, 4))
    out = ref.tree_draw(parent, np.zeros(n_trials, np.int32), cand_id, cand_logit, u, temperature=T)
    tc = out["tree_cand"][:, 1:].astype(np.int64)
    assert np.array_equal(out["tree_tok"][:, 1:], cand_id[0, 0][tc])
    assert (out["tree_tok"][:, 0] == 0).all()
    # no duplicate children
    assert (np.sort(tc, axis=1)[:, 1:] != np.sort(tc, axis=1)[:, :-1]).all()
    wgt = np.exp(logit.astype(np.float64) / np.float64(np.float32(T)))   # T travels as fp32
    code = tc[:, 0] * 16 + tc[:, 1] * 4 + tc[:, 2]
    for perm in itertools.permutations(range(4), 3):
        pr, left = 1.0, wgt.sum()
        for c in perm:
            pr *= wgt[c] / left
            left -= wgt[c]
        freq = np.mean(code == perm[0] * 16 + perm[1] * 4 + perm[2])
        assert abs(freq - pr) < 4.5 * np.sqrt(pr * (1 - pr) / n_trials), (perm, freq, pr)
    # slot_q of the first child is the full-support softmax; of the last, a 2-way split
    sel = (tc[:, 0] == 2)
    np.testing.assert_allclose(out["slot_q"][sel, 1], wgt[2] / wgt.sum(), rtol=1e-12)
    sel = (tc[:, 0] == 0) & (tc[:, 1] == 1) & (tc[:, 2] == 3)
    np.testing.assert_allclose(out["slot_q"][sel, 3], wgt[3] / (wgt[2] + wgt[3]), rtol=1e-12)


def test_tree_draw_uses_the_head_of_the_node_depth():
    # depth-1 nodes draw from head 1's list, depth-2 nodes from head 2's, whatever the parent.
    parent = np.array([-1, 0, 1, 0, 3], np.int32)
    B = 64
    cand_id = np.zeros((B, 2, 2), np.int32)
    cand_id[:, 0] = [100, 101]
    cand_id[:, 1] = [200, 201]
    cand_logit = np.zeros((B, 2, 2), np.float32)
    out = ref.tree_draw(parent, np.full(B, 9, np.int32), cand_id, cand_logit, I.uniforms24(5, (B, 5)))
    t = out["tree_tok"]
    assert (t[:, 0] == 9).all()
    assert np.isin(t[:, [1, 3]], [100, 101]).all() and (t[:, 1] != t[:, 3]).all()
    assert np.isin(t[:, [2, 4]], [200, 201]).all()
    np.testing.assert_allclose(out["slot_q"][:, [1, 2, 4]], 0.5)
    np.testing.assert_allclose(out["slot_q"][:, 3], 1.0)


def test_propose_is_the_composition_of_its_steps():
    w = I.scaled(I.WORKLOADS["tiny"], B=3, V=300)
    x = I.propose_inputs(w, peaked=True)
    full = ref.propose(x["h"], x["anchor"], x["A"], x["bias"], x["W"], x["m"], x["alpha"], x["parent"],
                       x["u_draw"], k=w.k, clip_c=w.clip_c)
    zt = ref.heads(x["h"], x["A"], x["bias"], m=x["m"], alpha=x["alpha"], clip_c=w.clip_c)["zt"]
    cid, cl = ref.lm_topk(zt, x["W"], w.k)
    assert np.array_equal(full["cand_id"].reshape(-1, w.k), cid)
    d = ref.tree_draw(x["parent"], x["anchor"], full["cand_id"], full["cand_logit"], x["u_draw"])
    assert np.array_equal(d["tree_tok"], full["tree_tok"])


def test_node_budget_values_from_the_paper_setting():
    # C_peak = 512, N in [1, 10] (App. C "Concurrency-aware sparse tree verification")
    for B, want in ((256, 2), (128, 4), (64, 8), (51, 10), (52, 9), (1, 10), (1024, 1)):
        assert ref.node_budget(512, B, 1, 10) == want


def test_topologies():
    p = I.topology(I.WORKLOADS["tiny"])
    assert p.tolist() == [-1, 0, 0, 1, 1, 2, 3, 3]
    for name in ("qwen1.5b", "qwen7b", "qwen14b", "sweep7b_B8"):
        w = I.WORKLOADS[name]
        p = I.topology(w)
        assert len(p) == w.N and p[0] == -1 and all(p[n] < n for n in range(1, w.N))
        assert I.node_depths(p).max() <= w.K
        assert np.bincount(p[1:], minlength=w.N).max() <= w.k
    assert I.node_depths(I.paper_540_topology()).tolist() == [0, 1, 1, 1, 1, 1, 2, 2, 2, 2]
