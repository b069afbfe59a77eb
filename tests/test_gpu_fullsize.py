"""GPU parity at the full benchmark sizes, in the launch configuration bench.py times.

The oracle cannot run a whole full-size step in seconds, so each test runs the CUDA path on the
complete workload (same tensors, same workspaces, same calls as the benchmark's step) and checks a
sample of sequences that the oracle computes one by one from the very same device data: the
shortest and the longest sequence (the longest is split over several CTAs and merged), the one
nearest the median, and a few seeded random ones.
"""
import numpy as np
import pytest
import torch

from oracle import ref
from paper_2608_04962_b200 import binding as S
from paper_2608_04962_b200 import inputs as I
from paper_2608_04962_b200.workload import StepWorkload

pytestmark = pytest.mark.gpu


def _sample(wl, n_random, seed):
    L = np.diff(wl.kv_indptr_host)
    picks = {int(L.argmin()), int(L.argmax()), int(np.abs(L - np.median(L)).argmin())}
    g = I.rng(seed)
    while len(picks) < min(wl.w.B, 3 + n_random):
        picks.add(int(g.integers(0, wl.w.B)))
    return sorted(picks)


def _bits(t):
    return S.bf16_bits(t)


@pytest.mark.parametrize("name,n_random", [("qwen1.5b", 3), ("qwen7b", 1), ("qwen14b", 1), ("sweep7b_B8", 1),
                                           ("sweep7b_B16", 0), ("sweep7b_B32", 0), ("sweep7b_B64", 0),
                                           ("sweep7b_B128", 0), ("sweep7b_B256", 0)])
def test_full_size_step_sampled_against_the_oracle(name, n_random):
    w = I.WORKLOADS[name]
    # three layers: the later ones keep the first one's plan and may load their first cache tiles while the layer
    # before is still finishing, as all but the first layer of the benchmark's step do
    wl = StepWorkload(w, torch.device("cuda", 0), layers=3)
    wl.step()
    torch.cuda.synchronize()
    assert S.workspace_status(wl.ws_attn) == 0 and S.workspace_status(wl.ws_propose) == 0
    picks = _sample(wl, n_random, seed=w.cfg_id)
    ip = wl.kv_indptr_host

    # ---- tree attention: the sampled sequences as a small oracle batch
    lens = np.array([ip[b + 1] - ip[b] for b in picks], np.int32)
    sub_ip = np.zeros(len(picks) + 1, np.int32)
    np.cumsum(lens, out=sub_ip[1:])
    Kc = np.concatenate([_bits(wl.Kc[0][ip[b]:ip[b + 1]]) for b in picks], 0)
    Vc = np.concatenate([_bits(wl.Vc[0][ip[b]:ip[b + 1]]) for b in picks], 0)
    idx = torch.tensor(picks, device=wl.device)
    o = ref.tree_attn(_bits(wl.Q[0][idx]), Kc, Vc, sub_ip, _bits(wl.Kt[0][idx]), _bits(wl.Vt[0][idx]), wl.parent)
    got = wl.O[0][idx].float().cpu().numpy().astype(np.float64)
    err = np.abs(got - o["O64"]).max()
    assert err <= 1e-2, (name, err)
    # ... and the last layer, on fewer sequences (the oracle's time)
    few = picks[:3]
    lens = np.array([ip[b + 1] - ip[b] for b in few], np.int32)
    sub_ip = np.zeros(len(few) + 1, np.int32)
    np.cumsum(lens, out=sub_ip[1:])
    last = wl.layers - 1
    Kc = np.concatenate([_bits(wl.Kc[last][ip[b]:ip[b + 1]]) for b in few], 0)
    Vc = np.concatenate([_bits(wl.Vc[last][ip[b]:ip[b + 1]]) for b in few], 0)
    fidx = torch.tensor(few, device=wl.device)
    o = ref.tree_attn(_bits(wl.Q[last][fidx]), Kc, Vc, sub_ip, _bits(wl.Kt[last][fidx]), _bits(wl.Vt[last][fidx]), wl.parent)
    got = wl.O[last][fidx].float().cpu().numpy().astype(np.float64)
    err = np.abs(got - o["O64"]).max()
    assert err <= 1e-2, (name, "last layer", err)
    assert torch.isfinite(wl.O[last].float()).all()

    # ---- verification: the oracle on the sampled sequences' logits, with the GPU's own proposal as input
    p = {k: v[idx].cpu().numpy() for k, v in wl.prop.items()}
    ov = ref.verify(_bits(wl.logits[idx]), wl.parent, p["tree_tok"], p["tree_cand"], p["cand_id"], p["cand_logit"],
                    wl.u_acc[idx].cpu().numpy(), wl.u_fin[idx].cpu().numpy(), temperature=w.temperature)
    gv = {k: v[idx].cpu().numpy() for k, v in wl.ver.items()}
    assert np.array_equal(gv["row_max"].astype(np.float64), ov["row_max"])
    assert np.abs(gv["row_sum"] / ov["row_sum"] - 1).max() < 2e-5
    for i in range(len(picks)):
        same = gv["n_acc"][i] == ov["n_acc"][i] and np.array_equal(gv["out_tok"][i], ov["out_tok"][i]) and \
            np.array_equal(gv["path_node"][i], ov["path_node"][i])
        assert same or ov["min_margin"][i] < 1e-4 or ov["fin_margin"][i] < 1e-6, (name, picks[i])

    # ---- proposal: heads + projection + top-k of the sampled sequences (tie-aware), then the draw
    A, bias, W = _bits(wl.A), _bits(wl.bias), _bits(wl.W)
    hd = ref.heads(_bits(wl.h[idx]), A, bias, m=wl.m[idx].cpu().numpy(), alpha=wl.alpha[idx].cpu().numpy(),
                   clip_c=w.clip_c)
    full = ref.lm_logits(hd["zt"], W)                             # [n*K, V]
    oid, ol = ref.topk(full, w.k)
    gid = p["cand_id"].reshape(-1, w.k)
    rows = np.arange(full.shape[0])[:, None]
    kth = ol[:, -1].astype(np.float64)
    picked = full[rows, gid]
    assert (picked >= kth[:, None] - 1e-3).all()
    must = full > (kth[:, None] + 1e-3)
    have = np.zeros_like(must)
    have[rows, gid] = True
    assert (have | ~must).all()
    # The bar is 1e-3 on a logit (= 1e-3 relative on its probability).  One explicit allowance: the GPU rounds the
    # corrected state z~ to bf16 from an fp32 value, the oracle from the fp64 one, so an element that lies within
    # the GPU's own error of the midpoint between two bf16 values may round to the other neighbour, which moves a
    # logit by (bf16 step of z_i) * |W[v, i]|.  Those elements are found from the oracle's unrounded z~ (fp32 sums
    # over d terms: 4e-6 relative is a generous bound on the GPU's error), the allowance is their worst case, and
    # few logits may need it at all.
    zc = hd["zc"].reshape(-1, w.d)
    zt = I.bf16_bits_to_f32(hd["zt"].reshape(-1, w.d)).astype(np.float64)
    step = 2.0 ** (np.floor(np.log2(np.maximum(np.abs(zt), 1e-30))) - 7)
    at_risk = np.abs(np.abs(zc - zt) - 0.5 * step) <= 4e-6 * np.abs(zc)
    Wf = I.bf16_bits_to_f32(W).astype(np.float64)
    allow = np.full(gid.shape, 1e-3)
    for r in np.nonzero(at_risk.any(-1))[0]:
        cols = np.nonzero(at_risk[r])[0]
        allow[r] += (np.abs(Wf[gid[r]][:, cols]) * step[r, cols][None, :]).sum(-1)
    dl = np.abs(p["cand_logit"].reshape(-1, w.k).astype(np.float64) - picked)
    assert (dl <= allow).all(), (name, float((dl - allow).max()))
    assert (dl > 1e-3).mean() < 0.01, (name, float((dl > 1e-3).mean()))
    d = ref.tree_draw(wl.parent, wl.anchor[idx].cpu().numpy(), p["cand_id"], p["cand_logit"],
                      wl.u_draw[idx].cpu().numpy(), temperature=w.temperature)
    assert np.array_equal(p["tree_tok"], d["tree_tok"])
    np.testing.assert_allclose(p["slot_q"], d["slot_q"], rtol=1e-5)

    # ---- the same chain with nothing of the GPU's in the oracle's inputs: for the sampled sequences whose
    #      candidate lists the oracle reproduces id for id (no ties at the cut), the oracle's own lists, its own
    #      draw and its own verification must give the GPU's tokens
    oid3, ol3 = oid.reshape(len(picks), w.K, w.k), ol.reshape(len(picks), w.K, w.k).astype(np.float32)
    clean = [i for i in range(len(picks)) if np.array_equal(oid3[i], p["cand_id"][i])]
    if clean:
        ci = np.array(clean)
        d2 = ref.tree_draw(wl.parent, wl.anchor[idx].cpu().numpy()[ci], oid3[ci], ol3[ci],
                           wl.u_draw[idx].cpu().numpy()[ci], temperature=w.temperature)
        ov2 = ref.verify(_bits(wl.logits[idx])[ci], wl.parent, d2["tree_tok"], d2["tree_cand"], oid3[ci], ol3[ci],
                         wl.u_acc[idx].cpu().numpy()[ci], wl.u_fin[idx].cpu().numpy()[ci], temperature=w.temperature)
        for j, i in enumerate(clean):
            if not np.array_equal(d2["tree_tok"][j], p["tree_tok"][i]):
                continue   # a draw decided within rounding of a uniform (the lists' logits differ in their last bits)
            same = gv["n_acc"][i] == ov2["n_acc"][j] and np.array_equal(gv["out_tok"][i], ov2["out_tok"][j]) and \
                np.array_equal(gv["path_node"][i], ov2["path_node"][j])
            assert same or ov2["min_margin"][j] < 1e-4 or ov2["fin_margin"][j] < 1e-6, (name, picks[i], "oracle-only chain")

    # ---- properties that hold for every sequence of the full batch
    n_acc = wl.ver["n_acc"].cpu().numpy()
    path = wl.ver["path_node"].cpu().numpy()
    out_tok = wl.ver["out_tok"].cpu().numpy()
    tree_tok = wl.prop["tree_tok"].cpu().numpy()
    assert (n_acc >= 0).all() and (n_acc <= w.K).all() and (path[:, 0] == 0).all()
    for b in range(w.B):
        n = n_acc[b]
        assert (path[b, n + 1:] == -1).all() and 0 <= out_tok[b, n] < w.V
        for i in range(1, n + 1):
            assert wl.parent[path[b, i]] == path[b, i - 1] and out_tok[b, i - 1] == tree_tok[b, path[b, i]]
    O_all = wl.O[0].float()
    assert torch.isfinite(O_all).all()
    cid = wl.prop["cand_id"].cpu().numpy()
    assert (cid >= 0).all() and (cid < w.V).all()
    assert (np.sort(cid, -1)[..., 1:] != np.sort(cid, -1)[..., :-1]).all()
    cl = wl.prop["cand_logit"].cpu().numpy()
    assert (np.diff(cl, axis=-1) <= 0).all()


def test_projection_and_top_k_of_a_whole_row_block():
    """Every row of the first 128-row block of the projection's M dimension (32 sequences x 4 heads of the 1.5B
    shape) against the oracle's full logits: the block is what one CTA column of the kernel owns."""
    w = I.WORKLOADS["qwen1.5b"]
    wl = StepWorkload(w, torch.device("cuda", 0), layers=1)
    wl.propose()
    torch.cuda.synchronize()
    assert S.workspace_status(wl.ws_propose) == 0
    n_seq = 128 // w.K
    sl = slice(0, n_seq)
    A, bias, W = _bits(wl.A), _bits(wl.bias), _bits(wl.W)
    hd = ref.heads(_bits(wl.h[sl]), A, bias, m=wl.m[sl].cpu().numpy(), alpha=wl.alpha[sl].cpu().numpy(),
                   clip_c=w.clip_c)
    full = ref.lm_logits(hd["zt"], W)                             # [128, V]
    oid, ol = ref.topk(full, w.k)
    gid = wl.prop["cand_id"][sl].cpu().numpy().reshape(-1, w.k)
    gl = wl.prop["cand_logit"][sl].cpu().numpy().reshape(-1, w.k).astype(np.float64)
    rows = np.arange(full.shape[0])[:, None]
    kth = ol[:, -1].astype(np.float64)
    picked = full[rows, gid]
    assert (picked >= kth[:, None] - 1e-3).all()                  # nothing below the cut (ties within 1e-3 aside)
    must = full > (kth[:, None] + 1e-3)
    have = np.zeros_like(must)
    have[rows, gid] = True
    assert (have | ~must).all()                                   # nothing above the cut is missing
    assert np.abs(gl - picked).max() <= 1e-3
    assert (np.diff(gl, axis=-1) <= 0).all()                      # lists sorted by logit
