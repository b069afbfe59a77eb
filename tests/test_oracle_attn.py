"""Pins for the tree-attention oracle (no GPU).

The packed evaluation must equal an ordinary autoregressive forward at every node's own
prefix; the pins rebuild that forward another way (per-path full softmax through torch's
SDPA in fp64) and check library special cases and invariants.
"""
import numpy as np
import torch
import torch.nn.functional as F
from scipy.special import logsumexp

from oracle import ref
from paper_2608_04962_b200 import inputs as I


def _f64(bits):
    return torch.from_numpy(I.bf16_bits_to_f32(bits).astype(np.float64))


def _path(parent, n):
    p = []
    while n >= 0:
        p.append(n)
        n = int(parent[n])
    return p[::-1]


def _small(**kw):
    return I.scaled(I.WORKLOADS["tiny"], **kw)


def test_each_node_equals_plain_decode_over_its_own_prefix():
    w = _small(B=3, Hq=6, Hkv=2, D=32, kv_a=5, kv_b=40)
    x = I.attn_inputs(w)
    out = ref.tree_attn(x["Q"], x["Kc"], x["Vc"], x["kv_indptr"], x["Kt"], x["Vt"], x["parent"],
                        want_lse=True)
    Q, Kc, Vc, Kt, Vt = (_f64(x[n]) for n in ("Q", "Kc", "Vc", "Kt", "Vt"))
    G = w.Hq // w.Hkv
    for b in range(w.B):
        lo, hi = x["kv_indptr"][b], x["kv_indptr"][b + 1]
        for n in range(w.N):
            path = _path(x["parent"], n)
            K_all = torch.cat([Kc[lo:hi], Kt[b, path]], 0)           # [S, Hkv, D]
            V_all = torch.cat([Vc[lo:hi], Vt[b, path]], 0)
            K_all = K_all.permute(1, 0, 2).repeat_interleave(G, 0)    # [Hq, S, D]
            V_all = V_all.permute(1, 0, 2).repeat_interleave(G, 0)
            q = Q[b, n][:, None, :]                                   # [Hq, 1, D]
            want = F.scaled_dot_product_attention(q[None], K_all[None], V_all[None])[0, :, 0]
            np.testing.assert_allclose(out["O64"][b, n], want.numpy(), rtol=1e-10, atol=1e-12)
            s = (q @ K_all.transpose(1, 2))[:, 0] / np.sqrt(w.D)
            np.testing.assert_allclose(out["lse"][b, n], logsumexp(s.numpy(), axis=-1), rtol=1e-12)
    assert np.array_equal(out["Obf"], ref.round_bf16(out["O64"]))


def test_chain_topology_is_causal_attention_over_the_appended_tokens():
    N = 6
    w = _small(B=2, N=N, Hq=4, Hkv=4, D=16, kv_a=9, kv_b=9, fixed_parent=tuple(range(-1, N - 1)))
    x = I.attn_inputs(w)
    out = ref.tree_attn(x["Q"], x["Kc"], x["Vc"], x["kv_indptr"], x["Kt"], x["Vt"], x["parent"])
    Q, Kc, Vc, Kt, Vt = (_f64(x[n]) for n in ("Q", "Kc", "Vc", "Kt", "Vt"))
    L = 9
    mask = torch.ones(N, L + N, dtype=torch.bool).tril(diagonal=L)   # query i sees cache + tokens 0..i
    for b in range(2):
        Kall = torch.cat([Kc[b * L:(b + 1) * L], Kt[b]], 0).permute(1, 0, 2)
        Vall = torch.cat([Vc[b * L:(b + 1) * L], Vt[b]], 0).permute(1, 0, 2)
        want = F.scaled_dot_product_attention(Q[b].permute(1, 0, 2)[None], Kall[None], Vall[None],
                                              attn_mask=mask)[0].permute(1, 0, 2)
        np.testing.assert_allclose(out["O64"][b], want.numpy(), rtol=1e-10, atol=1e-12)


def test_star_topology_siblings_do_not_see_each_other():
    # root + 4 leaves: leaf i sees cache, root, itself.  With identical leaf queries and
    # identical leaf K/V, outputs are identical; changing leaf 2's V changes only leaf 2.
    w = _small(B=1, N=5, Hq=2, Hkv=1, D=16, kv_a=7, kv_b=7, fixed_parent=(-1, 0, 0, 0, 0))
    x = I.attn_inputs(w)
    for name in ("Q", "Kt", "Vt"):
        x[name][:, 2:] = x[name][:, 1:2]
    o1 = ref.tree_attn(x["Q"], x["Kc"], x["Vc"], x["kv_indptr"], x["Kt"], x["Vt"], x["parent"])["O64"]
    assert np.array_equal(o1[0, 1], o1[0, 2]) and np.array_equal(o1[0, 1], o1[0, 4])
    x["Vt"][0, 2] = I.f32_to_bf16_bits(np.full((1, 16), 3.0, np.float32))
    o2 = ref.tree_attn(x["Q"], x["Kc"], x["Vc"], x["kv_indptr"], x["Kt"], x["Vt"], x["parent"])["O64"]
    assert np.array_equal(o2[0, [0, 1, 3, 4]], o1[0, [0, 1, 3, 4]])
    assert np.abs(o2[0, 2] - o1[0, 2]).max() > 1e-3


def test_invariants_permutation_and_convex_hull_and_gqa_mapping():
    w = _small(B=2, Hq=6, Hkv=3, D=16, kv_a=20, kv_b=30)
    x = I.attn_inputs(w)
    o = ref.tree_attn(x["Q"], x["Kc"], x["Vc"], x["kv_indptr"], x["Kt"], x["Vt"], x["parent"])["O64"]
    # permuting a sequence's cache rows (K and V together) changes nothing but rounding order
    perm = np.arange(x["Kc"].shape[0])
    lo, hi = x["kv_indptr"][1], x["kv_indptr"][2]
    perm[lo:hi] = perm[lo:hi][::-1]
    o2 = ref.tree_attn(x["Q"], x["Kc"][perm], x["Vc"][perm], x["kv_indptr"], x["Kt"], x["Vt"],
                       x["parent"])["O64"]
    np.testing.assert_allclose(o2, o, rtol=1e-11, atol=1e-13)
    # outputs are convex combinations of the attended V rows
    Vc, Vt = _f64(x["Vc"]).numpy(), _f64(x["Vt"]).numpy()
    G = 2
    for b in range(2):
        lo, hi = x["kv_indptr"][b], x["kv_indptr"][b + 1]
        for hq in range(6):
            cols = np.concatenate([Vc[lo:hi, hq // G], Vt[b, :, hq // G]], 0)
            assert (o[b, :, hq] <= cols.max(0) + 1e-12).all() and (o[b, :, hq] >= cols.min(0) - 1e-12).all()
    # query head hq reads KV head hq // G: zeroing KV head 0's values zeroes exactly heads 0,1
    Vc0, Vt0 = x["Vc"].copy(), x["Vt"].copy()
    Vc0[:, 0] = 0
    Vt0[:, :, 0] = 0
    o3 = ref.tree_attn(x["Q"], x["Kc"], Vc0, x["kv_indptr"], x["Kt"], Vt0, x["parent"])["O64"]
    assert (o3[:, :, :2] == 0).all() and np.array_equal(o3[:, :, 2:], o[:, :, 2:])


def test_scale_argument_and_empty_cache():
    w = _small(B=2, N=3, Hq=2, Hkv=1, D=16, kv_a=0, kv_b=0, fixed_parent=(-1, 0, 1))
    x = I.attn_inputs(w)
    assert x["Kc"].shape[0] == 0
    o = ref.tree_attn(x["Q"], x["Kc"], x["Vc"], x["kv_indptr"], x["Kt"], x["Vt"], x["parent"],
                      scale=0.0)["O64"]
    Vt = _f64(x["Vt"]).numpy()
    # zero scale -> uniform average over the visible tree rows
    np.testing.assert_allclose(o[:, 0, 0], Vt[:, 0, 0], rtol=1e-12)
    np.testing.assert_allclose(o[:, 2, 1], Vt[:, :3, 0].mean(1), rtol=1e-12)
