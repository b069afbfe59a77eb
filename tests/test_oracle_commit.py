"""Pins for the oracle's paged-cache functions (the cache bookkeeping between two speculative steps).

They are index arithmetic, so the pins are round trips against independently written code: the seeded
generator that scatters a contiguous cache into pages, plain Python list concatenation, and numpy fancy
indexing."""
import numpy as np

from oracle import ref
from paper_2608_04962_b200 import inputs as I


def _case(B=3, N=6, seed=5):
    w = I.scaled(I.WORKLOADS["tiny"], B=B, N=N, K=3)
    x = I.attn_inputs(w)
    lengths = np.array([130, 64, 257][:B], np.int32)
    ip = np.zeros(B + 1, np.int32)
    np.cumsum(lengths, out=ip[1:])
    g = I.rng(seed)
    x["kv_indptr"] = ip
    x["Kc"] = I.f32_to_bf16_bits(g.standard_normal((int(ip[-1]), w.Hkv, w.D), dtype=np.float32))
    x["Vc"] = I.f32_to_bf16_bits(g.standard_normal((int(ip[-1]), w.Hkv, w.D), dtype=np.float32))
    return w, x


def test_gathering_the_pages_gives_back_the_cache_that_was_scattered():
    w, x = _case()
    for seed in (1, 2):
        Kp, Vp, pt, pi, kl = I.paged_cache(x["Kc"], x["Vc"], x["kv_indptr"], spare_tokens=5, seed=seed)
        Kc, Vc, ip = ref.paged_to_contiguous(Kp, Vp, pt, pi, kl)
        assert np.array_equal(Kc, x["Kc"]) and np.array_equal(Vc, x["Vc"]) and np.array_equal(ip, x["kv_indptr"])


def test_paged_attention_does_not_depend_on_where_the_pages_are():
    w, x = _case()
    want = ref.tree_attn(x["Q"], x["Kc"], x["Vc"], x["kv_indptr"], x["Kt"], x["Vt"], x["parent"])
    for seed in (1, 2):
        Kp, Vp, pt, pi, kl = I.paged_cache(x["Kc"], x["Vc"], x["kv_indptr"], spare_tokens=5, seed=seed)
        got = ref.tree_attn_paged(x["Q"], Kp, Vp, pt, pi, kl, x["Kt"], x["Vt"], x["parent"])
        assert np.array_equal(got["O64"], want["O64"])


def test_commit_appends_anchor_and_accepted_rows_in_path_order():
    w, x = _case()
    B, N, K = w.B, w.N, w.K
    Kp, Vp, pt, pi, kl = I.paged_cache(x["Kc"], x["Vc"], x["kv_indptr"], spare_tokens=K + 1, seed=3)
    path = np.array([[0, 2, 5, -1], [0, -1, -1, -1], [0, 1, 3, 4]], np.int32)   # second sequence accepts nothing
    n_acc = np.array([2, 0, 3], np.int32)
    out = ref.commit_path(x["Kt"], x["Vt"], path, n_acc, Kp, Vp, pt, pi, kl)
    assert not out["overflow"] and np.array_equal(out["kv_len"], kl + n_acc + 1)
    Kc2, Vc2, ip2 = ref.paged_to_contiguous(out["Kp"], out["Vp"], pt, pi, out["kv_len"])
    # the same cache written out by hand: old rows, then the path's tree rows in order
    for b in range(B):
        rows_k = [x["Kc"][t] for t in range(x["kv_indptr"][b], x["kv_indptr"][b + 1])]
        rows_v = [x["Vc"][t] for t in range(x["kv_indptr"][b], x["kv_indptr"][b + 1])]
        for i in range(n_acc[b] + 1):
            rows_k.append(x["Kt"][b, path[b, i]])
            rows_v.append(x["Vt"][b, path[b, i]])
        assert np.array_equal(np.stack(rows_k), Kc2[ip2[b]:ip2[b + 1]])
        assert np.array_equal(np.stack(rows_v), Vc2[ip2[b]:ip2[b + 1]])
    # the third sequence crossed a page boundary (257 + 4 tokens > 2 pages would not, 256 is the edge)
    assert kl[2] // 128 != (out["kv_len"][2] - 1) // 128 or kl[2] % 128 != 0
    # untouched: everything outside the appended rows
    changed = (out["Kp"] != Kp).any(axis=(2, 3))
    assert changed.sum() <= int((n_acc + 1).sum())


def test_commit_then_attention_equals_attention_over_the_extended_sequence():
    # a committed token must be attended by the next step exactly like any cached token
    w, x = _case()
    Kp, Vp, pt, pi, kl = I.paged_cache(x["Kc"], x["Vc"], x["kv_indptr"], spare_tokens=8, seed=4)
    path = np.array([[0, 1, -1, -1], [0, 2, 5, -1], [0, -1, -1, -1]], np.int32)
    n_acc = np.array([1, 2, 0], np.int32)
    out = ref.commit_path(x["Kt"], x["Vt"], path, n_acc, Kp, Vp, pt, pi, kl)
    got = ref.tree_attn_paged(x["Q"], out["Kp"], out["Vp"], pt, pi, out["kv_len"], x["Kt"], x["Vt"], x["parent"])
    Kc = np.concatenate([np.concatenate([x["Kc"][x["kv_indptr"][b]:x["kv_indptr"][b + 1]],
                                         x["Kt"][b, path[b, :n_acc[b] + 1]]]) for b in range(w.B)])
    Vc = np.concatenate([np.concatenate([x["Vc"][x["kv_indptr"][b]:x["kv_indptr"][b + 1]],
                                         x["Vt"][b, path[b, :n_acc[b] + 1]]]) for b in range(w.B)])
    ip = np.zeros(w.B + 1, np.int32)
    np.cumsum(kl + n_acc + 1, out=ip[1:])
    want = ref.tree_attn(x["Q"], Kc, Vc, ip, x["Kt"], x["Vt"], x["parent"])
    assert np.array_equal(got["O64"], want["O64"])


def test_commit_reports_a_sequence_that_has_no_room():
    w, x = _case()
    Kp, Vp, pt, pi, kl = I.paged_cache(x["Kc"], x["Vc"], x["kv_indptr"], spare_tokens=0, seed=6)
    path = np.tile(np.array([0, 1, 2, 3], np.int32), (w.B, 1))
    n_acc = np.full(w.B, 3, np.int32)
    out = ref.commit_path(x["Kt"], x["Vt"], path, n_acc, Kp, Vp, pt, pi, kl)
    assert not out["overflow"]      # 130 of 256, 64 of 128 and 257 of 384 tokens: four more fit everywhere
    kl2 = kl.copy()
    kl2[1] = 126                    # 126 + 4 tokens do not fit the sequence's single page
    out2 = ref.commit_path(x["Kt"], x["Vt"], path, n_acc, Kp, Vp, pt, pi, kl2)
    assert out2["overflow"] and out2["kv_len"][1] == 130
    page = pt[pi[1]]
    assert np.array_equal(out2["Kp"][page, 126], x["Kt"][1, 0]) and np.array_equal(out2["Kp"][page, 127], x["Kt"][1, 1])


def test_gather_hidden_is_a_row_pick():
    g = I.rng(9)
    hidden = g.integers(0, 65535, size=(5, 7, 16), dtype=np.uint16)
    term = np.array([0, 6, 3, 3, 1], np.int32)
    assert np.array_equal(ref.gather_hidden(hidden, term), hidden[np.arange(5), term])
