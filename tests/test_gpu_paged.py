"""GPU parity of the paged-cache entry points: attention through a page table, committing the accepted
path, picking the next step's hidden state.  Attention within 1e-2 of the oracle (the bar of the contiguous
entry point); the copies bit-exact."""
import numpy as np
import pytest
import torch

from oracle import ref
from paper_2608_04962_b200 import binding as S
from paper_2608_04962_b200 import inputs as I
from tests.util import dev, dev_bf16, host

pytestmark = pytest.mark.gpu

O_ATOL = 1e-2


def _inputs(w, lengths, seed=77):
    x = I.attn_inputs(w)
    lengths = np.asarray(lengths, np.int32)
    ip = np.zeros(w.B + 1, np.int32)
    np.cumsum(lengths, out=ip[1:])
    g = I.rng(seed)
    x["kv_indptr"] = ip
    x["Kc"] = I.f32_to_bf16_bits(g.standard_normal((int(ip[-1]), w.Hkv, w.D), dtype=np.float32))
    x["Vc"] = I.f32_to_bf16_bits(g.standard_normal((int(ip[-1]), w.Hkv, w.D), dtype=np.float32))
    return x


def _gpu_paged(x, Kp, Vp, pt, pi, kl, **kw):
    return S.tree_attn_paged(dev_bf16(x["Q"]), dev_bf16(Kp), dev_bf16(Vp), dev(pt), dev(pi), dev(kl), kl,
                             dev_bf16(x["Kt"]), dev_bf16(x["Vt"]), x["parent"], check_status=True, **kw)


@pytest.mark.parametrize("Hq,Hkv,D,N,lengths", [
    (12, 2, 128, 16, [700, 64, 1, 333, 129]),          # one row block
    (28, 4, 128, 32, [900, 128, 70, 0, 257]),           # two row blocks (two units per chunk and KV head); an empty cache
    (14, 2, 64, 37, [640, 64, 300, 127, 129]),          # three row blocks, head dim 64
    (12, 2, 128, 16, [5000, 64, 700, 129, 256]),        # a sequence cut into many chunks (merge kernel)
])
def test_paged_attention_matches_the_oracle(Hq, Hkv, D, N, lengths):
    w = I.scaled(I.WORKLOADS["qwen7b"], B=5, N=N, K=5, Hq=Hq, Hkv=Hkv, D=D, kv_a=300, kv_b=900)
    x = _inputs(w, lengths)
    Kp, Vp, pt, pi, kl = I.paged_cache(x["Kc"], x["Vc"], x["kv_indptr"], spare_tokens=9, seed=11)
    want = ref.tree_attn_paged(x["Q"], Kp, Vp, pt, pi, kl, x["Kt"], x["Vt"], x["parent"], want_lse=True)
    O, lse = _gpu_paged(x, Kp, Vp, pt, pi, kl, want_lse=True)
    torch.cuda.synchronize()
    diff = np.abs(host(O.float()).astype(np.float64) - want["O64"])
    assert (diff <= O_ATOL * np.maximum(1.0, np.abs(want["O64"]))).all(), diff.max()
    np.testing.assert_allclose(host(lse).astype(np.float64), want["lse"], atol=2e-3, rtol=0)
    # and it is the same function as the contiguous entry point on the same cache
    O2 = S.tree_attn(dev_bf16(x["Q"]), dev_bf16(x["Kc"]), dev_bf16(x["Vc"]), dev(x["kv_indptr"]), x["kv_indptr"],
                     dev_bf16(x["Kt"]), dev_bf16(x["Vt"]), x["parent"])
    assert torch.equal(O, O2)


def test_plan_reuse_with_a_paged_cache():
    w = I.scaled(I.WORKLOADS["qwen1.5b"], B=6)
    x = _inputs(w, [700, 64, 1500, 333, 129, 2900])
    Kp, Vp, pt, pi, kl = I.paged_cache(x["Kc"], x["Vc"], x["kv_indptr"], spare_tokens=0, seed=12)
    ws = torch.empty(S.tree_attn_paged_workspace_bytes(w.B, w.N, w.Hq, w.Hkv, w.D, kl), dtype=torch.uint8, device="cuda")
    a = _gpu_paged(x, Kp, Vp, pt, pi, kl, workspace=ws)
    b = _gpu_paged(x, Kp, Vp, pt, pi, kl, workspace=ws, flags=S.ATTN_REUSE_PLAN)
    assert torch.equal(a, b)
    # back to back, with the first pages of a call fetched while the call before is finishing
    outs = [S.tree_attn_paged(dev_bf16(x["Q"]), dev_bf16(Kp), dev_bf16(Vp), dev(pt), dev(pi), dev(kl), kl,
                              dev_bf16(x["Kt"]), dev_bf16(x["Vt"]), x["parent"], workspace=ws,
                              flags=S.ATTN_REUSE_PLAN | S.ATTN_CACHE_SETTLED) for _ in range(4)]
    torch.cuda.synchronize()
    assert S.workspace_status(ws) == 0
    for o in outs:
        assert torch.equal(a, o)


def test_paged_needs_the_tcgen05_kernel():
    w = I.scaled(I.WORKLOADS["tiny"], B=2)
    x = I.attn_inputs(w)
    Kp, Vp, pt, pi, kl = I.paged_cache(x["Kc"], x["Vc"], x["kv_indptr"], spare_tokens=0, seed=13)
    with pytest.raises(S.SpecrollError):
        _gpu_paged(x, Kp, Vp, pt, pi, kl, flags=S.ATTN_LEGACY_MMA)


def test_commit_path_and_the_next_step():
    w = I.scaled(I.WORKLOADS["qwen1.5b"], B=4, N=16, K=4)
    x = _inputs(w, [126, 64, 257, 1000])
    K = w.K
    Kp, Vp, pt, pi, kl = I.paged_cache(x["Kc"], x["Vc"], x["kv_indptr"], spare_tokens=K + 1, seed=14)
    # paths as the walk writes them: root, then accepted nodes (a child of the previous one), then -1
    parent = x["parent"]
    kids = {u: [n for n in range(w.N) if parent[n] == u] for u in range(w.N)}
    path = np.full((w.B, K + 1), -1, np.int32)
    n_acc = np.array([3, 0, 2, 1], np.int32)
    g = I.rng(15)
    for b in range(w.B):
        path[b, 0] = 0
        for i in range(1, n_acc[b] + 1):
            ch = kids[int(path[b, i - 1])]
            if not ch:
                n_acc[b] = i - 1
                break
            path[b, i] = ch[int(g.integers(0, len(ch)))]
    want = ref.commit_path(x["Kt"], x["Vt"], path, n_acc, Kp, Vp, pt, pi, kl)
    dKp, dVp, dkl = dev_bf16(Kp), dev_bf16(Vp), dev(kl)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    S.commit_path(dev_bf16(x["Kt"]), dev_bf16(x["Vt"]), dev(path), dev(n_acc), dKp, dVp, dev(pt), dev(pi), dkl,
                  kv_len_out=dkl, status=status)           # lengths updated in place
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and not want["overflow"]
    assert np.array_equal(S.bf16_bits(dKp), want["Kp"]) and np.array_equal(S.bf16_bits(dVp), want["Vp"])
    assert np.array_equal(host(dkl), want["kv_len"])
    # the next step attends the committed tokens like any cached token
    nl = want["kv_len"]
    o = ref.tree_attn_paged(x["Q"], want["Kp"], want["Vp"], pt, pi, nl, x["Kt"], x["Vt"], parent)
    O = S.tree_attn_paged(dev_bf16(x["Q"]), dKp, dVp, dev(pt), dev(pi), dkl, nl, dev_bf16(x["Kt"]), dev_bf16(x["Vt"]),
                          parent, check_status=True)
    assert np.abs(host(O.float()).astype(np.float64) - o["O64"]).max() <= O_ATOL


def test_commit_without_room_is_reported_and_writes_nothing_out_of_place():
    w = I.scaled(I.WORKLOADS["qwen1.5b"], B=3, N=16, K=4)
    x = _inputs(w, [126, 64, 250])
    Kp, Vp, pt, pi, kl = I.paged_cache(x["Kc"], x["Vc"], x["kv_indptr"], spare_tokens=0, seed=16)
    path = np.tile(np.array([0, 1, 2, 3, 4], np.int32), (w.B, 1))
    n_acc = np.full(w.B, 4, np.int32)
    want = ref.commit_path(x["Kt"], x["Vt"], path, n_acc, Kp, Vp, pt, pi, kl)
    assert want["overflow"]
    dKp, dVp = dev_bf16(Kp), dev_bf16(Vp)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out_len = torch.zeros(w.B, dtype=torch.int32, device="cuda")
    S.commit_path(dev_bf16(x["Kt"]), dev_bf16(x["Vt"]), dev(path), dev(n_acc), dKp, dVp, dev(pt), dev(pi), dev(kl),
                  kv_len_out=out_len, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 6
    assert np.array_equal(S.bf16_bits(dKp), want["Kp"]) and np.array_equal(S.bf16_bits(dVp), want["Vp"])
    assert np.array_equal(host(out_len), want["kv_len"])


def test_commit_all_layers_in_one_call():
    w = I.scaled(I.WORKLOADS["qwen1.5b"], B=3, N=16, K=4)
    path = np.array([[0, 1, 4, -1, -1], [0, -1, -1, -1, -1], [0, 2, -1, -1, -1]], np.int32)
    n_acc = np.array([2, 0, 1], np.int32)
    layers, want, args = 3, [], ([], [], [], [])
    for l in range(layers):
        x = _inputs(w, [126, 64, 257], seed=100 + l)
        g = I.rng(200 + l)
        x["Kt"] = I.f32_to_bf16_bits(g.standard_normal(x["Kt"].shape, dtype=np.float32))
        x["Vt"] = I.f32_to_bf16_bits(g.standard_normal(x["Vt"].shape, dtype=np.float32))
        Kp, Vp, pt, pi, kl = I.paged_cache(x["Kc"], x["Vc"], x["kv_indptr"], spare_tokens=5, seed=19)  # same table
        want.append(ref.commit_path(x["Kt"], x["Vt"], path, n_acc, Kp, Vp, pt, pi, kl))
        for lst, a in zip(args, (x["Kt"], x["Vt"], Kp, Vp)):
            lst.append(dev_bf16(a))
    dkl = dev(kl)
    S.commit_path_layers(args[0], args[1], dev(path), dev(n_acc), args[2], args[3], dev(pt), dev(pi), dkl, kv_len_out=dkl)
    torch.cuda.synchronize()
    for l in range(layers):
        assert np.array_equal(S.bf16_bits(args[2][l]), want[l]["Kp"]) and np.array_equal(S.bf16_bits(args[3][l]), want[l]["Vp"])
    assert np.array_equal(host(dkl), want[0]["kv_len"])


def test_gather_hidden():
    g = I.rng(17)
    hidden = g.integers(0, 65535, size=(9, 16, 1536), dtype=np.uint16)
    term = g.integers(0, 16, size=9).astype(np.int32)
    got = S.gather_hidden(dev_bf16(hidden), dev(term))
    assert np.array_equal(S.bf16_bits(got), ref.gather_hidden(hidden, term))


def test_bad_arguments():
    w = I.scaled(I.WORKLOADS["tiny"], B=2)
    x = I.attn_inputs(w)
    Kp, Vp, pt, pi, kl = I.paged_cache(x["Kc"], x["Vc"], x["kv_indptr"], spare_tokens=0, seed=18)
    bad = kl.copy()
    bad[0] = -1
    with pytest.raises(S.SpecrollError):
        _gpu_paged(x, Kp, Vp, pt, pi, bad)
    with pytest.raises(S.SpecrollError):
        S.tree_attn_paged(dev_bf16(x["Q"]), dev_bf16(Kp[:, :64]), dev_bf16(Vp[:, :64]), dev(pt), dev(pi), dev(kl), kl,
                          dev_bf16(x["Kt"]), dev_bf16(x["Vt"]), x["parent"])
