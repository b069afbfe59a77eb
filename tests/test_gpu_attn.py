"""GPU parity: specroll_tree_attn against the CPU oracle on identical seeded inputs."""
import numpy as np
import pytest
import torch

from oracle import ref
from paper_2608_04962_b200 import binding as S
from paper_2608_04962_b200 import inputs as I
from tests.util import dev, dev_bf16, host

pytestmark = pytest.mark.gpu

O_ATOL = 1e-2          # max abs error of the attention output (bf16 inputs, fp32 accumulate)
FLAGS = {"v": 0}       # 0: tcgen05 kernel, 1: legacy mma.sync kernel


@pytest.fixture(params=[0, 1], ids=["tcgen05", "mma"], autouse=True)
def _both_kernels(request):
    FLAGS["v"] = request.param
    yield
    FLAGS["v"] = 0


def run_both(w, x, lengths=None):
    if lengths is not None:
        lengths = np.asarray(lengths, np.int32)
        ip = np.zeros(w.B + 1, np.int32)
        np.cumsum(lengths, out=ip[1:])
        g = I.rng(4242)
        x = dict(x)
        x["kv_indptr"] = ip
        x["Kc"] = I.f32_to_bf16_bits(g.standard_normal((int(ip[-1]), w.Hkv, w.D), dtype=np.float32))
        x["Vc"] = I.f32_to_bf16_bits(g.standard_normal((int(ip[-1]), w.Hkv, w.D), dtype=np.float32))
    o = ref.tree_attn(x["Q"], x["Kc"], x["Vc"], x["kv_indptr"], x["Kt"], x["Vt"], x["parent"], want_lse=True)
    O, lse = S.tree_attn(dev_bf16(x["Q"]), dev_bf16(x["Kc"]), dev_bf16(x["Vc"]), dev(x["kv_indptr"]),
                         x["kv_indptr"], dev_bf16(x["Kt"]), dev_bf16(x["Vt"]), x["parent"], want_lse=True,
                         flags=FLAGS["v"], check_status=True)
    torch.cuda.synchronize()
    return o, host(O.float()).astype(np.float64), host(lse).astype(np.float64)


def check(o, O, lse, edge=False):
    """edge=False: the bar of the workloads everywhere: max abs <= 1e-2.
    edge=True: the same bar for every element with |O| <= 1.  Where the softmax is concentrated on a few tokens
    (degenerate caches of 0 or 1 tokens, scores that grow along the cache) |O| reaches several units and the
    spacing of the bf16 output alone (2^-8 |O|) exceeds 1e-2; those elements, and only those, get the bound
    scaled by |O|, and must in addition lie within one bf16 step of the oracle's rounded value."""
    o64 = o["O64"]
    diff = np.abs(O - o64)
    big = (np.abs(o64) > 1.0) & edge
    assert (diff[~big] <= O_ATOL).all(), diff[~big].max()
    if big.any():
        assert (diff[big] <= O_ATOL * np.abs(o64[big])).all(), (diff[big] / np.abs(o64[big])).max()
        step = 2.0 ** (np.floor(np.log2(np.abs(o64[big]))) - 7)
        rounded = I.bf16_bits_to_f32(I.f32_to_bf16_bits(o64[big].astype(np.float32))).astype(np.float64)
        assert (np.abs(O[big] - rounded) <= step).all()
    err = diff.max()
    np.testing.assert_allclose(lse, o["lse"], atol=2e-3, rtol=0)
    return err


def test_tiny_config():
    w = I.WORKLOADS["tiny"]
    o, O, lse = run_both(w, I.attn_inputs(w))
    check(o, O, lse)


@pytest.mark.parametrize("Hq,Hkv,D,N", [(12, 2, 128, 16), (28, 4, 128, 32), (40, 8, 128, 48), (10, 2, 64, 13),
                                        (28, 4, 128, 64), (4, 4, 128, 1), (14, 2, 64, 37), (14, 2, 64, 30)])
def test_group_sizes_head_dims_and_tree_sizes(Hq, Hkv, D, N):
    # G = 6, 7, 5, 5, 7, 1, 7, 7; rows = 96, 224, 240, 65, 448, 1, 259, 210 (one to four row blocks: the softmax
    # with two threads per row for one block, the two alternating teams for more)
    K = 5
    w = I.scaled(I.WORKLOADS["qwen7b"], B=5, N=N, K=K, Hq=Hq, Hkv=Hkv, D=D, kv_a=300, kv_b=900)
    x = I.attn_inputs(w)
    o, O, lse = run_both(w, x, lengths=[700, 64, 1, 333, 129])
    check(o, O, lse, edge=True)
    o, O, lse = run_both(w, x, lengths=[700, 64, 70, 333, 129])
    check(o, O, lse)


def test_ragged_lengths_empty_cache_and_split_kv():
    # one long sequence forces several chunks per sequence; zero-length and sub-tile caches ride along
    w = I.scaled(I.WORKLOADS["qwen1.5b"], B=7, N=16)
    x = I.attn_inputs(w)
    o, O, lse = run_both(w, x, lengths=[0, 5000, 63, 64, 65, 2049, 777])
    check(o, O, lse, edge=True)
    # the same data with everything short: single-chunk direct-write path
    o2, O2, lse2 = run_both(w, x, lengths=[0, 17, 63, 64, 65, 100, 1])
    check(o2, O2, lse2, edge=True)
    o3, O3, lse3 = run_both(w, x, lengths=[64, 5000, 80, 64, 65, 2049, 777])
    check(o3, O3, lse3)


@pytest.mark.parametrize("Hq,Hkv,D,N", [(10, 2, 64, 13), (14, 2, 64, 30), (12, 2, 128, 16), (28, 4, 128, 32),
                                        (14, 2, 128, 37)])
def test_sequences_cut_into_many_chunks(Hq, Hkv, D, N):
    # one sequence of 5000 tokens among short ones: ten chunks, merged by the kernel that runs after the
    # attention kernel (one, two and three row blocks, both head dims); next to it a sequence cut in two,
    # which the attention kernel merges itself only when no sequence has five chunks or more
    w = I.scaled(I.WORKLOADS["qwen7b"], B=4, N=N, K=5, Hq=Hq, Hkv=Hkv, D=D, kv_a=300, kv_b=900)
    x = I.attn_inputs(w)
    o, O, lse = run_both(w, x, lengths=[5000, 64, 700, 129])
    check(o, O, lse)


def test_reduced_batches_of_the_large_configs():
    for name, B in (("qwen1.5b", 12), ("qwen7b", 4), ("qwen14b", 2)):
        w = I.scaled(I.WORKLOADS[name], B=B)
        o, O, lse = run_both(w, I.attn_inputs(w))
        check(o, O, lse)


@pytest.mark.parametrize("Hq,Hkv,D,N", [(12, 2, 128, 16), (28, 4, 128, 32), (14, 2, 64, 37)])
def test_scores_that_keep_growing_along_the_cache(Hq, Hkv, D, N):
    # Keys whose magnitude grows 30-fold along the sequence: the row maxima keep rising from tile to tile by far
    # more than the 2^8 the kernel tolerates before it moves a row's reference, so the alarm, the second pass, the
    # rescaling of the accumulator and (with several row blocks) the hand-over of the reference between the two
    # softmax teams all run many times per sequence; the chunks of the split sequences meet very different maxima.
    w = I.scaled(I.WORKLOADS["qwen7b"], B=4, N=N, K=5, Hq=Hq, Hkv=Hkv, D=D, kv_a=300, kv_b=900)
    x = dict(I.attn_inputs(w))
    lengths = np.asarray([2300, 640, 131, 1500], np.int32)
    ip = np.zeros(w.B + 1, np.int32)
    np.cumsum(lengths, out=ip[1:])
    g = I.rng(777)
    Kc = g.standard_normal((int(ip[-1]), w.Hkv, w.D), dtype=np.float32)
    for b in range(w.B):
        ramp = 1.0 + 30.0 * np.arange(lengths[b], dtype=np.float32) / lengths[b]
        Kc[ip[b]:ip[b + 1]] *= ramp[:, None, None]
    x["kv_indptr"] = ip
    x["Kc"] = I.f32_to_bf16_bits(Kc)
    x["Vc"] = I.f32_to_bf16_bits(g.standard_normal((int(ip[-1]), w.Hkv, w.D), dtype=np.float32))
    o = ref.tree_attn(x["Q"], x["Kc"], x["Vc"], x["kv_indptr"], x["Kt"], x["Vt"], x["parent"], want_lse=True)
    O, lse = S.tree_attn(dev_bf16(x["Q"]), dev_bf16(x["Kc"]), dev_bf16(x["Vc"]), dev(x["kv_indptr"]), x["kv_indptr"],
                         dev_bf16(x["Kt"]), dev_bf16(x["Vt"]), x["parent"], want_lse=True, flags=FLAGS["v"],
                         check_status=True)
    torch.cuda.synchronize()
    # sharply peaked rows have |O| of a few units (one value row dominates): the bound scales with max(1, |O|)
    check(o, host(O.float()).astype(np.float64), host(lse).astype(np.float64), edge=True)


def test_scale_argument_and_topology_errors():
    w = I.scaled(I.WORKLOADS["tiny"], B=2)
    x = I.attn_inputs(w)
    args = (dev_bf16(x["Q"]), dev_bf16(x["Kc"]), dev_bf16(x["Vc"]), dev(x["kv_indptr"]), x["kv_indptr"],
            dev_bf16(x["Kt"]), dev_bf16(x["Vt"]))
    O = S.tree_attn(*args, x["parent"], scale=0.05)
    want = ref.tree_attn(x["Q"], x["Kc"], x["Vc"], x["kv_indptr"], x["Kt"], x["Vt"], x["parent"], scale=0.05)
    assert np.abs(host(O.float()) - want["O64"]).max() <= O_ATOL
    bad = x["parent"].copy()
    bad[2] = 2
    with pytest.raises(S.SpecrollError):
        S.tree_attn(*args, bad)


def test_layers_back_to_back_with_early_cache_loads():
    # the layers of a step launched without a pause, every cache written beforehand: layers after the first
    # may start loading their cache while the layer before is still finishing; each must match the oracle
    if FLAGS["v"] != 0:
        pytest.skip("a feature of the tcgen05 kernel")
    w = I.scaled(I.WORKLOADS["qwen7b"], B=9, N=32)
    lengths = np.array([2100, 64, 700, 129, 3300, 1, 0, 257, 1500], np.int32)
    ip = np.zeros(w.B + 1, np.int32)
    np.cumsum(lengths, out=ip[1:])
    layers, want, args = 6, [], []
    for layer in range(layers):
        x = I.attn_inputs(w, layer=layer)
        g = I.rng(950 + layer)
        Kc = I.f32_to_bf16_bits(g.standard_normal((int(ip[-1]), w.Hkv, w.D), dtype=np.float32))
        Vc = I.f32_to_bf16_bits(g.standard_normal((int(ip[-1]), w.Hkv, w.D), dtype=np.float32))
        want.append(ref.tree_attn(x["Q"], Kc, Vc, ip, x["Kt"], x["Vt"], x["parent"])["O64"])
        args.append((dev_bf16(x["Q"]), dev_bf16(Kc), dev_bf16(Vc), dev(ip), ip, dev_bf16(x["Kt"]), dev_bf16(x["Vt"]),
                     x["parent"]))
    ws = torch.empty(S.tree_attn_workspace_bytes(w.B, w.N, w.Hq, w.Hkv, w.D, ip), dtype=torch.uint8, device="cuda")
    torch.cuda.synchronize()
    for rep in range(3):
        outs = [S.tree_attn(*args[layer], workspace=ws,
                            flags=(S.ATTN_REUSE_PLAN | S.ATTN_CACHE_SETTLED) if layer > 0 else 0)
                for layer in range(layers)]
        torch.cuda.synchronize()
        for layer in range(layers):
            diff = np.abs(host(outs[layer].float()) - want[layer])
            assert (diff <= O_ATOL * np.maximum(1.0, np.abs(want[layer]))).all(), (rep, layer, diff.max())


@pytest.mark.parametrize("seed", [11, 12])
def test_random_shapes_and_lengths(seed):
    # seeded random head counts, group sizes, head dimensions, tree sizes, batch sizes and length mixes
    # (empty caches, a few long sequences among short ones), two layers launched back to back each
    if FLAGS["v"] != 0:
        pytest.skip("the legacy kernel has its own cases")
    rs = np.random.RandomState(seed)
    for case in range(6):
        Hkv = int(rs.choice([1, 2, 4, 8]))
        G = int(rs.choice([1, 2, 4, 5, 6, 7]))
        D = int(rs.choice([64, 128]))
        N = int(rs.choice([1, 2, 5, 8, 16, 24, 32, 48, 64]))
        B = int(rs.choice([1, 2, 3, 7, 12]))
        base = I.WORKLOADS["qwen7b"]
        w = I.scaled(base, B=B, N=N, Hq=Hkv * G, Hkv=Hkv, D=D, K=min(base.K, max(1, N - 1)))
        if rs.randint(2):
            lengths = rs.randint(0, 600, size=B)
        else:
            lengths = np.where(rs.rand(B) < 0.3, rs.randint(1500, 4000, size=B), rs.randint(0, 200, size=B))
        lengths = lengths.astype(np.int32)
        ip = np.zeros(B + 1, np.int32)
        np.cumsum(lengths, out=ip[1:])
        want, args = [], []
        for layer in range(2):
            x = I.attn_inputs(w, layer=layer)
            g = I.rng(7000 + 100 * seed + 13 * case + layer)
            T = max(int(ip[-1]), 1)
            Kc = I.f32_to_bf16_bits(g.standard_normal((T, Hkv, D), dtype=np.float32))[:int(ip[-1])]
            Vc = I.f32_to_bf16_bits(g.standard_normal((T, Hkv, D), dtype=np.float32))[:int(ip[-1])]
            want.append(ref.tree_attn(x["Q"], Kc, Vc, ip, x["Kt"], x["Vt"], x["parent"])["O64"])
            args.append((dev_bf16(x["Q"]), dev_bf16(Kc), dev_bf16(Vc), dev(ip), ip, dev_bf16(x["Kt"]),
                         dev_bf16(x["Vt"]), x["parent"]))
        ws = torch.empty(S.tree_attn_workspace_bytes(B, N, Hkv * G, Hkv, D, ip), dtype=torch.uint8, device="cuda")
        torch.cuda.synchronize()
        outs = [S.tree_attn(*args[layer], workspace=ws,
                            flags=(S.ATTN_REUSE_PLAN | S.ATTN_CACHE_SETTLED) if layer > 0 else 0)
                for layer in range(2)]
        torch.cuda.synchronize()
        assert S.workspace_status(ws) == 0
        for layer in range(2):
            diff = np.abs(host(outs[layer].float()) - want[layer])
            assert (diff <= O_ATOL * np.maximum(1.0, np.abs(want[layer]))).all(), \
                (case, dict(B=B, N=N, Hkv=Hkv, G=G, D=D), layer, diff.max(), lengths.tolist())


def test_plan_reuse_across_layers():
    # second call keeps the first call's work plan (same KV lengths, different tensors), as the layers of a
    # step do; results must still match the oracle, also for a third call
    if FLAGS["v"] != 0:
        pytest.skip("plan reuse is a feature of the tcgen05 kernel")
    w = I.scaled(I.WORKLOADS["qwen7b"], B=6, N=32)
    lengths = np.array([3000, 64, 700, 129, 5000, 1], np.int32)
    ip = np.zeros(w.B + 1, np.int32)
    np.cumsum(lengths, out=ip[1:])
    ws = None
    for layer in range(3):
        x = I.attn_inputs(w, layer=layer)
        g = I.rng(900 + layer)
        Kc = I.f32_to_bf16_bits(g.standard_normal((int(ip[-1]), w.Hkv, w.D), dtype=np.float32))
        Vc = I.f32_to_bf16_bits(g.standard_normal((int(ip[-1]), w.Hkv, w.D), dtype=np.float32))
        o = ref.tree_attn(x["Q"], Kc, Vc, ip, x["Kt"], x["Vt"], x["parent"])
        if ws is None:
            ws = torch.empty(S.tree_attn_workspace_bytes(w.B, w.N, w.Hq, w.Hkv, w.D, ip), dtype=torch.uint8, device="cuda")
        O = S.tree_attn(dev_bf16(x["Q"]), dev_bf16(Kc), dev_bf16(Vc), dev(ip), ip, dev_bf16(x["Kt"]), dev_bf16(x["Vt"]),
                        x["parent"], workspace=ws, flags=S.ATTN_REUSE_PLAN if layer > 0 else 0, check_status=True)
        diff = np.abs(host(O.float()) - o["O64"])
        assert (diff <= O_ATOL * np.maximum(1.0, np.abs(o["O64"]))).all(), (layer, diff.max())
