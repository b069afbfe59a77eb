"""The largest admitted tree (64 nodes, 8 heads, 64 candidates per head) through proposal, tree attention and
verification, against the oracle; and a star with 63 children of the root."""
import numpy as np
import pytest
import torch

from oracle import ref
from paper_2608_04962_b200 import binding as S
from paper_2608_04962_b200 import inputs as I
from tests.test_gpu_propose import LOGIT_ATOL, check_candidates, check_tree, gpu_propose
from tests.test_gpu_verify import check as check_verify
from tests.test_gpu_verify import run_both
from tests.util import dev, dev_bf16, host

pytestmark = pytest.mark.gpu


def test_largest_tree_through_the_three_calls():
    w = I.scaled(I.WORKLOADS["tiny"], B=5, N=64, K=8, k=64, d=256, V=4096, Hq=4, Hkv=2, D=64,
                 alpha_heads=(0.02,) * 8, kv_a=100, kv_b=400)
    # proposal (k > 8: the mma.sync projection and the general merge)
    x = I.propose_inputs(w, peaked=True)
    assert x["parent"].shape[0] == 64 and I.node_depths(x["parent"]).max() <= 8
    g = gpu_propose(w, x)
    same, oid, ol = check_candidates(w, x, g, logit_atol=LOGIT_ATOL)
    check_tree(w, x, g, same, oid=oid, ol=ol)
    # attention: 64 nodes x 2 query heads per KV head = one block of 128 rows, 64-bit ancestor masks full
    a = I.attn_inputs(w)
    oa = ref.tree_attn(a["Q"], a["Kc"], a["Vc"], a["kv_indptr"], a["Kt"], a["Vt"], a["parent"])
    O = S.tree_attn(dev_bf16(a["Q"]), dev_bf16(a["Kc"]), dev_bf16(a["Vc"]), dev(a["kv_indptr"]), a["kv_indptr"],
                    dev_bf16(a["Kt"]), dev_bf16(a["Vt"]), a["parent"], check_status=True)
    torch.cuda.synchronize()
    assert np.abs(host(O.float()).astype(np.float64) - oa["O64"]).max() <= 1e-2
    # verification on the oracle's draw from the oracle's lists
    cid, cl = I.synthetic_candidates(w)
    d = ref.tree_draw(x["parent"], np.zeros(w.B, np.int32), cid, cl, I.uniforms24(3, (w.B, w.N)))
    lg = I.target_logits(w, x["parent"], d["tree_tok"], boost=6.0)
    u_acc, u_fin = I.verify_uniforms(w)
    o, gv = run_both(w, x["parent"], lg, d["tree_tok"], d["tree_cand"], cid, cl, u_acc, u_fin)
    check_verify(w, o, gv, lg)
    # and the draw alone, exactly
    gd = S.tree_draw(x["parent"], dev(np.zeros(w.B, np.int32)), dev(cid), dev(cl), dev(I.uniforms24(3, (w.B, w.N))))
    torch.cuda.synchronize()
    assert np.array_equal(host(gd["tree_tok"]), d["tree_tok"]) and np.array_equal(host(gd["tree_cand"]), d["tree_cand"])


def test_star_of_sixty_three_children():
    star = [-1] + [0] * 63
    w = I.scaled(I.WORKLOADS["tiny"], B=6, N=64, K=1, k=64, V=2048, fixed_parent=tuple(star))
    parent = np.array(star, np.int32)
    cid, cl = I.synthetic_candidates(w)
    u = I.uniforms24(17, (w.B, w.N))
    d = ref.tree_draw(parent, np.zeros(w.B, np.int32), cid, cl, u)
    gd = S.tree_draw(parent, dev(np.zeros(w.B, np.int32)), dev(cid), dev(cl), dev(u))
    torch.cuda.synchronize()
    assert np.array_equal(host(gd["tree_tok"]), d["tree_tok"]) and np.array_equal(host(gd["tree_cand"]), d["tree_cand"])
    assert all(len(set(r[1:].tolist())) == 63 for r in d["tree_cand"])                   # 63 distinct candidates drawn
    lg = I.target_logits(w, parent, d["tree_tok"], boost=5.0)
    u_acc, u_fin = I.verify_uniforms(w)
    o, gv = run_both(w, parent, lg, d["tree_tok"], d["tree_cand"], cid, cl, u_acc, u_fin)
    check_verify(w, o, gv, lg)


def test_empty_batch_is_accepted_and_launches_nothing_wrong():
    # B = 0 (a scheduler round with no live sequence): every entry point returns without touching its outputs
    d, V, K, k, N = 128, 1024, 3, 4, 8
    z = lambda shape, dt: torch.zeros(shape, dtype=dt, device="cuda")
    parent = I.best_first_topology(N, K, k)
    p = S.propose(z((0, d), torch.bfloat16), z((0,), torch.int32), z((K, d, d), torch.bfloat16), z((K, d), torch.bfloat16),
                  z((V, d), torch.bfloat16), None, None, parent, z((0, N), torch.float32), k=k)
    assert p["cand_id"].shape == (0, K, k) and p["tree_tok"].shape == (0, N)
    t = S.tree_draw(parent, z((0,), torch.int32), z((0, K, k), torch.int32), z((0, K, k), torch.float32),
                    z((0, N), torch.float32))
    assert t["tree_tok"].shape == (0, N)
    Hq, Hkv, D = 4, 2, 64
    ip = np.zeros(1, np.int32)
    O = S.tree_attn(z((0, N, Hq, D), torch.bfloat16), z((0, Hkv, D), torch.bfloat16), z((0, Hkv, D), torch.bfloat16),
                    dev(ip), ip, z((0, N, Hkv, D), torch.bfloat16), z((0, N, Hkv, D), torch.bfloat16), parent)
    assert O.shape[0] == 0
    v = S.verify(z((0, N, V), torch.bfloat16), parent, z((0, N), torch.int32), z((0, N), torch.uint8),
                 z((0, K, k), torch.int32), z((0, K, k), torch.float32), z((0, N), torch.float32), z((0,), torch.float32))
    torch.cuda.synchronize()
    assert v["n_acc"].shape == (0,) and v["out_tok"].shape == (0, K + 1)
