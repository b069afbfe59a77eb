"""The library's per-device set-up (a kernel's shared-memory limit, the SM count) is looked up per (kernel, device)
the first time a kernel runs on a device and found again afterwards: calls keep working across changes of the
current device.  (One GPU here, so the device is set to itself; the table is keyed by device all the same.)"""
import numpy as np
import pytest
import torch

from oracle import ref
from paper_2608_04962_b200 import binding as S
from paper_2608_04962_b200 import inputs as I
from tests.util import dev, dev_bf16, host

pytestmark = pytest.mark.gpu


def test_calls_across_device_round_trips():
    w = I.scaled(I.WORKLOADS["qwen7b"], B=3, N=32, K=4, kv_a=200, kv_b=600)
    a = I.attn_inputs(w)
    oa = ref.tree_attn(a["Q"], a["Kc"], a["Vc"], a["kv_indptr"], a["Kt"], a["Vt"], a["parent"])
    targs = (dev_bf16(a["Q"]), dev_bf16(a["Kc"]), dev_bf16(a["Vc"]), dev(a["kv_indptr"]), a["kv_indptr"],
             dev_bf16(a["Kt"]), dev_bf16(a["Vt"]), a["parent"])
    wv = I.scaled(I.WORKLOADS["qwen1.5b"], B=6, V=4096)
    parent = I.topology(wv)
    cid, cl = I.synthetic_candidates(wv)
    d = ref.tree_draw(parent, np.zeros(wv.B, np.int32), cid, cl, I.uniforms24(5, (wv.B, wv.N)))
    lg = I.target_logits(wv, parent, d["tree_tok"])
    u_acc, u_fin = I.verify_uniforms(wv)
    vargs = (dev_bf16(lg), parent, dev(d["tree_tok"]), dev(d["tree_cand"]), dev(cid), dev(cl), dev(u_acc), dev(u_fin))
    first = None
    for _ in range(3):
        torch.cuda.set_device(0)
        O = S.tree_attn(*targs, check_status=True)
        assert np.abs(host(O.float()).astype(np.float64) - oa["O64"]).max() <= 1e-2
        torch.cuda.set_device(torch.device("cuda", 0))
        v = S.verify_nucleus(*vargs, 0.9)
        torch.cuda.synchronize()
        toks = host(v["out_tok"])
        if first is None:
            first = toks
        assert np.array_equal(toks, first)
