"""Two host threads, each with a stream of its own, call the entry points at the same time on different problems.

The library keeps a little host state behind locks (a kernel's set-up per device, attention plans per lengths,
encoded tensor maps per buffer) and none on the device besides the caller's workspaces, so calls on different
streams with different workspaces must not disturb one another: every result has to equal what the same call
gives alone.  (A stand-in for a race detector on the host side of the library; ctypes releases the
interpreter lock during a call, so the two threads really are inside the library together.)"""
import threading

import numpy as np
import pytest
import torch

from oracle import ref
from paper_2608_04962_b200 import binding as S
from paper_2608_04962_b200 import inputs as I
from tests.util import dev, dev_bf16, host

pytestmark = pytest.mark.gpu


def _problem(seed):
    wp = I.scaled(I.WORKLOADS["qwen1.5b"], B=40 + 8 * seed, K=4, k=8, d=512, V=4096 + 256 * seed, N=16, cfg_id=50 + seed)
    x = I.propose_inputs(wp, peaked=True)
    pargs = (dev_bf16(x["h"]), dev(x["anchor"]), dev_bf16(x["A"]), dev_bf16(x["bias"]), dev_bf16(x["W"]), dev(x["m"]),
             dev(x["alpha"]), x["parent"], dev(x["u_draw"]))
    wa = I.scaled(I.WORKLOADS["qwen7b"], B=3 + seed, N=32, K=4, kv_a=150 + 40 * seed, kv_b=500 + 90 * seed, cfg_id=60 + seed)
    a = I.attn_inputs(wa)
    aargs = (dev_bf16(a["Q"]), dev_bf16(a["Kc"]), dev_bf16(a["Vc"]), dev(a["kv_indptr"]), a["kv_indptr"],
             dev_bf16(a["Kt"]), dev_bf16(a["Vt"]), a["parent"])
    wv = I.scaled(I.WORKLOADS["qwen1.5b"], B=30 + 5 * seed, V=8192, cfg_id=70 + seed)
    parent = I.topology(wv)
    cid, cl = I.synthetic_candidates(wv)
    d = ref.tree_draw(parent, np.zeros(wv.B, np.int32), cid, cl, I.uniforms24(5 + seed, (wv.B, wv.N)))
    lg = I.target_logits(wv, parent, d["tree_tok"], boost=6.0)
    u_acc, u_fin = I.verify_uniforms(wv)
    vargs = (dev_bf16(lg), parent, dev(d["tree_tok"]), dev(d["tree_cand"]), dev(cid), dev(cl), dev(u_acc), dev(u_fin))
    return wp, pargs, aargs, vargs


def _run(wp, pargs, aargs, vargs, stream, rounds):
    out = []
    with torch.cuda.stream(stream):
        for _ in range(rounds):
            p = S.propose(*pargs, k=wp.k, temperature=wp.temperature, clip_c=wp.clip_c)
            O = S.tree_attn(*aargs)
            v = S.verify(*vargs)
            out.append((p, O, v))
        stream.synchronize()
    return out


def _same(a, b):
    (pa, Oa, va), (pb, Ob, vb) = a, b
    for key in ("cand_id", "cand_logit", "tree_tok", "tree_cand", "slot_q"):
        assert torch.equal(pa[key], pb[key]), key
    assert torch.equal(Oa, Ob)
    for key in ("n_acc", "path_node", "out_tok", "term_node", "term_kind", "row_max", "row_sum"):
        assert torch.equal(va[key], vb[key]), key


def test_two_threads_two_streams_do_not_disturb_each_other():
    probs = [_problem(0), _problem(1)]
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    torch.cuda.synchronize()
    alone = [_run(*probs[i], streams[i], 1)[0] for i in range(2)]     # each alone first: the reference
    results, errors = [None, None], []

    def worker(i):
        try:
            torch.cuda.set_device(0)
            results[i] = _run(*probs[i], streams[i], 6)
        except Exception as e:  # noqa: BLE001 - reported below
            errors.append(e)

    threads = [threading.Thread(target=worker, args=(i,)) for i in range(2)]
    for t in threads:
        t.start()
    for t in threads:
        t.join(timeout=120)
    assert not errors, errors
    torch.cuda.synchronize()
    for i in range(2):
        assert results[i] is not None and len(results[i]) == 6
        for r in results[i]:
            _same(r, alone[i])
