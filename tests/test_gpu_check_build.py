"""The debug build of the library (-DSPECROLL_CHECK: the kernels check the indices they read from the caller's
device arrays) gives the same results as the normal build on the tiny configuration and reports nothing; given a
candidate token id outside the vocabulary it completes, reports the sequence, and leaves the context usable.  It
also carries the one hook with which a bounded device-side wait can be made to run out (a barrier arrival left out,
nothing abandoned): the kernel gives up, returns SPECROLL_ETIMEOUT, and the next call on the same workspace is right.

No memory checker can be run on these kernels where they are developed; this build, the guard bytes around every
buffer of the GPU tests and the comparison with the oracle stand in for it.  Runs in a child process, because a
process loads one build of the library.
"""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import sys
sys.path.insert(0, %r)
import numpy as np, torch
from oracle import ref
from paper_2608_04962_b200 import binding as S, inputs as I
from tests.util import dev, dev_bf16, host
assert S.check_status()[0] == 0, "not a build with index checks"
w = I.WORKLOADS["tiny"]
x = I.propose_inputs(w, peaked=True)
g = S.propose(dev_bf16(x["h"]), dev(x["anchor"]), dev_bf16(x["A"]), dev_bf16(x["bias"]), dev_bf16(x["W"]), dev(x["m"]),
              dev(x["alpha"]), x["parent"], dev(x["u_draw"]), k=w.k, clip_c=w.clip_c)
o = ref.propose(x["h"], x["anchor"], x["A"], x["bias"], x["W"], x["m"], x["alpha"], x["parent"], x["u_draw"], k=w.k,
                clip_c=w.clip_c)
assert np.array_equal(host(g["cand_id"]), o["cand_id"]) and np.array_equal(host(g["tree_tok"]), o["tree_tok"])
a = I.attn_inputs(w)
O = S.tree_attn(dev_bf16(a["Q"]), dev_bf16(a["Kc"]), dev_bf16(a["Vc"]), dev(a["kv_indptr"]), a["kv_indptr"],
                dev_bf16(a["Kt"]), dev_bf16(a["Vt"]), a["parent"], check_status=True)
oa = ref.tree_attn(a["Q"], a["Kc"], a["Vc"], a["kv_indptr"], a["Kt"], a["Vt"], a["parent"])
assert np.abs(host(O.float()).astype(np.float64) - oa["O64"]).max() <= 1e-2
lg = I.target_logits(w, x["parent"], o["tree_tok"])
u_acc, u_fin = I.verify_uniforms(w)
args = (dev_bf16(lg), x["parent"], dev(o["tree_tok"]), dev(o["tree_cand"]), dev(o["cand_id"]), dev(o["cand_logit"]),
        dev(u_acc), dev(u_fin))
v = S.verify(*args)
ov = ref.verify(lg, x["parent"], o["tree_tok"], o["tree_cand"], o["cand_id"], o["cand_logit"], u_acc, u_fin)
for key in ("n_acc", "out_tok", "path_node"):
    assert np.array_equal(host(v[key]), ov[key]), key
assert S.check_status() == (0, 0)
# a candidate id beyond the vocabulary in sequence 2: the walk must not follow it
bad = o["cand_id"].copy()
bad[2, 0, 0] = w.V + 5
S.verify(args[0], args[1], args[2], args[3], dev(bad), *args[5:])
rc, where = S.check_status()
assert (rc, where) == (7, 2), (rc, where)
# the context is intact and the memory of the check is cleared
v2 = S.verify(*args)
assert np.array_equal(host(v2["out_tok"]), ov["out_tok"]) and S.check_status() == (0, 0)
# ---- a bounded wait that runs out: the projection kernel leaves out one barrier arrival, the warps waiting for it
#      give up after the debug build's limit, every role leaves, the kernel returns and says so in the status word
import ctypes as C
ws = torch.zeros(S.propose_workspace_bytes(w.B, w.N, w.K, w.k, w.d, w.V, clip_c=w.clip_c), dtype=torch.uint8, device="cuda")
pargs = (dev_bf16(x["h"]), dev(x["anchor"]), dev_bf16(x["A"]), dev_bf16(x["bias"]), dev_bf16(x["W"]), dev(x["m"]),
         dev(x["alpha"]), x["parent"], dev(x["u_draw"]))
assert S.lib().specroll_check_inject(C.c_int32(1)) == 0
S.propose(*pargs, k=w.k, clip_c=w.clip_c, workspace=ws)
torch.cuda.synchronize()
assert S.workspace_status(ws) == 5, S.workspace_status(ws)            # SPECROLL_ETIMEOUT
# the same workspace, the same context: a normal call right after it is complete and correct
g2 = S.propose(*pargs, k=w.k, clip_c=w.clip_c, workspace=ws)
torch.cuda.synchronize()
assert S.workspace_status(ws) == 0
assert np.array_equal(host(g2["cand_id"]), o["cand_id"]) and np.array_equal(host(g2["tree_tok"]), o["tree_tok"])
print("check build ok")
"""


def test_debug_build_matches_and_reports_a_bad_index():
    from paper_2608_04962_b200 import build as B
    lib = B.build(check=True)
    env = dict(os.environ, SPECROLL_LIB=lib)
    p = subprocess.run([sys.executable, "-c", CHILD % ROOT], env=env, capture_output=True, text=True, timeout=600)
    assert p.returncode == 0, p.stdout + p.stderr
    assert "check build ok" in p.stdout


def test_normal_build_has_no_checks():
    import ctypes as C
    from paper_2608_04962_b200 import binding as S
    assert S.check_status()[0] == -1
    assert S.lib().specroll_check_inject(C.c_int32(1)) == -1
