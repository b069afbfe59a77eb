"""GPU test of specroll_verify_static, the verification entry point for hosts that cannot allocate.

A serving process that gave all device memory to its KV-cache pool, or a C client that only
receives device pointers, has no way to provide the workspace specroll_verify asks for.  The
static variant keeps its scratch inside the library.  It must give exactly what specroll_verify
gives, also on a second call that finds the first call's leftovers in the shared scratch, and it
must refuse problems beyond its fixed limits instead of overrunning the array.

Collected last on purpose (file name), so a run that stops at the first failure has already run
every other test; it passes alone in a fresh process as well as after the rest of the suite.
"""
import numpy as np
import pytest
import torch

from oracle import ref
from paper_2608_04962_b200 import binding as S
from paper_2608_04962_b200 import inputs as I
from tests.util import dev, dev_bf16, host

pytestmark = pytest.mark.gpu

INT_KEYS = ("n_acc", "path_node", "out_tok", "term_node", "term_kind")


def _case(B, N, K, k, V, seed, boost):
    w = I.scaled(I.WORKLOADS["qwen1.5b"], B=B, N=N, K=K, k=k, V=V, cfg_id=70 + seed)
    parent = I.topology(w)
    cid, cl = I.synthetic_candidates(w)
    d = ref.tree_draw(parent, np.zeros(B, np.int32), cid, cl, I.uniforms24(seed, (B, N)))
    lg = I.target_logits(w, parent, d["tree_tok"], boost=boost)
    u_acc, u_fin = I.verify_uniforms(w)
    return (dev_bf16(lg), parent, dev(d["tree_tok"]), dev(d["tree_cand"]), dev(cid), dev(cl), dev(u_acc),
            dev(u_fin))


def _same(a, b):
    for key in INT_KEYS:                                   # integer outputs: bit-exact
        assert torch.equal(a[key], b[key]), key
    assert torch.equal(a["row_max"], b["row_max"])
    for key in ("row_sum", "min_margin"):                  # same kernels, same order: identical floats
        np.testing.assert_allclose(host(a[key]), host(b[key]), rtol=1e-6, atol=0)


def test_two_calls_in_a_row_match_the_workspace_entry_point():
    # first call: many sequences, wide candidate lists (B * k = 2400 of the 16384 candidate slots the scratch holds)
    args1 = _case(B=300, N=16, K=4, k=8, V=4096, seed=1, boost=6.0)
    want1 = S.verify(*args1)
    got1 = S.verify_static(*args1)
    torch.cuda.synchronize()
    _same(got1, want1)
    assert int(want1["n_acc"].max()) >= 1
    # second call, different shape and data: must not be disturbed by what the first one left behind
    args2 = _case(B=37, N=9, K=3, k=4, V=1024, seed=2, boost=3.0)
    got2 = S.verify_static(*args2)
    want2 = S.verify(*args2)
    torch.cuda.synchronize()
    _same(got2, want2)
    # and the first problem again, now after a smaller one
    got3 = S.verify_static(*args1)
    torch.cuda.synchronize()
    _same(got3, want1)


def test_the_largest_admitted_problem_fits_the_scratch():
    # exactly at both limits: B = 4096 sequences and B * k = 16384 candidate slots; small tree and vocabulary
    args = _case(B=4096, N=5, K=2, k=4, V=512, seed=3, boost=4.0)
    want = S.verify(*args)
    got = S.verify_static(*args)
    torch.cuda.synchronize()
    _same(got, want)
    # and a small problem right after it
    args2 = _case(B=5, N=3, K=2, k=2, V=256, seed=4, boost=3.0)
    got2 = S.verify_static(*args2)
    want2 = S.verify(*args2)
    torch.cuda.synchronize()
    _same(got2, want2)


def test_sizes_beyond_the_fixed_limit_are_refused_with_a_clear_error():
    B, N, K, k, V = 4097, 1, 1, 1, 8                        # one sequence too many
    z = lambda shape, dt: torch.zeros(shape, dtype=dt, device="cuda")
    with pytest.raises(S.SpecrollError, match="limit"):
        S.verify_static(z((B, N, V), torch.bfloat16), np.array([-1], np.int32), z((B, N), torch.int32),
                        z((B, N), torch.uint8), z((B, K, k), torch.int32), z((B, K, k), torch.float32),
                        z((B, N), torch.float32), z((B,), torch.float32))
    B, k = 1024, 32                                         # B * k = 32768 > 16384
    with pytest.raises(S.SpecrollError, match="limit"):
        S.verify_static(z((B, N, 64), torch.bfloat16), np.array([-1], np.int32), z((B, N), torch.int32),
                        z((B, N), torch.uint8), z((B, K, k), torch.int32), z((B, K, k), torch.float32),
                        z((B, N), torch.float32), z((B,), torch.float32))
