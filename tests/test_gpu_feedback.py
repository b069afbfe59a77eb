"""GPU parity: specroll_reflex_feedback against the CPU oracle on identical seeded inputs."""
import numpy as np
import pytest
import torch

from oracle import ref
from paper_2608_04962_b200 import binding as S
from paper_2608_04962_b200 import inputs as I
from tests.util import dev, dev_bf16, host

pytestmark = pytest.mark.gpu


def _case(seed, R, V, d, k, rows, spread=1.0, boost=6.0):
    g = I.rng(seed)
    W = I.f32_to_bf16_bits((0.05 * g.standard_normal((V, d))).astype(np.float32))
    lg = spread * g.standard_normal((rows, V))
    rec_row = g.permutation(rows)[:R].astype(np.int32)
    head = g.standard_normal((R, V))
    order = np.argsort(-head, axis=-1)[:, :k]
    cand_id = order.astype(np.int32)
    cand_logit = np.take_along_axis(head, order, -1).astype(np.float32)
    # the target likes some of the candidates and some tokens the head missed
    for r in range(R):
        lg[rec_row[r], cand_id[r, : k // 2]] += boost * g.random(k // 2)
        lg[rec_row[r], g.integers(0, V, 3)] += boost
    logits = I.f32_to_bf16_bits(lg.astype(np.float32))
    y = g.integers(0, V, size=R).astype(np.int32)
    m = g.standard_normal((R + 2, d)).astype(np.float32)
    rec_mem = g.permutation(R + 2)[:R].astype(np.int32)
    rho = g.choice(np.array([0.85, 0.9, 0.95], np.float32), size=R)
    return W, logits, rec_row, cand_id, cand_logit, y, m, rec_mem, rho


@pytest.mark.parametrize("R,V,d,k,kS,T", [(6, 4096, 256, 4, 8, 1.0), (5, 151936, 1536, 8, 48, 1.0),
                                          (3, 2056, 3584, 8, 16, 0.7), (4, 1024, 96, 2, 2, 1.3)])
def test_feedback_matches_the_oracle(R, V, d, k, kS, T):
    rows = R + 3
    W, logits, rec_row, cand_id, cand_logit, y, m, rec_mem, rho = _case(11 + R, R, V, d, k, rows)
    o = ref.reflex_feedback(logits[rec_row], W, cand_id, cand_logit, y, m[rec_mem], rho, kS, temperature=T)
    # row statistics as specroll_verify leaves them (plain fp64 here: they are inputs of this call)
    lf = I.bf16_bits_to_f32(logits).astype(np.float64)
    row_max = lf.max(-1)
    row_sum = np.exp((lf - row_max[:, None]) / np.float32(T)).sum(-1)
    dm = dev(m.copy())
    g = S.reflex_feedback(dev_bf16(logits), dev(rec_row), dev(row_max.astype(np.float32)), dev(row_sum.astype(np.float32)),
                          dev(cand_id), dev(cand_logit), dev(y), dev_bf16(W), dev(rho), dev(rec_mem), dm, kS,
                          temperature=T)
    torch.cuda.synchronize()
    np.testing.assert_allclose(host(g["d_dist"]), o["d_dist"], rtol=2e-4, atol=1e-6)
    np.testing.assert_allclose(host(g["d_cov"]), o["d_cov"], rtol=2e-4, atol=1e-6)
    np.testing.assert_allclose(host(g["tv"]), o["tv"], rtol=2e-4, atol=1e-6)
    got = host(dm)
    want = m.astype(np.float64).copy()
    want[rec_mem] = o["m"]
    scale = np.abs(want).max()
    np.testing.assert_allclose(got, want, rtol=1e-3, atol=1e-4 * scale)
    untouched = np.setdiff1d(np.arange(m.shape[0]), rec_mem)
    assert np.array_equal(got[untouched], m[untouched])


def test_ties_in_the_target_top_set_follow_the_id_order():
    # many equal logits around the cut of the top set: the lower ids win, as in the oracle
    R, V, d, k, kS = 2, 1024, 64, 4, 8
    W, logits, rec_row, cand_id, cand_logit, y, m, rec_mem, rho = _case(31, R, V, d, k, R)
    lf = np.zeros((R, V), np.float32)
    lf[:, ::7] = 2.0                      # 147 tokens share the maximum
    lf[0, 500] = 3.0
    logits = I.f32_to_bf16_bits(lf)
    rec_row = np.arange(R, dtype=np.int32)
    o = ref.reflex_feedback(logits, W, cand_id, cand_logit, y, m[rec_mem], rho, kS)
    row_max = lf.max(-1).astype(np.float32)
    row_sum = np.exp(lf.astype(np.float64) - row_max[:, None]).sum(-1).astype(np.float32)
    dm = dev(m.copy())
    g = S.reflex_feedback(dev_bf16(logits), dev(rec_row), dev(row_max), dev(row_sum), dev(cand_id), dev(cand_logit),
                          dev(y), dev_bf16(W), dev(rho), dev(rec_mem), dm, kS)
    np.testing.assert_allclose(host(g["d_cov"]), o["d_cov"], rtol=2e-4, atol=1e-6)
    want = m.astype(np.float64).copy()
    want[rec_mem] = o["m"]
    np.testing.assert_allclose(host(dm), want, rtol=1e-3, atol=1e-4 * np.abs(want).max())


def test_bad_arguments():
    W, logits, rec_row, cand_id, cand_logit, y, m, rec_mem, rho = _case(41, 2, 512, 64, 4, 4)
    args = (dev_bf16(logits), dev(rec_row), dev(np.zeros(4, np.float32)), dev(np.ones(4, np.float32)), dev(cand_id),
            dev(cand_logit), dev(y), dev_bf16(W), dev(rho), dev(rec_mem), dev(m))
    with pytest.raises(S.SpecrollError):
        S.reflex_feedback(*args, 2)            # support smaller than k
    with pytest.raises(S.SpecrollError):
        S.reflex_feedback(*args, 128)          # above the limit


def test_thousands_of_equal_maxima_take_the_exact_fallback():
    # more equal large values than the candidate list of the two-pass method holds: the radix search takes over,
    # and the lowest ids win the ties, as in the oracle
    R, V, d, k, kS = 2, 8192, 64, 4, 16
    W, logits, rec_row, cand_id, cand_logit, y, m, rec_mem, rho = _case(33, R, V, d, k, R)
    lf = np.full((R, V), -1.0, np.float32)
    lf[:, 1::2] = 1.5                     # 4096 tokens share the maximum
    lf[1, 4000] = 2.5
    logits = I.f32_to_bf16_bits(lf)
    rec_row = np.arange(R, dtype=np.int32)
    o = ref.reflex_feedback(logits, W, cand_id, cand_logit, y, m[rec_mem], rho, kS)
    row_max = lf.max(-1).astype(np.float32)
    row_sum = np.exp(lf.astype(np.float64) - row_max[:, None]).sum(-1).astype(np.float32)
    dm = dev(m.copy())
    g = S.reflex_feedback(dev_bf16(logits), dev(rec_row), dev(row_max), dev(row_sum), dev(cand_id), dev(cand_logit),
                          dev(y), dev_bf16(W), dev(rho), dev(rec_mem), dm, kS)
    np.testing.assert_allclose(host(g["d_cov"]), o["d_cov"], rtol=2e-4, atol=1e-6)
    np.testing.assert_allclose(host(g["d_dist"]), o["d_dist"], rtol=2e-4, atol=1e-6)
    want = m.astype(np.float64).copy()
    want[rec_mem] = o["m"]
    np.testing.assert_allclose(host(dm), want, rtol=1e-3, atol=1e-4 * np.abs(want).max())

