"""GPU parity: observation severity, sketches and the reliability gate against the CPU oracle."""
import numpy as np
import pytest
import torch

from oracle import ref
from paper_2608_04962_b200 import binding as S
from paper_2608_04962_b200 import inputs as I
from tests.test_gpu_feedback import _case
from tests.util import dev, dev_bf16, host

pytestmark = pytest.mark.gpu


def _stats(logits, T):
    lf = I.bf16_bits_to_f32(logits).astype(np.float64)
    row_max = lf.max(-1)
    row_sum = np.exp((lf - row_max[:, None]) / np.float32(T)).sum(-1)
    return row_max.astype(np.float32), row_sum.astype(np.float32)


@pytest.mark.parametrize("R,V,d,k,kS,w_min", [(8, 4096, 256, 4, 8, 0.03), (6, 151936, 1536, 8, 48, None),
                                               (5, 2056, 3584, 8, 16, 0.0)])
def test_weighted_update_severity_and_feedback_vectors(R, V, d, k, kS, w_min):
    rows = R + 2
    W, logits, rec_row, cand_id, cand_logit, y, m, rec_mem, rho = _case(40 + R, R, V, d, k, rows)
    discards = w_min is None
    if discards:  # a threshold in the widest gap of the severities: some records are kept, some discarded
        ws = np.sort(ref.reflex_feedback(logits[rec_row], W, cand_id, cand_logit, y, m[rec_mem], rho, kS)["w"])
        i = int(np.argmax(np.diff(ws)))
        w_min = float(0.5 * (ws[i] + ws[i + 1]))
    o = ref.reflex_feedback(logits[rec_row], W, cand_id, cand_logit, y, m[rec_mem], rho, kS, severity=True,
                            severity_min=w_min)
    row_max, row_sum = _stats(logits, 1.0)
    dm = dev(m.copy())
    g = S.reflex_feedback(dev_bf16(logits), dev(rec_row), dev(row_max), dev(row_sum), dev(cand_id), dev(cand_logit),
                          dev(y), dev_bf16(W), dev(rho), dev(rec_mem), dm, kS, severity_min=w_min, want_e=True)
    torch.cuda.synchronize()
    w = host(g["severity"])
    np.testing.assert_allclose(w, o["w"], rtol=2e-4, atol=1e-6)
    # a severity within rounding of the threshold may fall on either side: such records are left out of the
    # memory comparison (none in these cases, checked)
    near = np.abs(o["w"] - w_min) < 1e-5
    assert not near.any()
    escale = np.abs(o["e"]).max()
    np.testing.assert_allclose(host(g["e"]), o["e"], rtol=1e-3, atol=2e-4 * escale)
    want = m.astype(np.float64).copy()
    want[rec_mem] = o["m"]
    got = host(dm)
    np.testing.assert_allclose(got, want, rtol=1e-3, atol=1e-4 * np.abs(want).max())
    if discards:
        assert (~o["kept"]).any() and o["kept"].any()
        for r in np.nonzero(~o["kept"])[0]:
            assert np.array_equal(got[rec_mem[r]], m[rec_mem[r]])


@pytest.mark.parametrize("R,d,rank", [(7, 1536, 24), (300, 3584, 24), (3, 40, 32), (5, 17, 1)])
def test_sketches(R, d, rank):
    g = I.rng(29)
    Pi = g.standard_normal((rank, d)).astype(np.float32)
    X = g.standard_normal((R + 4, d)).astype(np.float32)
    X[1] = 0.0
    rows = g.permutation(R + 4)[:R].astype(np.int32)
    want = ref.reflex_sketch(X[rows], Pi)
    got = host(S.reflex_sketch(dev(X), dev(Pi), rows=dev(rows)))
    np.testing.assert_allclose(got, want, rtol=0, atol=2e-5)
    got_all = host(S.reflex_sketch(dev(X), dev(Pi)))
    np.testing.assert_allclose(got_all, ref.reflex_sketch(X, Pi), rtol=0, atol=2e-5)
    assert (got_all[1] == 0).all()


@pytest.mark.parametrize("R,S_,rank,d,use_keep", [(500, 37, 24, 1536, True), (64, 5, 24, 96, False), (0, 4, 24, 32, False),
                                                   (1000, 1, 8, 64, True)])
def test_gate(R, S_, rank, d, use_keep):
    g = I.rng(100 + R)
    s = g.standard_normal((R, rank)).astype(np.float32)
    xi = (0.7 * s + g.standard_normal((R, rank))).astype(np.float32)
    if R > 3:
        xi[3] = 0.0
    slot = g.integers(0, S_, size=R).astype(np.int32)
    keep = (g.random(R) > 0.25) if use_keep else None
    H = 3
    horizon = (np.arange(S_) % H).astype(np.int32)
    m = g.standard_normal((S_, d)).astype(np.float32)
    if S_ > 2:
        m[2] = 0.0
    # the slots start from an earlier state
    n0 = g.integers(0, 5, size=S_).astype(np.int32)
    mean0 = (0.2 * g.standard_normal(S_)).astype(np.float32)
    M20 = (0.1 * g.random(S_) * np.maximum(n0 - 1, 0)).astype(np.float32)
    nfb0 = n0.copy()
    n_align = np.array([6, 16, 48], np.int32)
    n_fb = np.array([1, 2, 4], np.int32)
    lo = np.array([0.010, 0.004, 0.0025], np.float32)
    hi = np.array([0.025, 0.010, 0.0060], np.float32)
    o = ref.reflex_gate(s, xi, slot, keep, n0, mean0, M20, nfb0, m, horizon, n_align, n_fb, lo, hi, z_delta=0.6)
    dn, dmean, dM2, dnfb = dev(n0.copy()), dev(mean0.copy()), dev(M20.copy()), dev(nfb0.copy())
    out = S.reflex_gate(dev(s), dev(xi), dev(slot), dev(keep.astype(np.uint8)) if use_keep else None, dn, dmean, dM2, dnfb,
                        dev(m), dev(horizon), dev(n_align), dev(n_fb), dev(lo), dev(hi), z_delta=0.6)
    torch.cuda.synchronize()
    assert np.array_equal(host(dn), o["n"]) and np.array_equal(host(dnfb), o["n_fb"])
    a = host(out["a"])
    kept = np.ones(R, bool) if keep is None else keep
    np.testing.assert_allclose(a[kept], o["a"][kept], rtol=0, atol=2e-6)
    assert np.isnan(a[~kept]).all()
    np.testing.assert_allclose(host(dmean), o["mean"], rtol=0, atol=2e-5)
    np.testing.assert_allclose(host(dM2), o["M2"], rtol=2e-4, atol=2e-5)
    rel, want_rel = host(out["rel"]), o["rel"]
    fin = np.isfinite(want_rel)
    assert np.array_equal(np.isneginf(rel), ~fin)
    np.testing.assert_allclose(rel[fin], want_rel[fin], rtol=0, atol=5e-5)
    # the gate is a comparison of the score with zero: slots whose score is within rounding of zero may differ
    sure = ~fin | (np.abs(want_rel) > 1e-4)
    np.testing.assert_allclose(host(out["alpha"])[sure], o["alpha"][sure], rtol=1e-4, atol=1e-7)
    if S_ > 2:
        assert host(out["alpha"])[2] == 0.0  # an empty memory row never opens the gate
    if R >= 500 and S_ > 10:
        assert (o["alpha"] > 0).any() and (o["alpha"] == 0).any()
