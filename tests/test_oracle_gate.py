"""Pins for the oracle's observation severity, sketches and reliability gate."""
import numpy as np

from oracle import ref
from paper_2608_04962_b200 import inputs as I
from tests.test_oracle_feedback import _bits, _case, _f


def test_severity_against_its_definition_and_the_discard_rule():
    W, logits, cand_id, cand_logit, y, m, rho = _case(21, R=3)
    plain = ref.reflex_feedback(logits, W, cand_id, cand_logit, y, m, rho, k_support=6)
    sev = ref.reflex_feedback(logits, W, cand_id, cand_logit, y, m, rho, k_support=6, severity=True, severity_min=0.03)
    for r in range(3):
        l = _f(logits[r])
        p = np.exp(l - l.max())
        p /= p.sum()
        S = plain["support"][r]
        pS = p[S] / p[S].sum()
        q = np.exp(cand_logit[r].astype(np.float64) - cand_logit[r].max())
        q /= q.sum()
        qS = np.zeros(len(S))
        for j, c in enumerate(cand_id[r]):
            qS[S.index(int(c))] += q[j]
        tv = 0.5 * np.abs(pS - qS).sum()
        w = np.clip(0.3 * tv + 0.7 * (1.0 - p[cand_id[r]].sum()), 0.0, 1.0)
        assert abs(sev["w"][r] - w) < 1e-12 and abs(sev["tv_S"][r] - tv) < 1e-12
        assert 0.0 <= w <= 1.0
        # the weighted update is the plain one with e scaled by w
        np.testing.assert_allclose(sev["m"][r], rho[r] * m[r] + (1 - rho[r]) * w * plain["e"][r], rtol=0, atol=1e-12)
    # a threshold above every severity discards everything: the memory keeps its value
    none = ref.reflex_feedback(logits, W, cand_id, cand_logit, y, m, rho, k_support=6, severity=True, severity_min=2.0)
    assert not none["kept"].any()
    np.testing.assert_array_equal(none["m"], m.astype(np.float64))


def test_severity_of_a_perfect_proposal_is_the_uncovered_mass_alone():
    # q equal to p restricted to the candidates and S = C: TV(p_S, q_S) = 0, so w = 0.7 (1 - p(C))
    g = I.rng(5)
    V, d, k = 24, 6, 4
    W = _bits(g.standard_normal((V, d)))
    l = _f(_bits(2.0 * g.standard_normal(V)))
    order = np.argsort(-l)[:k]
    out = ref.reflex_feedback(_bits(l)[None], W, order[None].astype(np.int32), l[order][None].astype(np.float32),
                              np.array([order[0]], np.int32), np.zeros((1, d), np.float32), np.array([0.9]), k_support=k)
    p = np.exp(l - l.max())
    p /= p.sum()
    assert out["tv_S"][0] < 1e-7
    assert abs(out["w"][0] - 0.7 * (1.0 - p[order].sum())) < 1e-7


def test_sketch_is_a_unit_vector_invariant_to_scale_and_exact_for_a_coordinate_projection():
    g = I.rng(29)
    d, rank = 40, 24
    Pi = g.standard_normal((rank, d))
    X = g.standard_normal((5, d))
    sk = ref.reflex_sketch(X, Pi)
    np.testing.assert_allclose(np.sqrt((sk ** 2).sum(-1)), 1.0, atol=1e-12)
    np.testing.assert_allclose(ref.reflex_sketch(7.5 * X, Pi), sk, atol=1e-12)
    np.testing.assert_allclose(ref.reflex_sketch(-X, Pi), -sk, atol=1e-12)
    assert (ref.reflex_sketch(np.zeros((1, d)), Pi) == 0).all()
    # rows of the identity: the sketch is the normalised leading coordinates
    E = np.eye(rank, d)
    np.testing.assert_allclose(ref.reflex_sketch(X, E), X[:, :rank] / np.linalg.norm(X[:, :rank], axis=-1, keepdims=True),
                               atol=1e-12)
    # a Gaussian projection keeps angles approximately (Johnson-Lindenstrauss): same vector -> cosine 1
    assert abs(np.dot(sk[0], ref.reflex_sketch(X[:1] * 3, Pi)[0]) - 1.0) < 1e-12


def _gate_case(seed, R=40, S=5, rank=24, d=16):
    g = I.rng(seed)
    s = g.standard_normal((R, rank))
    xi = 0.6 * s + g.standard_normal((R, rank))   # positively aligned on average
    slot = g.integers(0, S, size=R).astype(np.int32)
    keep = g.random(R) > 0.2
    horizon = (np.arange(S) % 3).astype(np.int32)
    m = g.standard_normal((S, d))
    return s, xi, slot, keep, horizon, m


def test_online_moments_equal_the_batch_sample_moments():
    s, xi, slot, keep, horizon, m = _gate_case(7)
    S = m.shape[0]
    out = ref.reflex_gate(s, xi, slot, keep, np.zeros(S, int), np.zeros(S), np.zeros(S), np.zeros(S, int), m, horizon,
                          [1, 1, 1], [1, 1, 1], [0.01, 0.004, 0.0025], [0.025, 0.01, 0.006])
    cos = (s * xi).sum(-1) / np.linalg.norm(s, axis=-1) / np.linalg.norm(xi, axis=-1)
    for j in range(S):
        sel = keep & (slot == j)
        a = cos[sel]
        assert out["n"][j] == a.size == out["n_fb"][j]
        np.testing.assert_allclose(out["a"][sel], a, atol=1e-12)
        if a.size:
            assert abs(out["mean"][j] - a.mean()) < 1e-12
        if a.size >= 2:
            assert abs(out["M2"][j] / (a.size - 1) - a.var(ddof=1)) < 1e-12
            rel = a.mean() - 0.6 * a.std(ddof=1) / np.sqrt(a.size)
            assert abs(out["rel"][j] - rel) < 1e-12
    assert np.isnan(out["a"][~keep]).all()
    # the update can be split over two calls without changing the result (it is online)
    h = 17
    first = ref.reflex_gate(s[:h], xi[:h], slot[:h], keep[:h], np.zeros(S, int), np.zeros(S), np.zeros(S), np.zeros(S, int),
                            m, horizon, [1, 1, 1], [1, 1, 1], [0.01, 0.004, 0.0025], [0.025, 0.01, 0.006])
    second = ref.reflex_gate(s[h:], xi[h:], slot[h:], keep[h:], first["n"], first["mean"], first["M2"], first["n_fb"], m,
                             horizon, [1, 1, 1], [1, 1, 1], [0.01, 0.004, 0.0025], [0.025, 0.01, 0.006])
    np.testing.assert_allclose(second["mean"], out["mean"], atol=1e-12)
    np.testing.assert_allclose(second["M2"], out["M2"], atol=1e-12)
    np.testing.assert_array_equal(second["n"], out["n"])


def test_score_of_a_worked_example_and_the_gate_conditions():
    # three alignments 0.5, 0.7, 0.9: mean 0.7, sample std 0.2, Rel = 0.7 - 0.6 * 0.2 / sqrt(3)
    rank = 4
    s = np.tile(np.array([1.0, 0, 0, 0]), (3, 1))
    xi = np.array([[a, np.sqrt(1 - a * a), 0, 0] for a in (0.5, 0.7, 0.9)])
    base = dict(slot=np.zeros(3, np.int32), keep=None, n=np.zeros(1, int), mean=np.zeros(1), M2=np.zeros(1),
                n_fb=np.zeros(1, int), m=np.ones((1, 8)), horizon=np.zeros(1, np.int32))
    out = ref.reflex_gate(s, xi, n_align_min=[3], n_fb_min=[1], alpha_lo=[0.01], alpha_hi=[0.025], **base)
    rel = 0.7 - 0.6 * 0.2 / np.sqrt(3.0)
    assert abs(out["rel"][0] - rel) < 1e-12
    assert abs(out["alpha"][0] - (0.01 + 0.015 * rel)) < 1e-12 and 0.01 <= out["alpha"][0] <= 0.025
    # each condition closes the gate on its own: too few alignments, too few feedback records, empty memory,
    # non-positive score
    assert ref.reflex_gate(s, xi, n_align_min=[4], n_fb_min=[1], alpha_lo=[0.01], alpha_hi=[0.025], **base)["alpha"][0] == 0
    assert ref.reflex_gate(s, xi, n_align_min=[3], n_fb_min=[4], alpha_lo=[0.01], alpha_hi=[0.025], **base)["alpha"][0] == 0
    empty = dict(base, m=np.zeros((1, 8)))
    assert ref.reflex_gate(s, xi, n_align_min=[3], n_fb_min=[1], alpha_lo=[0.01], alpha_hi=[0.025], **empty)["alpha"][0] == 0
    neg = ref.reflex_gate(s, -xi, n_align_min=[3], n_fb_min=[1], alpha_lo=[0.01], alpha_hi=[0.025], **base)
    assert neg["rel"][0] < 0 and neg["alpha"][0] == 0
    # one record: no sample variance, not eligible
    one = ref.reflex_gate(s[:1], xi[:1], n_align_min=[1], n_fb_min=[1], alpha_lo=[0.01], alpha_hi=[0.025],
                          **dict(base, slot=np.zeros(1, np.int32)))
    assert one["rel"][0] == -np.inf and one["alpha"][0] == 0
