"""Pins for the oracle's verifier feedback (distribution and coverage directions, memory update)."""
import numpy as np

from oracle import ref
from paper_2608_04962_b200 import inputs as I


def _bits(x):
    return I.f32_to_bf16_bits(np.asarray(x, np.float32))


def _f(bits):
    return I.bf16_bits_to_f32(bits).astype(np.float64)


def _case(seed, V=40, d=12, k=4, R=3, spread=2.0):
    g = I.rng(seed)
    W = _bits(g.standard_normal((V, d)))
    logits = _bits(spread * g.standard_normal((R, V)))
    head = g.standard_normal((R, V))
    order = np.argsort(-head, axis=-1)[:, :k]
    cand_id = order.astype(np.int32)
    cand_logit = np.take_along_axis(head, order, -1).astype(np.float32)
    y = g.integers(0, V, size=R).astype(np.int32)
    m = g.standard_normal((R, d)).astype(np.float32)
    rho = np.array([0.85, 0.9, 0.95][:R])
    return W, logits, cand_id, cand_logit, y, m, rho


def test_distribution_direction_is_the_descent_direction_of_the_cross_entropy():
    # When the target's top-k are the candidates themselves and y* is one of them, S = C and nothing is omitted;
    # with q = softmax(W_C z / T) for a head state z, r_dist = W_C^T (p_C - q_C) = -T * grad_z CE(p_C || q(z)),
    # and the feedback e keeps that direction.  Checked against central differences of the cross-entropy.
    g = I.rng(3)
    V, d, k, T = 30, 8, 5, 0.8
    W = _bits(g.standard_normal((V, d)))
    Wf = _f(W)
    z = g.standard_normal(d)
    C = np.array([3, 11, 17, 22, 29], np.int32)
    cl = (Wf[C] @ z).astype(np.float32)
    order = np.argsort(-cl, kind="stable")
    C, cl = C[order], cl[order]
    lg = -20.0 + 0.1 * g.standard_normal(V)
    lg[C] = np.array([1.5, 0.25, 1.0, -0.5, 0.75])                 # the target's top-5 are exactly C
    logits = _bits(lg[None])
    out = ref.reflex_feedback(logits, W, C[None], cl[None], np.array([C[0]], np.int32), np.zeros((1, d), np.float32),
                              np.array([0.0]), k_support=k, temperature=T)
    assert sorted(out["support"][0]) == sorted(C.tolist()) and abs(out["d_cov"][0]) < 1e-12
    p = np.exp(_f(logits[0]) / np.float32(T))
    pC = p[C] / p[C].sum()

    def ce(zz):
        s = Wf[C] @ zz / np.float32(T)
        ls = s - (np.log(np.exp(s - s.max()).sum()) + s.max())
        return -(pC * ls).sum()

    grad = np.array([(ce(z + 1e-6 * np.eye(d)[i]) - ce(z - 1e-6 * np.eye(d)[i])) / 2e-6 for i in range(d)])
    e = out["e"][0]
    cos = (e @ -grad) / (np.linalg.norm(e) * np.linalg.norm(grad))
    assert cos > 0.999999, cos                                      # (cand_logit is fp32: q moves by ~1e-7)


def test_perfect_proposal_leaves_only_the_decay():
    # q equal to p on C and C equal to the target's top-k: both magnitudes vanish, the memory just decays
    g = I.rng(4)
    V, d, k = 24, 6, 4
    W = _bits(g.standard_normal((V, d)))
    lg = np.full(V, -8.0)
    C = np.array([5, 9, 2, 17], np.int32)
    lg[C] = [2.0, 1.0, 0.5, 0.0]
    logits = _bits(lg[None])
    cl = np.array([2.0, 1.0, 0.5, 0.0], np.float32)
    m = g.standard_normal((1, d)).astype(np.float32)
    out = ref.reflex_feedback(logits, W, C[None], cl[None], np.array([5], np.int32), m, np.array([0.9]), k_support=8)
    assert abs(out["tv"][0]) < 1e-12 and abs(out["d_cov"][0]) < 1e-12
    assert np.allclose(out["m"][0], 0.9 * m[0].astype(np.float64), atol=1e-12)


def test_magnitudes_and_support_against_their_definitions():
    W, logits, cand_id, cand_logit, y, m, rho = _case(5)
    kS = 6
    out = ref.reflex_feedback(logits, W, cand_id, cand_logit, y, m, rho, k_support=kS)
    for r in range(logits.shape[0]):
        l = _f(logits[r])
        p = np.exp(l) / np.exp(l).sum()
        q = np.exp(cand_logit[r].astype(np.float64))
        q /= q.sum()
        C = list(cand_id[r])
        top = sorted(range(len(l)), key=lambda v: (-l[v], v))
        assert set(out["support"][r]) == set(C) | set(top[:kS]) | {int(y[r])}
        pC = p[C].sum()
        assert np.isclose(out["p_C"][r], pC)
        assert np.isclose(out["d_dist"][r], pC * 0.5 * np.abs(p[C] / pC - q).sum())
        assert np.isclose(out["d_cov"][r], p[top[:len(C)]].sum() - pC) and out["d_cov"][r] >= -1e-15
        # the decomposition of the paper: p(C*) - p(C) (1 - TV) = d_dist + d_cov
        assert np.isclose(p[top[:len(C)]].sum() - pC * (1 - out["tv"][r]), out["d_dist"][r] + out["d_cov"][r])


def test_feedback_norm_direction_and_memory_update():
    W, logits, cand_id, cand_logit, y, m, rho = _case(6)
    eps = 1e-6
    out = ref.reflex_feedback(logits, W, cand_id, cand_logit, y, m, rho, k_support=6, eps=eps)
    for r in range(3):
        e = out["e"][r]
        s = out["d_dist"][r] + out["d_cov"][r]
        rms_e = np.sqrt(np.mean(e * e))
        assert rms_e <= s + 1e-12 and rms_e > s * (1 - 1e-3)          # RMS(e) = s RMS(g)/(RMS(g)+eps)
        assert np.allclose(out["m"][r], rho[r] * m[r] + (1 - rho[r]) * e, atol=1e-12)
    # the same feedback applied n times from zero memory: m = (1 - rho^n) e
    mm = np.zeros_like(m[:1])
    for _ in range(5):
        o = ref.reflex_feedback(logits[:1], W, cand_id[:1], cand_logit[:1], y[:1], mm, rho[:1], k_support=6)
        mm = o["m"].astype(np.float32)
    assert np.allclose(mm[0], (1 - rho[0] ** 5) * o["e"][0], rtol=1e-5, atol=1e-7)


def test_coverage_direction_promotes_the_omitted_token_over_the_weakest_candidate():
    # one omitted target-important token y: r_cov = p_S(y) (W_y - W_b*); with d_dist forced to 0 the feedback is
    # along it, so it raises logit(y) - logit(b*)
    g = I.rng(7)
    V, d = 20, 10
    W = _bits(g.standard_normal((V, d)))
    Wf = _f(W)
    C = np.array([1, 2, 3], np.int32)
    cl = np.array([1.0, 0.0, -1.0], np.float32)
    lg = np.full(V, -9.0)
    q = np.exp(cl.astype(np.float64))
    q /= q.sum()
    lg[C] = np.log(q)                     # p proportional to q on C: no distribution error
    lg[7] = 3.0                            # a token the head missed
    logits = _bits(lg[None])
    out = ref.reflex_feedback(logits, W, C[None], cl[None], np.array([7], np.int32), np.zeros((1, d), np.float32),
                              np.array([0.0]), k_support=4)
    assert out["d_cov"][0] > 0.5 and out["tv"][0] < 2e-2
    e = out["e"][0]
    assert e @ (Wf[7] - Wf[3]) > 0
    cos = e @ (Wf[7] - Wf[3]) / (np.linalg.norm(e) * np.linalg.norm(Wf[7] - Wf[3]))
    assert cos > 0.99
