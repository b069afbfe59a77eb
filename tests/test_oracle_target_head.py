"""Pins for the oracle's target projection with row statistics."""
import numpy as np

from oracle import ref
from paper_2608_04962_b200 import inputs as I


def _bits(x):
    return I.f32_to_bf16_bits(np.asarray(x, np.float32))


def _f(b):
    return I.bf16_bits_to_f32(b).astype(np.float64)


def test_unit_rows_read_off_the_columns_of_the_projection():
    # H = rows of the identity: l[r, :] is column r of W exactly (already bf16), so the statistics follow from W alone
    g = I.rng(2)
    V, d = 50, 8
    W = _bits(g.standard_normal((V, d)))
    H = _bits(np.eye(d))
    for T in (1.0, 0.7):
        o = ref.target_head(H, W, temperature=T, want_id=np.tile(np.array([[3, 49, 0]]), (d, 1)))
        Wf = _f(W)
        for r in range(d):
            col = Wf[:, r]
            assert np.array_equal(_f(o["logits"][r]), col)
            assert o["row_max"][r] == col.max()
            s = sum(np.exp((x - col.max()) / np.float32(T)) for x in col)
            assert abs(o["row_sum"][r] - s) < 1e-12 * s
            assert np.array_equal(_f(o["want_logit"][r]), col[[3, 49, 0]])


def test_logits_are_the_rounded_products_and_the_probabilities_sum_to_one():
    g = I.rng(3)
    R, V, d = 5, 64, 32
    H, W = _bits(g.standard_normal((R, d))), _bits(0.3 * g.standard_normal((V, d)))
    o = ref.target_head(H, W, temperature=1.3)
    exact = _f(H) @ _f(W).T
    l = _f(o["logits"])
    # one rounding to bf16: within half a unit in the last place (2^-9 relative)
    assert (np.abs(l - exact) <= np.abs(exact) * 2.0 ** -8 + 1e-30).all()
    p = np.exp((l - o["row_max"][:, None]) / np.float32(1.3)) / o["row_sum"][:, None]
    np.testing.assert_allclose(p.sum(-1), 1.0, atol=1e-12)
    assert (o["row_max"] == l.max(-1)).all()
    # scaling every hidden row by 2 doubles the logits exactly (a power of two commutes with the rounding)
    o2 = ref.target_head(_bits(2.0 * _f(H)), W, temperature=1.3)
    assert np.array_equal(_f(o2["logits"]), 2.0 * l)
