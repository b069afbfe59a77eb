"""GPU parity: the target projection with fused row statistics against the CPU oracle."""
import numpy as np
import pytest
import torch

from oracle import ref
from paper_2608_04962_b200 import binding as S
from paper_2608_04962_b200 import inputs as I
from tests.util import dev, dev_bf16, host

pytestmark = pytest.mark.gpu


def _case(seed, R, d, V, kw, spread=1.0):
    g = I.rng(seed)
    H = I.f32_to_bf16_bits((spread * g.standard_normal((R, d))).astype(np.float32))
    W = I.f32_to_bf16_bits((g.standard_normal((V, d)) / np.sqrt(d)).astype(np.float32))
    want = g.integers(0, V, size=(R, kw)).astype(np.int32) if kw else None
    if kw:
        want[:, 0] = 0            # the ends of the vocabulary
        want[:, -1] = V - 1
    return H, W, want


def _ulp_close(got_bits, want_bits, H, W, rows=None, cols=None):
    """bf16 values produced from fp32 sums against values rounded once from fp64 sums: equal, except where the
    exact value sits within the fp32 accumulation error of a bf16 midpoint (then one unit in the last place
    apart) or is so close to zero, by cancellation, that the accumulation error itself exceeds its bf16 spacing.
    Bound: one bf16 unit of the value plus 2e-6 of the sum of the absolute products."""
    a = I.bf16_bits_to_f32(got_bits).astype(np.float64)
    b = I.bf16_bits_to_f32(want_bits).astype(np.float64)
    Hf = np.abs(I.bf16_bits_to_f32(H).astype(np.float64))
    Wf = np.abs(I.bf16_bits_to_f32(W).astype(np.float64))
    mag = Hf @ Wf.T
    if cols is not None:
        mag = np.take_along_axis(mag, cols.astype(np.int64), -1)
    diff = np.abs(a - b)
    assert (diff <= np.abs(b) * 2.0 ** -7 * 1.0001 + 2e-6 * mag).all(), float(diff.max())
    return float((diff > 0).mean())


@pytest.mark.parametrize("R,d,V,kw,T", [(300, 256, 4096, 8, 1.0), (130, 1536, 20008, 4, 0.7), (64, 64, 1000, 0, 1.0),
                                        (1, 128, 264, 8, 1.3), (513, 320, 777 * 8, 3, 1.0)])
def test_statistics_and_wanted_logits(R, d, V, kw, T):
    H, W, want = _case(5 + R, R, d, V, kw, spread=2.0)
    o = ref.target_head(H, W, temperature=T, want_id=want)
    g = S.target_head_stats(dev_bf16(H), dev_bf16(W), dev(want) if kw else None, temperature=T)
    torch.cuda.synchronize()
    # the maximum is a bf16 value: equal, or one unit apart where the rounding flipped
    gm = host(g["row_max"]).astype(np.float64)
    assert (np.abs(gm - o["row_max"]) <= np.abs(o["row_max"]) * 2.0 ** -7 + 1e-30).all()
    # the sum moves with every flipped logit by at most 2^-7 / T of that term: well inside 2e-3
    np.testing.assert_allclose(host(g["row_sum"]).astype(np.float64) * np.exp((gm - o["row_max"]) / np.float32(T)),
                               o["row_sum"], rtol=2e-3)
    if kw:
        flipped = _ulp_close(host(g["want_logit"].view(torch.uint16)), o["want_logit"], H, W, cols=want)
        assert flipped < 0.05


@pytest.mark.parametrize("R,d,V", [(256, 256, 4096), (5, 1536, 20008), (129, 64, 264)])
def test_stored_rows_and_consistency_with_the_fused_form(R, d, V):
    H, W, want = _case(77 + R, R, d, V, 8)
    o = ref.target_head(H, W, want_id=want)
    lg = S.target_head_rows(dev_bf16(H), dev_bf16(W))
    torch.cuda.synchronize()
    got = host(lg.view(torch.uint16))
    flipped = _ulp_close(got, o["logits"], H, W)
    assert flipped < 0.02
    # the fused form sees exactly the logits the storing form writes: its statistics and wanted logits follow
    # from the stored rows
    g = S.target_head_stats(dev_bf16(H), dev_bf16(W), dev(want))
    l = I.bf16_bits_to_f32(got).astype(np.float64)
    assert np.array_equal(host(g["row_max"]).astype(np.float64), l.max(-1))
    np.testing.assert_allclose(host(g["row_sum"]), np.exp(l - l.max(-1, keepdims=True)).sum(-1), rtol=2e-5)
    assert np.array_equal(host(g["want_logit"].view(torch.uint16)), np.take_along_axis(got, want.astype(np.int64), -1))
