"""The capacity profile of Eq. "verification-budget" runs and is self-consistent on a small shape."""
import pytest
import torch

from paper_2608_04962_b200 import binding as S
from paper_2608_04962_b200 import chw
from paper_2608_04962_b200 import inputs as I

pytestmark = pytest.mark.gpu


def test_profile_on_a_small_shape():
    w = I.scaled(I.WORKLOADS["tiny"], layers=2)
    res = chw.profile(w, Bs=(4, 2), Ns=(2, 4, 8), device=torch.device("cuda", 0), layers_measured=1, warmup=1, steps=2,
                      tau=0.5)
    assert len(res["points"]) == 6
    for p in res["points"]:
        assert p["nodes"] == p["B"] * p["N"] and p["verification_side_ms"] > 0
        assert abs(p["verification_side_ms"] - (w.layers * p["attn_ms_per_layer"] + p["verify_ms"])) < 1e-9
    # the capacity at a batch size is one of the swept node totals, and C_hw their median
    for B, cap in res["capacity_per_B"].items():
        assert cap in {int(B) * n for n in (2, 4, 8)}
    assert res["C_hw"] > 0
    # the budget rule turns it into nodes per sequence
    assert S.node_budget(res["C_hw"], 4, 1, 8) == max(1, min(8, res["C_hw"] // 4))
