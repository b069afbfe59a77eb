"""Profiling the verification capacity C_hw of Eq. "verification-budget" (Sec. 3.2: "the profiled verification
capacity of the model-hardware pair") for the part of the target step this library runs.

For each active batch size B the per-sequence node count N is swept; a point's cost is the device time of the
step's verification side, ``layers`` tree-attention calls plus one exact verification, measured with CUDA events
on seeded synthetic inputs of the workload's shape.  While the hardware is under-used the cost is flat in N; the
capacity at B is the largest B * N whose cost stays within ``tau`` of the cheapest point at that B, and C_hw is
the median of those over the B swept.  The target's dense layers are not part of this library: a caller adds
its own per-token cost to the table before taking the knee if it wants the whole step.
"""
from __future__ import annotations

from dataclasses import replace
from typing import Dict, Iterable, List

import numpy as np
import torch

from . import inputs as I
from .workload import StepWorkload


def _time_ms(fn, warmup: int, steps: int) -> float:
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(steps):
        fn()
    b.record()
    torch.cuda.synchronize()
    return a.elapsed_time(b) / steps


def profile(w: I.Workload, Bs: Iterable[int], Ns: Iterable[int], device, layers_measured: int = 2, warmup: int = 3,
            steps: int = 5, tau: float = 0.10) -> Dict:
    """Sweeps (B, N) and returns the cost table, the capacity per B and C_hw.  ``layers_measured`` caches are
    allocated per point (each larger than L2) and the attention time is scaled to the model's ``w.layers``."""
    Ns = sorted(set(int(n) for n in Ns))
    table: List[Dict] = []
    per_B: Dict[int, int] = {}
    for B in Bs:
        row = []
        for N in Ns:
            wp = replace(w, name=f"{w.name}_chw_B{B}_N{N}", B=int(B), N=int(N), fixed_parent=None)
            wl = StepWorkload(wp, device, layers=layers_measured)
            wl.propose()
            L = wl.layers

            def attn():
                for layer in range(L):
                    wl.attn(layer)

            t_attn = _time_ms(attn, warmup, steps) / L
            t_ver = _time_ms(wl.verify, warmup, steps)
            cost = w.layers * t_attn + t_ver
            row.append(cost)
            table.append({"B": int(B), "N": N, "nodes": int(B) * N, "attn_ms_per_layer": t_attn, "verify_ms": t_ver,
                          "verification_side_ms": cost})
            del wl
            torch.cuda.empty_cache()
        floor = min(row)
        ok = [n for n, c in zip(Ns, row) if c <= (1.0 + tau) * floor]
        per_B[int(B)] = int(B) * max(ok)
    c_hw = int(np.median(list(per_B.values()))) if per_B else 0
    return {"workload": w.name, "tau": tau, "layers": w.layers, "points": table, "capacity_per_B": per_B, "C_hw": c_hw}
