#!/usr/bin/env python
"""Benchmark of the SpecRoll per-step speculative hot path on B200.

One step = specroll_propose -> specroll_tree_attn for every layer -> specroll_verify over one
batch of synthetic input.  Prints ONE JSON line (rank 0).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

`--impl reference` times the CPU oracle (the only reference there is: the paper ships no code)
on the host cores, each step a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "verified tree tokens/sec per speculative step"
UNIT = "tokens/s"


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def recorded_traffic(kernel: str, workload: str):
    """DRAM bytes per launch from the committed ncu summary, or None."""
    p = os.path.join(ROOT, "profiles", "traffic.json")
    if not os.path.exists(p):
        return None
    try:
        return json.load(open(p)).get(workload, {}).get(kernel)
    except Exception:
        return None


# ------------------------------------------------------------------------------------ clocks


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU from a background thread (NVML) while the timed
    region runs; falls back to one `nvidia-smi` query when NVML is not importable."""

    REASONS = (("hw_slowdown", 0x8), ("hw_thermal_slowdown", 0x40), ("sw_thermal_slowdown", 0x20),
               ("sw_power_cap", 0x4))

    def __init__(self, gpu_index: int, period_s: float = 0.002):
        self.idx = gpu_index
        self.period = period_s
        self.sm, self.power, self.reasons = [], [], set()
        self.max_mhz = None
        self._stop = False
        self._thread = None
        self._nvml = None

    def _run(self):
        nv, h = self._nvml, self._h
        while not self._stop:
            try:
                self.sm.append(float(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM)))
                try:
                    self.power.append(nv.nvmlDeviceGetPowerUsage(h) / 1000.0)
                except Exception:
                    pass
                bits = int(nv.nvmlDeviceGetCurrentClocksEventReasons(h))
                for name, mask in self.REASONS:
                    if bits & mask:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def start(self):
        try:
            import pynvml as nv
            nv.nvmlInit()
            vis = os.environ.get("CUDA_VISIBLE_DEVICES")
            phys = self.idx
            if vis:
                ids = [x for x in vis.split(",") if x.strip() != ""]
                if self.idx < len(ids) and ids[self.idx].strip().isdigit():
                    phys = int(ids[self.idx])
            self._h = nv.nvmlDeviceGetHandleByIndex(phys)
            self.max_mhz = float(nv.nvmlDeviceGetMaxClockInfo(self._h, nv.NVML_CLOCK_SM))
            self._nvml = nv
            import threading
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        except Exception:
            self._nvml = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        if self._thread is not None:
            self._stop = True
            self._thread.join(timeout=2)
        if not self.sm:
            try:  # one-shot fallback right after the timed region
                q = subprocess.run(["nvidia-smi", "--query-gpu=clocks.sm,clocks.max.sm", "--format=csv,noheader,nounits",
                                    "-i", str(self.idx)], capture_output=True, text=True, timeout=10).stdout
                c = [x.strip() for x in q.strip().splitlines()[0].split(",")]
                out.update(sm_mhz=float(c[0]), sm_max_mhz=float(c[1]), samples=1, note="sampled after the timed region")
            except Exception:
                pass
            return out
        out.update(sm_mhz=float(np.median(self.sm)), reasons=sorted(self.reasons), samples=len(self.sm))
        if self.power:
            out.update(power_w_median=float(np.median(self.power)), power_w_max=float(np.max(self.power)))
        return out


# ------------------------------------------------------------------------------------ CPU oracle legs


def use_host_cores_under_a_launcher():
    """torchrun exports OMP_NUM_THREADS=1 to its ranks unless the caller set it.  The CPU legs run on rank 0 alone
    (the other ranks do no CPU work) and are meant to use the machine's host cores, as they do when bench.py is
    started directly: give the OpenMP runtime the cores this process may run on."""
    if "TORCHELASTIC_RUN_ID" not in os.environ or os.environ.get("OMP_NUM_THREADS") != "1":
        return
    try:
        import ctypes
        ctypes.CDLL("libgomp.so.1").omp_set_num_threads(len(os.sched_getaffinity(0)))
    except OSError:
        pass


def oracle_sample_step(w, n_seq: int, layers: int, ref_layers: int):
    """One pass of the whole path by the CPU oracle over the first n_seq sequences of `w`.  The attention is run
    for min(ref_layers, layers) layers and its time scaled to `layers` (every layer costs the oracle the same: same
    shapes, and its loops do not depend on the values), so that a step of the deep shapes stays within seconds.
    Returns (callable -> seconds of one step, tokens processed, threads, layers actually run)."""
    from oracle import ref
    from paper_2608_04962_b200 import inputs as I
    ref.lib()
    use_host_cores_under_a_launcher()
    ws = I.scaled(w, B=n_seq)
    x = I.propose_inputs(ws)
    a = I.attn_inputs(ws)
    u_acc, u_fin = I.verify_uniforms(ws)
    run_layers = max(1, min(ref_layers, layers))
    # target logits need the proposal's tokens; that first (untimed) pass also warms the caches
    pr = ref.propose(x["h"], x["anchor"], x["A"], x["bias"], x["W"], x["m"], x["alpha"], x["parent"], x["u_draw"],
                     k=ws.k, temperature=ws.temperature, clip_c=ws.clip_c)
    lg = I.target_logits(ws, x["parent"], pr["tree_tok"])

    def one():
        t0 = time.perf_counter()
        p = ref.propose(x["h"], x["anchor"], x["A"], x["bias"], x["W"], x["m"], x["alpha"], x["parent"],
                        x["u_draw"], k=ws.k, temperature=ws.temperature, clip_c=ws.clip_c)
        t1 = time.perf_counter()
        for _ in range(run_layers):   # same arrays every layer: the oracle's cost does not depend on the values
            ref.tree_attn(a["Q"], a["Kc"], a["Vc"], a["kv_indptr"], a["Kt"], a["Vt"], a["parent"])
        t2 = time.perf_counter()
        ref.verify(lg, x["parent"], p["tree_tok"], p["tree_cand"], p["cand_id"], p["cand_logit"], u_acc, u_fin,
                   temperature=ws.temperature)
        t3 = time.perf_counter()
        return (t1 - t0) + (t2 - t1) * (layers / run_layers) + (t3 - t2)

    return one, ws.B * ws.N, ref.num_threads(), run_layers


def oracle_sample_text(w, n_seq, layers, run_layers):
    s = f"first {n_seq} of {w.B} sequences of {w.name}, per step: proposal, verification and {run_layers} attention layer(s)"
    if run_layers != layers:
        s += f" with the attention time scaled to all {layers} layers"
    return s


def run_reference(args, w, layers):
    from paper_2608_04962_b200 import dist as D
    rank, _, world = D.env_world()
    if rank != 0:
        return 0
    n_seq = args.ref_seqs
    one, tokens, threads, run_layers = oracle_sample_step(w, n_seq, layers, args.ref_layers)
    for _ in range(args.warmup):
        one()
    t = [one() for _ in range(args.steps)]
    total = float(sum(t))
    value = tokens * args.steps / total
    sample = oracle_sample_text(w, n_seq, layers, run_layers)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "B": w.B, "N": w.N, "K": w.K, "k": w.k, "layers": layers,
                       "sample": sample},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)
    return 0


# ------------------------------------------------------------------------------------ our arm


def phase_fractions(w, wl, prop_ms, attn_layer_ms, ver_ms, peaks):
    """Roofline fraction of each call: the time the binding resource needs at the measured peak / the time taken.
    Attention: HBM (every cached element once) or the tensor pipe (its FLOPs at the burst bf16 peak), whichever
    needs longer.  Proposal: the tensor pipe where the projection has B K >= 253 rows (its arithmetic intensity is
    B K FLOP per byte of W), else HBM (the weights W and A once).  Verification: HBM (the logits once)."""
    bw, tf = peaks["hbm_gbs"] * 1e9, peaks["bf16_tflops"] * 1e12
    t_mem = wl.attn_algorithmic_bytes() / bw
    t_tc = wl.attn_algorithmic_flops() / tf
    attn = {"us_per_layer": attn_layer_ms * 1e3, "bound": "hbm" if t_mem >= t_tc else "tensor",
            "t_mem_us": t_mem * 1e6, "t_tensor_us": t_tc * 1e6, "frac": max(t_mem, t_tc) / (attn_layer_ms * 1e-3)}
    p_flops = wl.lmhead_algorithmic_flops() + 2 * w.B * w.K * w.d * w.d
    p_bytes = wl.lmhead_algorithmic_bytes() + wl.heads_algorithmic_bytes()
    if w.B * w.K >= 253:
        prop = {"ms": prop_ms, "bound": "tensor", "frac": (p_flops / tf) / (prop_ms * 1e-3)}
    else:
        prop = {"ms": prop_ms, "bound": "hbm", "frac": (p_bytes / bw) / (prop_ms * 1e-3)}
    ver = {"ms": ver_ms, "bound": "hbm", "frac": (wl.rowstats_algorithmic_bytes() / bw) / (ver_ms * 1e-3)}
    return attn, prop, ver


def measure_power_roof(wl, local, secs=2.0):
    """The board's power limit as a roof for the attention kernel (rank 0, one GPU).  Board power (NVML, 50 Hz, median of
    the second half of each loop) of: the idle context, a device-to-device copy at full speed, a bf16 GEMM loop, and
    this workload's attention layers back to back.  With the energy per byte of the copy and per FLOP of the GEMM, a
    kernel with the attention's mix of bytes and FLOPs can sustain at most `max_hbm_frac` of the copy rate under the
    board's limit.  None when NVML is not there."""
    import threading
    import torch
    try:
        import pynvml as nv
        nv.nvmlInit()
        phys, vis = local, os.environ.get("CUDA_VISIBLE_DEVICES")
        if vis:
            ids = [x for x in vis.split(",") if x.strip() != ""]
            if local < len(ids) and ids[local].strip().isdigit():
                phys = int(ids[local])
        h = nv.nvmlDeviceGetHandleByIndex(phys)
        limit_w = nv.nvmlDeviceGetPowerManagementLimit(h) / 1000.0
    except Exception:
        return None
    dev = torch.device("cuda", local)

    def loop(body):
        stop, out = threading.Event(), []

        def run():
            while not stop.is_set():
                try:
                    out.append(nv.nvmlDeviceGetPowerUsage(h) / 1000.0)
                except Exception:
                    pass
                time.sleep(0.02)

        th = threading.Thread(target=run, daemon=True)
        torch.cuda.synchronize()
        th.start()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        t0, n = time.perf_counter(), 0
        while time.perf_counter() - t0 < secs:
            n += body()
            torch.cuda.synchronize()
        e1.record()
        torch.cuda.synchronize()
        stop.set()
        th.join(timeout=2)
        tail = sorted(out[len(out) // 2:]) or [float("nan")]
        return tail[len(tail) // 2], n, e0.elapsed_time(e1) * 1e-3

    def idle():
        time.sleep(0.1)
        return 0

    try:
        src = torch.empty(2 << 30, dtype=torch.uint8, device=dev)
        dst = torch.empty_like(src)
        A = torch.randn(8192, 8192, device=dev, dtype=torch.bfloat16)
        Bm = torch.randn(8192, 8192, device=dev, dtype=torch.bfloat16)
    except Exception:
        return None

    def copy():
        for _ in range(8):
            dst.copy_(src)
        return 8

    def gemm():
        for _ in range(40):
            torch.matmul(A, Bm)
        return 40

    def attn():
        for l in range(wl.layers):
            wl.attn(l)
        return wl.layers

    idle_w, _, _ = loop(idle)
    copy_w, nc, tc = loop(copy)
    gemm_w, ng, tg = loop(gemm)
    attn_w, na, ta = loop(attn)
    copy_gbs = nc * 2 * src.numel() / tc / 1e9
    gemm_tf = ng * 2 * 8192 ** 3 / tg / 1e12
    attn_gbs = na * wl.attn_algorithmic_bytes() / ta / 1e9
    attn_tf = na * wl.attn_algorithmic_flops() / ta / 1e12
    del src, dst, A, Bm
    torch.cuda.empty_cache()
    x_h, x_t = attn_gbs / copy_gbs, attn_tf / gemm_tf
    denom = (copy_w - idle_w) + (x_t / x_h) * (gemm_w - idle_w)
    max_h = (limit_w - idle_w) / denom if denom > 0 else float("nan")
    return {"limit_w": limit_w, "idle_w": idle_w, "copy_w": copy_w, "copy_gbs_read_plus_write": copy_gbs,
            "gemm_w": gemm_w, "gemm_tflops": gemm_tf, "attn_w": attn_w, "attn_gbs_sustained": attn_gbs,
            "attn_tflops_sustained": attn_tf,
            "model_w": idle_w + x_h * (copy_w - idle_w) + x_t * (gemm_w - idle_w),
            "max_frac_of_copy_rate": max_h, "attn_frac_of_copy_rate": x_h, "attn_frac_of_power_roof": x_h / max_h,
            "note": "power = idle + (copy - idle) * (bytes/s over the copy's) + (gemm - idle) * (FLOP/s over the GEMM's); "
                    "max_frac_of_copy_rate = the largest byte rate, as a fraction of the copy's, that a kernel with the "
                    "attention's ratio of FLOPs to bytes sustains under limit_w by that model; loops of %.0f s each" % secs}


def measure_workload(w, dev, layers, steps, peaks, local):
    """One entry of the `workloads` array: the step of workload `w` with `layers` attention layers (enough for the
    per-layer time: every layer has its own cache, larger than L2), its per-call times and roofline fractions, and
    the step time and throughput of the shape's full depth put together from them."""
    import torch
    from paper_2608_04962_b200.workload import StepWorkload
    wl = StepWorkload(w, dev, layers=min(layers, w.layers))
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(steps)]
    for _ in range(3):
        wl.step()
    torch.cuda.synchronize()
    sampler = ClockSampler(local)
    sampler.start()
    for i in range(steps):
        wl.step(ev[i])
    torch.cuda.synchronize()
    clocks = sampler.stop()
    prop_ms = float(np.median([e[0].elapsed_time(e[1]) for e in ev]))
    attn_ms = float(np.median([e[1].elapsed_time(e[2]) for e in ev])) / wl.layers
    ver_ms = float(np.median([e[2].elapsed_time(e[3]) for e in ev]))
    attn, prop, ver = phase_fractions(w, wl, prop_ms, attn_ms, ver_ms, peaks)
    full_ms = prop_ms + w.layers * attn_ms + ver_ms
    out = {"workload": w.name, "B": w.B, "N": w.N, "rows_per_kv_head": w.N * (w.Hq // w.Hkv), "layers": w.layers,
           "layers_run": wl.layers, "ms_per_step": full_ms, "tokens_per_s": w.B * w.N / (full_ms * 1e-3),
           "attn_us_per_layer": attn["us_per_layer"], "attn_bound": attn["bound"], "attn_frac": attn["frac"],
           "propose_ms": prop_ms, "propose_bound": prop["bound"], "propose_frac": prop["frac"],
           "verify_ms": ver_ms, "verify_frac": ver["frac"], "clocks": clocks}
    del wl
    torch.cuda.empty_cache()
    return out


def run_ours(args, w, layers):
    import torch
    from paper_2608_04962_b200 import binding as S
    from paper_2608_04962_b200 import dist as D
    from paper_2608_04962_b200.workload import StepWorkload

    rank, local, world = D.env_world()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback of the hot path")
    S.lib()                                   # fails loudly if the library is not built
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    D.init("nccl")
    wl = StepWorkload(w, dev, seed=rank, layers=layers, paged=args.paged, top_p=args.top_p, lazy_stats=args.lazy_stats)
    peaks = measured_peaks()

    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(args.steps)]
    for _ in range(max(args.warmup, 3)):
        wl.step()
    torch.cuda.synchronize()
    graph = None
    if args.graph:
        # the whole step as one CUDA graph: the entry points only enqueue work on the caller's stream (kernels,
        # one memset; tensor maps travel as kernel arguments), so a step can be captured and replayed
        try:
            side = torch.cuda.Stream(dev)
            side.wait_stream(torch.cuda.current_stream(dev))
            with torch.cuda.stream(side):
                wl.step()
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph, stream=side):
                    wl.step()
            torch.cuda.current_stream(dev).wait_stream(side)
            for _ in range(3):
                graph.replay()
            torch.cuda.synchronize()
        except Exception as exc:                       # capture refused: time plain launches instead
            print(f"bench: CUDA graph capture failed ({exc}); timing plain launches", file=sys.stderr)
            graph = None
            torch.cuda.synchronize()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    D.barrier()
    torch.cuda.synchronize()
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    for i in range(args.steps):
        if graph is not None:
            graph.replay()
        else:
            wl.step(ev[i])
    t1.record()
    torch.cuda.synchronize()
    D.barrier()
    clocks = sampler.stop() if rank == 0 else None
    elapsed_ms = t0.elapsed_time(t1)
    tokens = wl.tokens_per_step() * args.steps
    tmax, tok_all = D.aggregate(elapsed_ms, tokens, device=dev)
    value = tok_all / (tmax * 1e-3)

    if graph is not None:
        # phase times are not visible inside a replayed graph: take them from a few plain steps afterwards
        torch.cuda.synchronize()
        for i in range(args.steps):
            wl.step(ev[i])
        torch.cuda.synchronize()
    prop_ms = float(np.mean([e[0].elapsed_time(e[1]) for e in ev]))
    attn_ms = float(np.mean([e[1].elapsed_time(e[2]) for e in ev]))
    ver_ms = float(np.mean([e[2].elapsed_time(e[3]) for e in ev]))
    attn_launch_s = attn_ms * 1e-3 / wl.layers

    # accepted-length statistics of the synthetic workload (reporting only)
    n_acc = wl.ver["n_acc"].float()
    aal = float(1.0 + n_acc.mean().item())
    ar = float(n_acc.sum().item() / max(1, w.B * (w.N - 1)))

    # ---- end to end through host buffers
    e2e = None if args.no_e2e else run_e2e(args, wl, dev, world)
    e2e_fused = None
    if not args.no_e2e and w.k <= 8:
        e2e_fused = run_e2e(args, wl, dev, world, fused=True)

    if rank != 0:
        D.finish()
        return 0

    attn_gbs = wl.attn_algorithmic_bytes() / attn_launch_s / 1e9
    attn_tfs = wl.attn_algorithmic_flops() / attn_launch_s / 1e12
    roofline = {"kernel": "tree_attn_tc_kernel (timed as the specroll_tree_attn call: prep kernel + attention kernel)",
                "bound": "hbm",
                "achieved": attn_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": attn_gbs / peaks["hbm_gbs"],
                "peak_source": peaks["source"], "frac_of_nominal_8TBs": attn_gbs / 8000.0,
                "algorithmic_bytes_per_launch": wl.attn_algorithmic_bytes(),
                "algorithmic_flops_per_launch": wl.attn_algorithmic_flops(),
                "tensor_side": {"achieved": attn_tfs, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                                "frac": attn_tfs / peaks["bf16_tflops"],
                                "note": "the same launch against the dense bf16 peak: shapes with more than 128 query "
                                        "rows per KV head sit near the ridge between the two roofs"},
                "traffic": recorded_traffic("tree_attn_tc_kernel", w.name)}
    ver_gbs = wl.rowstats_algorithmic_bytes() / (ver_ms * 1e-3) / 1e9
    lm_tf = (wl.lmhead_algorithmic_flops() + 2 * w.B * w.K * w.d * w.d) / (prop_ms * 1e-3) / 1e12
    phases = {
        "propose": {"ms": prop_ms, "bound": "tensor", "achieved": lm_tf, "peak": peaks["bf16_tflops_sustained"],
                    "unit": "TFLOP/s", "frac": lm_tf / peaks["bf16_tflops_sustained"],
                    "note": "whole call (6 launches); flops = 2*B*K*d*(d+V)"},
        "tree_attn": {"ms": attn_ms, "ms_per_layer": attn_ms / wl.layers, "layers": wl.layers,
                      "tflops": wl.attn_algorithmic_flops() / attn_launch_s / 1e12},
        "verify": {"ms": ver_ms, "bound": "hbm", "achieved": ver_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                   "frac": ver_gbs / peaks["hbm_gbs"], "note": "whole call (%d launches); bytes = logits once" % wl.LAUNCHES_VERIFY},
    }

    a_f, p_f, v_f = phase_fractions(w, wl, prop_ms, attn_ms / wl.layers, ver_ms, peaks)
    phases["tree_attn"].update(bound=a_f["bound"], frac=a_f["frac"], t_mem_us=a_f["t_mem_us"], t_tensor_us=a_f["t_tensor_us"])
    phases["propose"].update(bound=p_f["bound"], frac_of_burst_or_hbm=p_f["frac"])
    if args.paged:
        # committing the accepted paths to every layer's pages (what follows a step in an engine; outside the
        # metric's step).  Repeatable: the workload's lengths are not advanced, the same rows are rewritten.
        len_out = torch.empty_like(wl.kv_len)
        st_word = torch.zeros(1, dtype=torch.int32, device=dev)
        for _ in range(3):
            wl.commit(len_out, st_word)
        c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        c0.record()
        for _ in range(5):
            wl.commit(len_out, st_word)
        c1.record()
        torch.cuda.synchronize()
        rows = int((wl.ver["n_acc"] + 1).sum().item())
        phases["commit"] = {"ms": c0.elapsed_time(c1) / 5, "layers": wl.layers, "tokens_appended": rows,
                            "bytes": rows * wl.layers * 2 * 2 * w.Hkv * w.D * 2, "status": int(st_word.item()),
                            "note": "specroll_commit_path_layers, all layers in one launch; latency-bound (a few MB)"}

    n_layers = wl.layers
    launches = wl.launches_per_step() * args.steps
    headline_entry = {"workload": w.name, "B": w.B, "N": w.N, "rows_per_kv_head": w.N * (w.Hq // w.Hkv),
                      "layers": w.layers, "layers_run": wl.layers, "ms_per_step": tmax / args.steps,
                      "tokens_per_s": value, "attn_us_per_layer": a_f["us_per_layer"], "attn_bound": a_f["bound"],
                      "attn_frac": a_f["frac"], "propose_ms": prop_ms, "propose_bound": p_f["bound"],
                      "propose_frac": p_f["frac"], "verify_ms": ver_ms, "verify_frac": v_f["frac"], "clocks": clocks}
    cfg_line = {"T_kv": wl.T_kv, "top_p": wl.top_p}
    # ---- every other configuration, in the same process: three attention layers each (per-layer time; every layer
    #      has its own cache), the full-depth step put together from the per-call times
    workloads = None
    power_roof = None
    if world == 1 and not args.no_workloads:
        power_roof = measure_power_roof(wl, local)
    if world == 1 and not args.no_workloads:
        from paper_2608_04962_b200 import inputs as I
        del wl
        import gc
        gc.collect()
        torch.cuda.empty_cache()
        workloads = []
        names = ["tiny", "qwen1.5b", "qwen7b", "qwen14b"] + [f"sweep7b_B{b}" for b in (256, 128, 64, 32, 16, 8)]
        for nm in names:
            if nm == w.name and layers == w.layers and not (args.paged or args.top_p or args.lazy_stats):
                # the headline's own numbers (all layers back to back; on the large shapes the board is at its power
                # limit then), and beside them the same calls in a three-layer step like the other entries
                short = measure_workload(I.WORKLOADS[nm], dev, 3, 5, peaks, local)
                headline_entry["three_layer_step"] = {
                    k_: short[k_] for k_ in ("layers_run", "attn_us_per_layer", "attn_bound", "attn_frac", "propose_ms",
                                             "propose_bound", "propose_frac", "verify_ms", "verify_frac", "clocks")}
                headline_entry["three_layer_step"]["note"] = (
                    "the same calls in a step of three attention layers, as for the other entries: no sustained "
                    "load, so not what the full step reaches")
                workloads.append(headline_entry)
            else:
                workloads.append(measure_workload(I.WORKLOADS[nm], dev, 3, 5, peaks, local))
    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        one, ctok, threads, run_layers = oracle_sample_step(w, args.ref_seqs, n_layers, args.ref_layers)
        reps, tt, wall = 0, 0.0, time.perf_counter()
        while reps < 1 or (time.perf_counter() - wall < 10.0 and reps < 8):
            tt += one()
            reps += 1
        cpu = {"value": ctok * reps / tt, "unit": UNIT, "cores": threads, "kind": "oracle",
               "sample": oracle_sample_text(w, args.ref_seqs, n_layers, run_layers) +
                         f"; {reps} passes in {time.perf_counter() - wall:.1f} s"}

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": tmax / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": w.name, "B": w.B, "N": w.N, "K": w.K, "k": w.k, "d": w.d, "V": w.V, "Hq": w.Hq,
                       "Hkv": w.Hkv, "D": w.D, "layers": n_layers, "T_kv": cfg_line["T_kv"], "temperature": w.temperature,
                       "kv_cache": "128-token pages in a seeded random order (specroll_tree_attn_paged)" if args.paged
                       else "contiguous ragged (specroll_tree_attn)",
                       "top_p": cfg_line["top_p"], "lazy_stats": bool(args.lazy_stats), "cuda_graph": graph is not None,
                       "parallelism": f"replicas x{world} (sharded by sequence, no collective)",
                       "l2": "inputs larger than L2: per-layer KV cache, logits and W each exceed 126 MB and every "
                             "layer has its own cache"},
            "clocks": clocks, "e2e": e2e, "e2e_fused": e2e_fused, "gpu_launches": launches,
            "roofline": dict(roofline, power_roof=power_roof), "cpu_baseline": cpu, "phases": phases,
            "accepted": {"aal": aal, "acceptance_rate": ar}, "workloads": workloads}
    print(json.dumps(line), flush=True)
    D.finish()
    return 0


def run_e2e(args, wl, dev, world, fused=False):
    """The same step driven from HOST buffers: per-step activations (hidden state, Reflex memory, uniforms,
    every layer's Q and tree K/V, target logits) are copied from pinned memory inside the timed region and
    the step's results are read back.  Weights and the KV cache are resident state.
    fused: the target's final hidden states [B, N, d] are uploaded instead of its logits [B, N, V], and the
    verification is specroll's fused form (vocabulary projection with the row statistics in its epilogue, sparse
    walk, terminal rows), so the logits never cross PCIe or reach HBM."""
    import torch
    from paper_2608_04962_b200 import binding as S
    from paper_2608_04962_b200 import dist as D
    w = wl.w
    host_in = {}
    if fused:
        gen = torch.Generator(device=dev)
        gen.manual_seed(11)
        wl.hidden = (0.02 * torch.randn((w.B, w.N, w.d), generator=gen, device=dev)).to(torch.bfloat16)

    def pin(t):
        h = torch.empty(t.shape, dtype=t.dtype, pin_memory=True)
        h.copy_(t)
        return h

    big = "hidden" if fused else "logits"
    names = ["h", "anchor", "m", "alpha", "u_draw", "u_acc", "u_fin", big]
    for n in names:
        host_in[n] = pin(getattr(wl, n))
    hQ = [pin(t) for t in wl.Q]
    hKt = [pin(t) for t in wl.Kt]
    hVt = [pin(t) for t in wl.Vt]
    out_names_p = ["cand_id", "cand_logit", "tree_tok", "tree_cand", "slot_q"]
    out_names_v = ["n_acc", "path_node", "out_tok", "term_node", "term_kind"]
    host_out = {n: torch.empty(wl.prop[n].shape, dtype=wl.prop[n].dtype, pin_memory=True) for n in out_names_p}
    host_out.update({n: torch.empty(wl.ver[n].shape, dtype=wl.ver[n].dtype, pin_memory=True) for n in out_names_v})
    hO = [torch.empty(t.shape, dtype=t.dtype, pin_memory=True) for t in wl.O]
    h2d = sum(t.numel() * t.element_size() for t in list(host_in.values()) + hQ + hKt + hVt)
    d2h = sum(t.numel() * t.element_size() for t in list(host_out.values()) + hO)

    # Three streams: uploads, the kernels, downloads.  A kernel waits only for the upload of its own inputs, so
    # the bulk of the bytes (target logits, needed last) crosses PCIe while the proposal and the attention layers
    # run, and results go back while later layers compute (the link is full duplex).
    s_cmp = torch.cuda.current_stream(dev)
    s_in, s_out = torch.cuda.Stream(dev), torch.cuda.Stream(dev)
    n_ev = 2 * wl.layers + 4
    evs = [torch.cuda.Event() for _ in range(n_ev)]

    def step():
        ev = iter(evs)
        small = [n for n in names if n != big]
        with torch.cuda.stream(s_in):
            for n in small:
                getattr(wl, n).copy_(host_in[n], non_blocking=True)
            e_small = next(ev)
            e_small.record(s_in)
            e_layer = []
            for l in range(wl.layers):
                wl.Q[l].copy_(hQ[l], non_blocking=True)
                wl.Kt[l].copy_(hKt[l], non_blocking=True)
                wl.Vt[l].copy_(hVt[l], non_blocking=True)
                e = next(ev)
                e.record(s_in)
                e_layer.append(e)
            getattr(wl, big).copy_(host_in[big], non_blocking=True)
            e_logits = next(ev)
            e_logits.record(s_in)
        s_cmp.wait_event(e_small)
        wl.propose()
        e = next(ev)
        e.record(s_cmp)
        with torch.cuda.stream(s_out):
            s_out.wait_event(e)
            for n in out_names_p:
                host_out[n].copy_(wl.prop[n], non_blocking=True)
        for l in range(wl.layers):
            s_cmp.wait_event(e_layer[l])
            wl.attn(l)
            e = next(ev)
            e.record(s_cmp)
            with torch.cuda.stream(s_out):
                s_out.wait_event(e)
                hO[l].copy_(wl.O[l], non_blocking=True)
        s_cmp.wait_event(e_logits)
        if fused:
            p = wl.prop
            fv = S.verify_fused(wl.hidden, wl.W, wl.parent, p["tree_tok"], p["tree_cand"], p["cand_id"], p["cand_logit"],
                                wl.u_acc, wl.u_fin, temperature=w.temperature)
            for n in out_names_v:
                wl.ver[n].copy_(fv[n])
        else:
            wl.verify()
        e = next(ev)
        e.record(s_cmp)
        with torch.cuda.stream(s_out):
            s_out.wait_event(e)
            for n in out_names_v:
                host_out[n].copy_(wl.ver[n], non_blocking=True)

    steps = max(2, min(args.steps, 5))
    step()
    torch.cuda.synchronize()
    D.barrier()
    t0 = time.perf_counter()
    for _ in range(steps):
        step()
        torch.cuda.synchronize()      # the host holds the step's result before the next step starts
    dt = time.perf_counter() - t0
    D.barrier()
    tmax, tok = D.aggregate(dt * 1e3, wl.tokens_per_step() * steps, device=dev)
    out = {"value": tok / (tmax * 1e-3), "unit": UNIT, "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
           "ms_per_step": tmax / steps, "steps": steps}
    if fused:
        out["note"] = ("hidden states uploaded instead of target logits; verification = projection with fused row "
                       "statistics + sparse walk + terminal rows (the projection's 2 B (N+1) d V FLOP are inside the step)")
    return out


def run_calls(args, w, layers):
    """Per-call timings, each entry point alone: 20 warm-up + 100 timed launches with CUDA events, median and
    minimum; once with a 256 MB write between launches (cold L2: the roofline number) and once back to back.
    Prints one JSON object (not the bench line)."""
    import torch
    from paper_2608_04962_b200.workload import StepWorkload
    from paper_2608_04962_b200 import binding as S
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback of the hot path")
    S.lib()
    dev = torch.device("cuda", 0)
    wl = StepWorkload(w, dev, layers=min(layers, 2), paged=args.paged, top_p=args.top_p)
    peaks = measured_peaks()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    wl.step()

    def attn_planned():
        wl.attn(0)

    def attn_reuse():
        wl.attn(1)

    # the proposal streams W once; with fewer than 253 rows (B K) in the projection that stream, not the tensor
    # pipe, is what bounds it
    if w.B * w.K >= 253:
        propose_call = (wl.propose, "tensor", (wl.lmhead_algorithmic_flops() + 2 * w.B * w.K * w.d * w.d) / 1e12,
                        peaks["bf16_tflops"], "TFLOP/s")
    else:
        propose_call = (wl.propose, "hbm", (wl.lmhead_algorithmic_bytes() + wl.heads_algorithmic_bytes()) / 1e9,
                        peaks["hbm_gbs"], "GB/s")
    calls = {
        "propose": propose_call,
        "tree_attn (plan kernel + attention)": (attn_planned, "hbm", wl.attn_algorithmic_bytes() / 1e9,
                                                peaks["hbm_gbs"], "GB/s"),
        "tree_attn (plan reused)": (attn_reuse, "hbm", wl.attn_algorithmic_bytes() / 1e9, peaks["hbm_gbs"], "GB/s"),
        "verify": (wl.verify, "hbm", wl.rowstats_algorithmic_bytes() / 1e9, peaks["hbm_gbs"], "GB/s"),
    }
    # the feedback call on one matured record per (sequence, head): a node of the matching depth, a random realised token
    R = w.B * w.K
    gen = torch.Generator(device=dev)
    gen.manual_seed(5)
    depth = np.zeros(w.N, np.int64)
    for n in range(1, w.N):
        depth[n] = depth[wl.parent[n]] + 1
    node_of_head = [int(np.flatnonzero(depth == min(h, depth.max()))[0]) for h in range(w.K)]
    rec_row = (torch.arange(w.B, device=dev)[:, None] * w.N +
               torch.tensor(node_of_head, device=dev)[None, :]).reshape(-1).to(torch.int32).contiguous()
    rec_mem = torch.arange(R, device=dev, dtype=torch.int32)
    y_star = torch.randint(0, w.V, (R,), generator=gen, device=dev, dtype=torch.int32)
    rho = torch.full((R,), 0.9, device=dev)
    mem = wl.m.reshape(R, w.d).clone()
    k_support = 48
    fb_ws = torch.empty(S.reflex_feedback_workspace_bytes(R, w.k, k_support, w.d, w.V, w.temperature), dtype=torch.uint8,
                        device=dev)
    cid = wl.prop["cand_id"].reshape(R, w.k).contiguous()
    clg = wl.prop["cand_logit"].reshape(R, w.k).contiguous()
    rmax = wl.ver["row_max"].reshape(-1).contiguous()
    rsum = wl.ver["row_sum"].reshape(-1).contiguous()

    def feedback():
        S.reflex_feedback(wl.logits, rec_row, rmax, rsum, cid, clg, y_star, wl.W, rho, rec_mem, mem, k_support,
                          temperature=w.temperature, workspace=fb_ws)

    fb_bytes = (R * w.V * 2 + R * (w.k + k_support + 1) * w.d * 2 + 2 * R * w.d * 4) / 1e9
    calls["reflex_feedback (B K records, support 48)"] = (feedback, "hbm", fb_bytes, peaks["hbm_gbs"], "GB/s")
    # reliability side: sketches (rank 24) of the R feedback vectors, then alignments, online moments and the gate
    # of the R slots (one record per slot here)
    rank = 24
    Pi = torch.randn((rank, w.d), generator=gen, device=dev)
    e_vec = torch.randn((R, w.d), generator=gen, device=dev)
    s_sk = S.reflex_sketch(mem, Pi)
    xi_sk = S.reflex_sketch(e_vec, Pi)
    slot = torch.arange(R, device=dev, dtype=torch.int32)
    st_n = torch.zeros(R, dtype=torch.int32, device=dev)
    st_fb = torch.zeros(R, dtype=torch.int32, device=dev)
    st_mean = torch.zeros(R, device=dev)
    st_M2 = torch.zeros(R, device=dev)
    hz = (torch.arange(R, device=dev) % w.K).to(torch.int32)
    n_al = torch.tensor([6, 16, 48, 48, 48][: w.K], dtype=torch.int32, device=dev)
    n_fbm = torch.tensor([1, 2, 4, 4, 4][: w.K], dtype=torch.int32, device=dev)
    a_lo = torch.tensor([0.010, 0.004, 0.0025, 0.0025, 0.0025][: w.K], device=dev)
    a_hi = torch.tensor([0.025, 0.010, 0.0060, 0.0060, 0.0060][: w.K], device=dev)

    def sketch():
        S.reflex_sketch(e_vec, Pi)

    def gate():
        S.reflex_gate(s_sk, xi_sk, slot, None, st_n, st_mean, st_M2, st_fb, mem, hz, n_al, n_fbm, a_lo, a_hi)

    calls["reflex_sketch (B K vectors, rank 24)"] = (sketch, "hbm", (R * w.d * 4 + rank * w.d * 4 + R * rank * 4) / 1e9,
                                                     peaks["hbm_gbs"], "GB/s")
    calls["reflex_gate (B K records, B K slots)"] = (gate, "hbm", (R * w.d * 4 + 2 * R * rank * 4 + 8 * R * 4) / 1e9,
                                                    peaks["hbm_gbs"], "GB/s")
    # the target projection with fused row statistics over all (sequence, node) rows, and its storing form on one
    # row per sequence (the terminal rows)
    hid = (0.02 * torch.randn((w.B * w.N, w.d), generator=gen, device=dev)).to(torch.bfloat16)
    want = wl.prop["cand_id"][:, 0, :].repeat_interleave(w.N, dim=0).contiguous()[:, : min(w.k, 8)].contiguous()
    th_ws = torch.empty(S.lib().specroll_target_head_stats_workspace_bytes(w.B * w.N, w.d, w.V) + 256,
                        dtype=torch.uint8, device=dev)
    rows_out = torch.empty((w.B, w.V), dtype=torch.bfloat16, device=dev)

    def head_stats():
        S.target_head_stats(hid, wl.W, want, temperature=w.temperature, workspace=th_ws)

    def head_rows():
        S.target_head_rows(hid[: w.B], wl.W, out=rows_out)

    hid3 = hid.reshape(w.B, w.N, w.d)
    p_ = wl.prop

    def verify_from_hidden():
        S.verify_fused(hid3, wl.W, wl.parent, p_["tree_tok"], p_["tree_cand"], p_["cand_id"][:, :, : min(w.k, 8)].contiguous(),
                       p_["cand_logit"][:, :, : min(w.k, 8)].contiguous(), wl.u_acc, wl.u_fin, temperature=w.temperature)

    if w.k <= 8:
        calls["verify_fused (projection + statistics + walk + terminal rows, from hidden states)"] = (
            verify_from_hidden, "tensor", 2.0 * w.B * (w.N + 1) * w.d * w.V / 1e12, peaks["bf16_tflops"], "TFLOP/s")
    calls["target_head_stats (B N rows, fused statistics)"] = (
        head_stats, "tensor", 2.0 * w.B * w.N * w.d * w.V / 1e12, peaks["bf16_tflops"], "TFLOP/s")
    calls["target_head_rows (B rows stored)"] = (
        head_rows, "hbm", (w.V * w.d * 2 + w.B * w.V * 2) / 1e9, peaks["hbm_gbs"], "GB/s")
    out = {"workload": w.name, "peak_source": peaks["source"], "calls": {}}
    for name, (fn, bound, work, peak, unit) in calls.items():
        rec = {"bound": bound, "unit": unit, "peak": peak, "work_per_call": work}
        for mode in ("cold_l2", "back_to_back"):
            for _ in range(20):
                fn()
            evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(100)]
            for a, b in evs:
                if mode == "cold_l2":
                    flush.fill_(1)
                a.record()
                fn()
                b.record()
            torch.cuda.synchronize()
            t = np.array([a.elapsed_time(b) for a, b in evs])
            med, mn = float(np.median(t)), float(t.min())
            rec[mode] = {"median_us": med * 1e3, "min_us": mn * 1e3, "achieved_median": work / (med * 1e-3),
                         "frac_median": work / (med * 1e-3) / peak}
        out["calls"][name] = rec
    print(json.dumps(out), flush=True)
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="qwen14b",
                    help="default: the largest single-GPU configuration (63 GB of KV cache over 48 layers)")
    ap.add_argument("--layers", type=int, default=None, help="attention layers per step (default: the model's)")
    ap.add_argument("--ref-seqs", type=int, default=2, help="sequences per CPU-oracle sample step")
    ap.add_argument("--ref-layers", type=int, default=2,
                    help="attention layers the CPU oracle runs per sample step (its time is scaled to the shape's depth)")
    ap.add_argument("--no-workloads", action="store_true",
                    help="skip the per-configuration array (every other configuration, three layers each)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling runs)")
    ap.add_argument("--top-p", type=float, default=None,
                    help="verify against nucleus-truncated target distributions (specroll_verify_nucleus); the "
                         "metric's step uses the plain temperature softmax (default)")
    ap.add_argument("--lazy-stats", action="store_true",
                    help="softmax statistics of the visited nodes only (SPECROLL_VERIFY_LAZY_STATS); the metric's step "
                         "evaluates every node (default)")
    ap.add_argument("--paged", action="store_true",
                    help="keep the KV cache in 128-token pages (specroll_tree_attn_paged) and time the commit of the "
                         "accepted paths after the step as well (reported beside the step, not inside it)")
    ap.add_argument("--graph", action="store_true",
                    help="capture the step in a CUDA graph and time replays instead of plain launches (the phase "
                         "times and the roofline line then come from plain steps run afterwards)")
    ap.add_argument("--chw", action="store_true",
                    help="profile the verification capacity C_hw of Eq. verification-budget for the workload's shape "
                         "(sweeps batch size and nodes per sequence; prints one JSON object)")
    ap.add_argument("--calls", action="store_true",
                    help="time each entry point alone (100 launches, cold and warm L2) instead of the step")
    args = ap.parse_args()
    from paper_2608_04962_b200 import dist as D
    from paper_2608_04962_b200 import inputs as I
    kind, msg = D.launch_plan(args.gpus)
    if kind == "refuse":
        print("bench.py: " + msg, file=sys.stderr)
        return 2
    if kind == "spawn":
        # replicas: one process per GPU, started here when no launcher did it
        import socket
        sk = socket.socket()
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
        sk.close()
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
               "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
        return subprocess.call(cmd)
    w = I.WORKLOADS[args.workload]
    layers = args.layers if args.layers is not None else w.layers
    if args.impl == "reference":
        return run_reference(args, w, layers)
    if args.calls:
        return run_calls(args, w, layers)
    if args.chw:
        import torch
        from paper_2608_04962_b200 import binding as S
        from paper_2608_04962_b200 import chw
        if not torch.cuda.is_available():
            raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback of the hot path")
        torch.cuda.set_device(0)
        res = chw.profile(w, Bs=(256, 128, 64, 32, 16), Ns=(4, 8, 12, 16, 24, 32, 48, 64),
                          device=torch.device("cuda", 0), warmup=args.warmup, steps=max(2, min(args.steps, 5)))
        res["node_budget"] = {str(B): S.node_budget(res["C_hw"], B, 4, 64) for B in (256, 128, 64, 32, 16, 8)}
        print(json.dumps(res), flush=True)
        return 0
    return run_ours(args, w, layers)


if __name__ == "__main__":
    sys.exit(main())
