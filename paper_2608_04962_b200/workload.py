"""Device-resident synthetic workload of one speculative step, and the step itself.

A step is: specroll_propose -> specroll_tree_attn for every layer of the named model shape ->
specroll_verify.  Tensors are drawn on the device with a seeded torch generator using the same
distributions as ``inputs`` (the host generators are too slow for the multi-GB tensors of the
full-size shapes); KV lengths and the tree topology come from ``inputs`` unchanged.
"""
from __future__ import annotations

from typing import Dict, List

import numpy as np
import torch

from . import binding as S
from . import inputs as I


def _randn_bf16(gen, shape, std, device):
    n = int(np.prod(shape))
    out = torch.empty(n, dtype=torch.bfloat16, device=device)
    step = 1 << 26
    for lo in range(0, n, step):            # bounded fp32 staging
        hi = min(n, lo + step)
        t = torch.randn(hi - lo, generator=gen, device=device, dtype=torch.float32)
        if std != 1.0:
            t.mul_(std)
        out[lo:hi] = t.to(torch.bfloat16)
    return out.view(*shape)


class StepWorkload:
    """All tensors of one step for workload ``w`` on ``device`` (seed offset for replicas)."""

    def __init__(self, w: I.Workload, device, seed: int = 0, layers: int | None = None, paged: bool = False,
                 top_p: float | None = None, lazy_stats: bool = False):
        self.w = w
        self.verify_flags = S.VERIFY_LAZY_STATS if lazy_stats else 0
        self.lazy_stats = bool(lazy_stats)
        self.paged = bool(paged)
        self.top_p = top_p if (top_p is not None and 0.0 < top_p < 1.0) else None
        self.device = device
        self.layers = int(layers if layers is not None else w.layers)
        gen = torch.Generator(device=device)
        gen.manual_seed(1000 * w.cfg_id + 17 + seed)
        B, N, K, k, d, V = w.B, w.N, w.K, w.k, w.d, w.V
        self.parent = I.topology(w)
        L = I.kv_lengths(w)
        self.kv_indptr_host = np.zeros(B + 1, np.int32)
        np.cumsum(L, out=self.kv_indptr_host[1:])
        self.T_kv = int(self.kv_indptr_host[-1])
        self.kv_indptr = torch.from_numpy(self.kv_indptr_host).to(device)
        # proposal
        self.A = _randn_bf16(gen, (K, d, d), 0.02, device)
        self.bias = _randn_bf16(gen, (K, d), 0.02, device)
        self.W = _randn_bf16(gen, (V, d), 0.02, device)
        self.h = _randn_bf16(gen, (B, d), 0.02, device)
        self.anchor = torch.randint(0, V, (B,), generator=gen, device=device, dtype=torch.int32)
        self.m = torch.randn((B, K, d), generator=gen, device=device, dtype=torch.float32)
        ah = torch.zeros(K, device=device)
        ah[:len(w.alpha_heads)] = torch.tensor(w.alpha_heads[:K], device=device)
        on = (torch.rand((B, K), generator=gen, device=device) < 0.5).float()
        self.alpha = (on * ah[None, :]).contiguous()
        self.u_draw = torch.rand((B, N), generator=gen, device=device, dtype=torch.float32)
        self.u_acc = torch.rand((B, N), generator=gen, device=device, dtype=torch.float32)
        self.u_fin = torch.rand((B,), generator=gen, device=device, dtype=torch.float32)
        # attention, one set per layer (each layer's cache is larger than L2)
        self.Q: List[torch.Tensor] = []
        self.Kc: List[torch.Tensor] = []
        self.Vc: List[torch.Tensor] = []
        self.Kt: List[torch.Tensor] = []
        self.Vt: List[torch.Tensor] = []
        for _ in range(self.layers):
            self.Q.append(_randn_bf16(gen, (B, N, w.Hq, w.D), 1.0, device))
            self.Kc.append(_randn_bf16(gen, (self.T_kv, w.Hkv, w.D), 1.0, device))
            self.Vc.append(_randn_bf16(gen, (self.T_kv, w.Hkv, w.D), 1.0, device))
            self.Kt.append(_randn_bf16(gen, (B, N, w.Hkv, w.D), 1.0, device))
            self.Vt.append(_randn_bf16(gen, (B, N, w.Hkv, w.D), 1.0, device))
        self.O = [S.alloc((B, N, w.Hq, w.D), dtype=torch.bfloat16, device=device)
                  for _ in range(self.layers)]
        if self.paged:
            # the same caches scattered into pools of 128-token pages in a seeded random page order, with room
            # for one more committed path per sequence; the contiguous copies are dropped
            PAGE = S.PAGE_TOKENS
            own = (L.astype(np.int64) + (K + 1) + PAGE - 1) // PAGE
            pi = np.zeros(B + 1, np.int32)
            np.cumsum(own, out=pi[1:])
            self.n_pages = int(pi[-1]) + 3
            pt = I.rng(1000 * w.cfg_id + 31 + seed).permutation(self.n_pages)[: int(pi[-1])].astype(np.int32)
            tok = np.arange(self.T_kv, dtype=np.int64)
            seq = np.repeat(np.arange(B), L)
            t_in = tok - self.kv_indptr_host[:-1].astype(np.int64)[seq]
            flat = pt[pi[:-1].astype(np.int64)[seq] + t_in // PAGE].astype(np.int64) * PAGE + t_in % PAGE
            flat_d = torch.from_numpy(flat).to(device)
            self.page_table = torch.from_numpy(pt).to(device)
            self.page_indptr = torch.from_numpy(pi).to(device)
            self.kv_len_host = L.astype(np.int32)
            self.kv_len = torch.from_numpy(self.kv_len_host).to(device)
            self.Kp, self.Vp = [], []
            for l in range(self.layers):
                for src, dst in ((self.Kc, self.Kp), (self.Vc, self.Vp)):
                    pool = torch.zeros((self.n_pages * PAGE, w.Hkv, w.D), dtype=torch.bfloat16, device=device)
                    pool[flat_d] = src[l]
                    dst.append(pool.view(self.n_pages, PAGE, w.Hkv, w.D))
                    src[l] = None
        # workspaces and outputs, allocated once
        self.ws_propose = S.alloc(S.propose_workspace_bytes(B, N, K, k, d, V, w.temperature),
                                      dtype=torch.uint8, device=device)
        ws_bytes = (S.tree_attn_paged_workspace_bytes(B, N, w.Hq, w.Hkv, w.D, self.kv_len_host) if self.paged else
                    S.tree_attn_workspace_bytes(B, N, w.Hq, w.Hkv, w.D, self.kv_indptr_host))
        self.ws_attn = S.alloc(ws_bytes, dtype=torch.uint8, device=device)
        self.ws_verify = S.alloc(max(S.verify_nucleus_workspace_bytes(B, N, K, k, V, w.temperature),
                                     S.verify_workspace_bytes(B, N, K, k, V, w.temperature)),
                                 dtype=torch.uint8, device=device)
        self.prop = None
        self.ver = None
        # target logits: N(0,1) background, one mode token per node boosted by +14
        # (first child w.p. 0.45, second child w.p. 0.15, else a random token)
        self.propose()
        tok = self.prop["tree_tok"].long()
        self.logits = _randn_bf16(gen, (B, N, V), 1.0, device)
        kids = [[] for _ in range(N)]
        for n in range(1, N):
            kids[int(self.parent[n])].append(n)
        pick = torch.rand((B, N), generator=gen, device=device)
        mode = torch.randint(0, V, (B, N), generator=gen, device=device)
        for n in range(N):
            if len(kids[n]) >= 1:
                sel = pick[:, n] < 0.45
                mode[sel, n] = tok[sel, kids[n][0]]
            if len(kids[n]) >= 2:
                sel = (pick[:, n] >= 0.45) & (pick[:, n] < 0.60)
                mode[sel, n] = tok[sel, kids[n][1]]
        idx = mode.unsqueeze(-1)
        boosted = self.logits.gather(2, idx).float() + 14.0
        self.logits.scatter_(2, idx, boosted.to(torch.bfloat16))
        torch.cuda.synchronize(device)

    # ---- the three calls
    def propose(self):
        w = self.w
        self.prop = S.propose(self.h, self.anchor, self.A, self.bias, self.W, self.m, self.alpha, self.parent,
                              self.u_draw, k=w.k, temperature=w.temperature, clip_c=w.clip_c,
                              workspace=self.ws_propose, out=self.prop)
        return self.prop

    def attn(self, layer: int):
        # every layer of a step sees the same KV lengths: layers after the first reuse the work plan, and the
        # caches were all written before the step began
        later = S.ATTN_REUSE_PLAN | S.ATTN_CACHE_SETTLED
        if self.paged:
            return S.tree_attn_paged(self.Q[layer], self.Kp[layer], self.Vp[layer], self.page_table, self.page_indptr,
                                     self.kv_len, self.kv_len_host, self.Kt[layer], self.Vt[layer], self.parent,
                                     workspace=self.ws_attn, out=self.O[layer],
                                     flags=later if layer > 0 else 0)
        return S.tree_attn(self.Q[layer], self.Kc[layer], self.Vc[layer], self.kv_indptr, self.kv_indptr_host,
                           self.Kt[layer], self.Vt[layer], self.parent, workspace=self.ws_attn,
                           out=self.O[layer], flags=later if layer > 0 else 0)

    def commit(self, kv_len_out=None, status=None):
        """Appends the committed paths of the last verification to every layer's paged cache (the workload's
        own lengths are left alone, so that the step can be repeated)."""
        S.commit_path_layers(self.Kt, self.Vt, self.ver["path_node"], self.ver["n_acc"], self.Kp, self.Vp,
                             self.page_table, self.page_indptr, self.kv_len, kv_len_out=kv_len_out, status=status)

    def verify(self):
        p = self.prop
        if self.top_p is not None:
            self.ver = S.verify_nucleus(self.logits, self.parent, p["tree_tok"], p["tree_cand"], p["cand_id"],
                                        p["cand_logit"], self.u_acc, self.u_fin, self.top_p,
                                        temperature=self.w.temperature, workspace=self.ws_verify, out=self.ver,
                                        flags=self.verify_flags)
            return self.ver
        self.ver = S.verify(self.logits, self.parent, p["tree_tok"], p["tree_cand"], p["cand_id"],
                            p["cand_logit"], self.u_acc, self.u_fin, temperature=self.w.temperature,
                            workspace=self.ws_verify, out=self.ver, flags=self.verify_flags)
        return self.ver

    def step(self, events=None):
        """One pass of the hot path.  ``events``: optional 4 CUDA events recorded at the phase edges."""
        if events:
            events[0].record()
        self.propose()
        if events:
            events[1].record()
        for layer in range(self.layers):
            self.attn(layer)
        if events:
            events[2].record()
        self.verify()
        if events:
            events[3].record()

    # ---- bookkeeping for the report
    LAUNCHES_PROPOSE = 6   # kernels per call: layernorm, heads, correction, projection, merge, draw

    @property
    def LAUNCHES_VERIFY(self) -> int:
        # plain verification with all rows' statistics: the statistics kernel, then walk + terminal draw in one;
        # with a nucleus: statistics, thresholds of the nodes with children, walk, draw; statistics of the visited
        # rows only: walk, draw
        if self.lazy_stats:
            return 2
        return 4 if self.top_p is not None else 2

    def launches_per_step(self) -> int:
        # the library says how many kernels an attention call enqueues: the plan kernel runs for the first layer
        # only (the plan is reused afterwards), a merge kernel only when a sequence is cut into many chunks
        w = self.w
        first = S.tree_attn_launches(w.B, w.N, w.Hq, w.Hkv, w.D, self.kv_indptr_host)
        later = S.tree_attn_launches(w.B, w.N, w.Hq, w.Hkv, w.D, self.kv_indptr_host, flags=S.ATTN_REUSE_PLAN)
        return self.LAUNCHES_PROPOSE + first + (self.layers - 1) * later + self.LAUNCHES_VERIFY

    def tokens_per_step(self) -> int:
        return self.w.B * self.w.N

    def attn_algorithmic_bytes(self) -> int:
        """Per layer: every cached K and V element once, plus Q, O and the tree K/V rows."""
        w = self.w
        return self.T_kv * w.Hkv * w.D * 2 * 2 + w.B * w.N * (2 * w.Hq + 2 * w.Hkv) * w.D * 2

    def attn_algorithmic_flops(self) -> int:
        w = self.w
        return 4 * w.D * w.Hq * w.N * (self.T_kv + w.B * (w.N + 1) // 2)

    def rowstats_algorithmic_bytes(self) -> int:
        w = self.w
        return w.B * w.N * w.V * 2 + w.B * w.N * 8

    def lmhead_algorithmic_flops(self) -> int:
        w = self.w
        return 2 * w.B * w.K * w.d * w.V

    def heads_algorithmic_bytes(self) -> int:
        w = self.w
        return w.K * w.d * w.d * 2

    def lmhead_algorithmic_bytes(self) -> int:
        w = self.w
        return w.V * w.d * 2
