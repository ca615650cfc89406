"""Seeded synthetic inputs shaped like the workloads the method is measured on.

This module only draws numbers: it holds none of the method's arithmetic and
is the one piece shared by the CUDA path's callers and the CPU oracle's
callers (both sides are handed the same bits).

Recipe (every config): q, k, v ~ N(0, 1); gates g = sigmoid(x) with
x ~ N(mean 4.12, sd 0.5) per token, head and channel, so that the mean gate is
about 0.984 and the memory length 1/(1-g) is about 64 tokens.  Values are drawn
in fp32 with a torch generator seeded from (seed, stream id) and cast to the
I/O dtype; draw order is q, k, v, x.  Two configs add structure:
  * "resets": each token (b, t) is, with probability 1 %, given g = 0.5 on all
    heads and channels (a reset-like token);
  * "needles": per (b, h), 8 distinct pages from [1, P-2] get their raw keys
    shifted by 2 * q/|q| (two standard deviations of a raw key along the decode
    query's direction) before the recurrence.
"""
from __future__ import annotations

import dataclasses
import math

import torch


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    B: int
    H: int
    D: int
    T: int                 # context length (tokens in the cache when the query attends)
    S: int = 16
    budget_num: int = 1    # budget = budget_num / budget_den of the pages
    budget_den: int = 16
    dtype: torch.dtype = torch.bfloat16
    gate_dtype: torch.dtype | None = None
    seed: int = 0
    steps: int = 1         # consecutive decode steps
    resets: bool = False
    needles: int = 0
    gate_zero: bool = False   # g = 0 everywhere: the cache holds k and v themselves (Eq. 2's paired baseline)

    @property
    def gdtype(self):
        return self.gate_dtype or self.dtype

    def pages(self, T=None):
        T = self.T if T is None else T
        return (T + self.S - 1) // self.S

    def budget_pages(self, T=None):
        """K = ceil(P * budget) for the context length at hand."""
        return max(1, math.ceil(self.pages(T) * self.budget_num / self.budget_den))


# The five configurations the benchmark definition lists, in its order.
CONFIGS = {
    0: Workload("tiny-fp32", B=1, H=4, D=64, T=1024, budget_den=4, dtype=torch.float32, seed=0),
    1: Workload("7b-layer-16k", B=1, H=32, D=128, T=16384, budget_den=16, seed=1),
    2: Workload("batched-multistep-32k", B=8, H=32, D=128, T=32768, budget_den=8, seed=2, steps=64),
    3: Workload("prefill-128k", B=1, H=32, D=128, T=131072, budget_den=16, seed=3, resets=True),
    4: Workload("needles-128k", B=4, H=32, D=128, T=131072, budget_den=16, seed=4, needles=8),
}
# The configuration the headline metric is quoted on: config 4's shapes at batch 1.
METRIC = dataclasses.replace(CONFIGS[4], name="decode-128k-b1", B=1)


def _gen(device, seed, stream):
    g = torch.Generator(device=device)
    g.manual_seed(seed * 1000003 + stream)
    return g


def make_query(w: Workload, device, step=0):
    """q for decode step `step`: [B, H, D] in the I/O dtype."""
    q = torch.randn(w.B, w.H, w.D, generator=_gen(device, w.seed, 10 + 4 * step), device=device,
                    dtype=torch.float32)
    return q.to(w.dtype)


def make_token(w: Workload, device, step=0):
    """(k_t, v_t, g_t) appended by decode step `step`: each [B, H, D]."""
    k = torch.randn(w.B, w.H, w.D, generator=_gen(device, w.seed, 11 + 4 * step), device=device)
    v = torch.randn(w.B, w.H, w.D, generator=_gen(device, w.seed, 12 + 4 * step), device=device)
    x = torch.randn(w.B, w.H, w.D, generator=_gen(device, w.seed, 13 + 4 * step), device=device)
    g = torch.zeros_like(x) if w.gate_zero else torch.sigmoid(4.12 + 0.5 * x)
    return k.to(w.dtype), v.to(w.dtype), g.to(w.gdtype)


def needle_pages(w: Workload, T=None):
    """[B, H, needles] int64 page indices (CPU), distinct per (b, h), from [1, P-2]."""
    P = w.pages(T)
    g = _gen("cpu", w.seed, 3)
    out = torch.empty(w.B, w.H, w.needles, dtype=torch.int64)
    for b in range(w.B):
        for h in range(w.H):
            out[b, h] = torch.randperm(P - 2, generator=g)[: w.needles] + 1
    return out


def make_prefill(w: Workload, device, T=None, q_for_needles=None):
    """(k, v, g) for the prefilled context: each [B, T, H, D].

    Built one batch item at a time so that the fp32 temporaries stay small.
    For a needle workload, pass the decode query the needles should align with.
    """
    T = w.T if T is None else T
    k = torch.empty(w.B, T, w.H, w.D, dtype=w.dtype, device=device)
    v = torch.empty_like(k)
    g = torch.empty(w.B, T, w.H, w.D, dtype=w.gdtype, device=device)
    gk, gv, gx = (_gen(device, w.seed, s) for s in (0, 1, 2))
    reset_gen = _gen("cpu", w.seed, 4)
    pages = needle_pages(w, T) if w.needles else None
    for b in range(w.B):
        kb = torch.randn(T, w.H, w.D, generator=gk, device=device)
        if w.needles:
            qh = q_for_needles[b].to(torch.float32)
            qh = qh / qh.norm(dim=-1, keepdim=True)                     # [H, D]
            kb = kb.view(-1, w.S, w.H, w.D) if T % w.S == 0 else kb
            for h in range(w.H):
                for p in pages[b, h].tolist():
                    if T % w.S == 0:
                        kb[p, :, h, :] += 2.0 * qh[h]
                    else:
                        kb[p * w.S:(p + 1) * w.S, h, :] += 2.0 * qh[h]
            kb = kb.view(T, w.H, w.D)
        k[b] = kb.to(w.dtype)
        del kb
        v[b] = torch.randn(T, w.H, w.D, generator=gv, device=device).to(w.dtype)
        gb = torch.sigmoid(4.12 + 0.5 * torch.randn(T, w.H, w.D, generator=gx, device=device))
        if w.resets:
            hit = (torch.rand(T, generator=reset_gen) < 0.01).to(device)
            gb[hit] = 0.5
        if w.gate_zero:
            gb.zero_()
        g[b] = gb.to(w.gdtype)
        del gb
    return k, v, g
