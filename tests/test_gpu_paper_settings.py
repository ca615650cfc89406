"""GPU parity at the paper's own Quest settings (App. A.1: 4K context, block 64 with K in
{16, 8, 4} kept pages, and block 16 with K = 4), each on the decayed states and on the paired
g = 0 baseline of Eq. 2, and the mechanics of the paper's two selection hypotheses (Sec. 2.3) on
synthetic planted pages: strict head-level hit rate of the query-aware selection against a
uniform random selector."""
import dataclasses

import numpy as np
import pytest
import torch

import paper_2605_28640_b200 as rq
from paper_2605_28640_b200 import selectors, workloads as wl

import parity
from test_gpu_parity import run_case

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.mark.parametrize("gate_zero", [False, True])
@pytest.mark.parametrize("S,K", [(64, 16), (64, 8), (64, 4), (16, 4)])
def test_quest_block_and_budget_of_the_paper(S, K, gate_zero):
    w = wl.Workload("quest-4k", B=1, H=4, D=128, T=4096, S=S, seed=300 + S + K, gate_zero=gate_zero)
    stats = {}
    run_case(w, w.T - 2, steps=2, budget=K, stats=stats)
    assert stats["heads"] == 2 * w.H
    assert stats.get("near_tie_mismatch", 0) <= stats.get("near_tie", 0)


def test_hit_rate_of_query_aware_and_random_selection():
    """One golden page per head is planted to align with the common direction of the decode queries of three steps.  The
    query-aware selection must keep it at every step (Hit_h = 1) for almost every head; a uniform
    random K-subset keeps it with probability (K / P)^steps.  The attention over the random pages
    is checked against the oracle on the same pages."""
    steps, S, T0 = 3, 16, 4096 - 3
    w = wl.Workload("hits", B=2, H=8, D=128, T=T0 + steps, S=S, budget_den=16, seed=41)
    P0 = w.pages(T0)
    gen = torch.Generator().manual_seed(5)
    gold = torch.randint(1, P0 - 2, (w.B, w.H), generator=gen)                  # not a forced page
    # the queries of consecutive steps look for the same thing: a common direction plus step noise
    q0 = wl.make_query(w, DEV, 0).float()
    qs = [(q0 + 0.5 * wl.make_query(w, DEV, 1 + s).float()).to(w.dtype) for s in range(steps)]
    k, v, g = wl.make_prefill(w, DEV, T0)
    # the golden page's keys line up with that direction (the decayed state keeps a fraction of it)
    qm = q0 / q0.norm(dim=-1, keepdim=True)
    kf = k.float()
    for b in range(w.B):
        for h in range(w.H):
            p = int(gold[b, h])
            kf[b, p * S:(p + 1) * S, h, :] += 6.0 * qm[b, h]
    k = kf.to(w.dtype)
    cap = T0 + steps + 2
    cache = rq.Cache(w.B, w.H, w.D, S, cap, w.dtype, max_budget_pages=w.pages(cap))
    rq.rq_build_cache(cache.handle, k, v, g)
    ohs = {(b, h): parity.oracle_head(w, k, v, g, b, h, cap) for b in range(w.B) for h in (0, w.H - 1)}
    sel_quest, sel_rand = [], [[] for _ in range(5)]
    for s in range(steps):
        kt, vt, gt = wl.make_token(w, DEV, s)
        T = T0 + s + 1
        K, P = w.budget_pages(T), w.pages(T)
        o = torch.empty(w.B, w.H, w.D, dtype=w.dtype, device=DEV)
        idx = torch.empty(w.B, w.H, K, dtype=torch.int32, device=DEV)
        rq.rq_decode_step(cache.handle, qs[s], kt, vt, gt, K, 0.0, o, idx)
        sel_quest.append(idx.cpu())
        for (b, h), hd in ohs.items():
            hd.append(parity.f64(kt[b, h]), parity.f64(vt[b, h]), parity.f64(gt[b, h]))
        for seed in range(5):                                                    # the paper's five seeds
            ridx = selectors.random_pages(w.B, w.H, P, K, seed=100 * s + seed, device=DEV)
            sel_rand[seed].append(ridx.cpu())
            if seed == 0:
                orand = torch.empty_like(o)
                rq.rq_attend_pages(cache.handle, qs[s], ridx, K, 0.0, orand)
                torch.cuda.synchronize()
                for (b, h), hd in ohs.items():
                    dev = parity.device_head_arrays(cache, b, h)
                    y = parity.oracle.sparse_attention(parity.f64(qs[s][b, h]), w.D ** -0.5, dev["k"], dev["v"],
                                                       ridx[b, h].cpu().numpy().astype(np.int64), S)
                    err = np.abs(parity.f64(orand[b, h]) - y)
                    assert err.max() <= parity.ATT_TOL[w.dtype][0]
    torch.cuda.synchronize()
    assert rq.rq_device_status(cache.handle) == rq.RQ_OK
    quest = selectors.hit_rate(sel_quest, gold)
    rand = float(np.mean([selectors.hit_rate(sr, gold) for sr in sel_rand]))
    assert quest >= 0.9, quest
    # (K / P)^3 = 2.4e-4 per head: over 5 seeds x 16 heads a hit is already unlikely
    assert rand <= 0.05, rand


@pytest.mark.parametrize("S,K,T", [(64, 16, 4096), (16, 4, 4096), (16, 9, 1000), (64, 3, 16384)])
def test_short_context_single_launch_path(S, K, T):
    """With at least 16 heads and at most 256 pages per head the update, the scoring and the selection
    run as one launch (one CTA per head); same staged parity as the three-launch path, three steps
    so that the token count crosses a page boundary, and the stage export must agree with it."""
    w = wl.Workload("short", B=2, H=16, D=128, T=T, S=S, seed=500 + S + K)
    heads = [(0, 0), (0, 7), (1, 3), (1, 15)]
    stats = {}
    run_case(w, T - 3, steps=3, heads=heads, budget=K, stats=stats)
    assert stats["heads"] == 3 * len(heads)
    assert stats.get("near_tie_mismatch", 0) <= stats.get("near_tie", 0)


def test_short_context_path_other_shapes():
    """fp32 I/O with 64 channels and fp32 gates on bf16 I/O through the single-launch path."""
    for dtype, gdt, D in ((torch.float32, None, 64), (torch.bfloat16, torch.float32, 128), (torch.bfloat16, None, 64)):
        w = wl.Workload("short-shapes", B=1, H=16, D=D, T=777, S=16, dtype=dtype, gate_dtype=gdt, budget_den=4, seed=600 + D)
        stats = {}
        run_case(w, w.T - 2, steps=2, heads=[(0, 0), (0, 9), (0, 15)], stats=stats)
        assert stats["heads"] == 6
