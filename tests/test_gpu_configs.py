"""GPU parity at the benchmark's full sizes, in the launch configuration the benchmark times.

The oracle cannot run every head of these workloads in seconds, and heads never interact, so
each case checks a fixed sample of (batch, head) pairs: the first, the last and a few in
between, through every level of the staged comparison (state, stored cache, page bounds,
selected pages, attention output)."""
import dataclasses

import numpy as np
import pytest
import torch

import paper_2605_28640_b200 as rq
from paper_2605_28640_b200 import workloads as wl

import parity

pytestmark = pytest.mark.gpu
DEV = "cuda"


def sample_heads(w, n):
    """First, last and n-2 evenly spaced (b, h) pairs."""
    flat = sorted({int(round(x)) for x in np.linspace(0, w.B * w.H - 1, n)})
    return [(i // w.H, i % w.H) for i in flat]


def build(w, T_prefill, cap, heads, q_for_needles=None, maxK=None):
    cache = rq.Cache(w.B, w.H, w.D, w.S, cap, w.dtype, w.gdtype, max_budget_pages=maxK or w.pages(cap))
    k, v, g = wl.make_prefill(w, DEV, T_prefill, q_for_needles=q_for_needles)
    rq.rq_build_cache(cache.handle, k, v, g)
    torch.cuda.synchronize()
    ohs = {bh: parity.oracle_head(w, k, v, g, bh[0], bh[1], cap) for bh in heads}
    del k, v, g
    torch.cuda.empty_cache()
    return cache, ohs


def decode_and_check(w, cache, ohs, step, K, stats, check_cache=True):
    q = wl.make_query(w, DEV, step)
    kt, vt, gt = wl.make_token(w, DEV, step)
    o = torch.empty(w.B, w.H, w.D, dtype=w.dtype, device=DEV)
    idx = torch.full((w.B, w.H, K), -7, dtype=torch.int32, device=DEV)
    rq.rq_decode_step(cache.handle, q, kt, vt, gt, K, 0.0, o, idx)
    P = w.pages(len(cache))
    scores = torch.empty(w.B, w.H, P, dtype=torch.float32, device=DEV)
    idx2 = torch.empty_like(idx)
    rq.rq_select_pages(cache.handle, q, K, scores, idx2)
    torch.cuda.synchronize()
    assert torch.equal(idx, idx2)
    assert rq.rq_device_status(cache.handle) == rq.RQ_OK
    for (b, h), hd in ohs.items():
        hd.append(parity.f64(kt[b, h]), parity.f64(vt[b, h]), parity.f64(gt[b, h]))
        if check_cache:
            dev = parity.check_cache_level(cache, hd, b, h, w.dtype)
        else:
            dev = parity.device_head_arrays(cache, b, h)
        parity.check_query_level(dev, hd, cache, b, h, q, K, w.D ** -0.5, o, idx, scores, w.dtype, stats)
    return idx


def test_config1_shape_is_covered_elsewhere():
    """Config 1 (16K context, all 32 heads) runs in test_gpu_parity.py::test_config1_all_heads."""
    assert wl.CONFIGS[1].budget_pages() == 64


def test_config2_batched_multistep_32k():
    """Config 2: batch 8, 32 heads, prefilled 32768, budget 1/8, 64 consecutive decode steps."""
    w = wl.CONFIGS[2]
    heads = sample_heads(w, 6)
    cache, ohs = build(w, w.T, w.T + w.steps + 8, heads, maxK=w.budget_pages(w.T + w.steps) + 1)
    for (b, h), hd in ohs.items():
        parity.check_cache_level(cache, hd, b, h, w.dtype)
    stats = {}
    for step in range(w.steps):
        K = w.budget_pages(w.T + step + 1)
        assert K == 257
        # the stored cache is compared in full on the first and last step, the appended token's
        # page and everything downstream on every step
        decode_and_check(w, cache, ohs, step, K, stats, check_cache=step in (0, w.steps - 1))
    assert stats["heads"] == len(heads) * w.steps
    assert stats.get("near_tie_mismatch", 0) <= stats.get("near_tie", 0)
    assert stats["e2e_overlap"] / stats["heads"] >= 0.99


def test_config3_prefill_128k_with_resets():
    """Config 3: batch 1, 32 heads, 131072 tokens, 1 % reset-like tokens: the prefill scan alone."""
    w = wl.CONFIGS[3]
    heads = sample_heads(w, 5)
    cache, ohs = build(w, w.T, w.T + 16, heads)
    assert len(cache) == w.T
    for (b, h), hd in ohs.items():
        parity.check_cache_level(cache, hd, b, h, w.dtype)
    # and one decode step on top of it
    stats = {}
    decode_and_check(w, cache, ohs, 0, w.budget_pages(w.T + 1), stats, check_cache=False)
    assert stats["heads"] == len(heads)


@pytest.mark.parametrize("den", [16, 8, 4])
def test_config4_needles_128k(den):
    """Config 4: batch 4, 32 heads, 131072 tokens, planted pages, budgets 1/16, 1/8, 1/4."""
    w = dataclasses.replace(wl.CONFIGS[4], budget_den=den)
    heads = sample_heads(w, 6)
    q0 = wl.make_query(w, DEV, 0)
    T0 = w.T - 1
    cache, ohs = build(w, T0, w.T + 8, heads, q_for_needles=q0, maxK=w.budget_pages(w.T) + 1)
    stats = {}
    K = w.budget_pages(w.T)
    idx = decode_and_check(w, cache, ohs, 0, K, stats, check_cache=False)
    assert stats["heads"] == len(heads)
    # recall of the planted pages over ALL heads (reported by the benchmark too)
    planted = wl.needle_pages(w, T0)
    sel = idx.cpu().numpy()
    hit = sum(len(set(planted[b, h].tolist()) & set(sel[b, h].tolist())) for b in range(w.B) for h in range(w.H))
    recall = hit / (w.B * w.H * w.needles)
    assert recall >= 0.9, f"recall of planted pages {recall:.3f}"


@pytest.mark.parametrize("T", [16384 * 16 + 40, 32768 * 16 - 9])
def test_long_context_selection_paths(T):
    """Heads of more than 16384 pages are selected with the keys in shared memory instead of registers;
    32768 pages is the largest head the selection supports.  One head pair of a narrow model keeps the
    oracle's work small."""
    w = wl.Workload("long", B=1, H=2, D=64, T=T, budget_num=1, budget_den=32, seed=77)
    heads = [(0, 0), (0, 1)]
    cache, ohs = build(w, T - 1, T + 4, heads, maxK=w.budget_pages(T) + 1)
    stats = {}
    decode_and_check(w, cache, ohs, 0, w.budget_pages(T), stats, check_cache=False)
    assert stats["heads"] == 2
    assert stats.get("near_tie_mismatch", 0) <= stats.get("near_tie", 0)
