"""GPU parity of the decode step run as ONE launch (update, scoring, selection by the warp that
completes a head's scoring, flash-decode and combine in one kernel, the heads in 2, 4 or 8 groups).

The library picks that path by itself for shapes that fill the GPU; here it is also forced
(rq_cache.reserved[2]) at sizes the oracle finishes in seconds, through the same staged
comparison as every other path: states, stored cache, page bounds, scores, page list (bit-exact
against the oracle on the device's bounds, and equal to the list of the separate selection
kernel), attention output.  (A head's team of CTAs must not outnumber the partial records the
workspace holds for it, so the forced shapes have enough heads per group or enough pages.)"""
import numpy as np
import pytest
import torch

import oracle
import paper_2605_28640_b200 as rq
from paper_2605_28640_b200 import workloads as wl

import parity
from test_gpu_parity import run_case

pytestmark = pytest.mark.gpu
DEV = "cuda"


STEP_SHAPES = [
    # B  H   D    S   T     dtype           gate dtype      budget   waves
    (2, 8, 128, 16, 1500, torch.bfloat16, None, (1, 8), 2),
    (4, 8, 128, 16, 1500, torch.bfloat16, None, (1, 8), 4),
    (4, 16, 128, 16, 3000, torch.bfloat16, torch.float32, (1, 16), 8),
    (1, 16, 64, 16, 2100, torch.bfloat16, None, (1, 4), 2),
    (2, 8, 128, 64, 5000, torch.bfloat16, None, (1, 4), 2),
    (1, 16, 64, 64, 6000, torch.bfloat16, torch.float32, (1, 2), 4),
    (2, 8, 128, 16, 900, torch.float32, None, (1, 4), 2),
    (2, 8, 64, 16, 1000, torch.float32, torch.bfloat16, (1, 4), 2),
    (1, 8, 128, 64, 2500, torch.float32, None, (1, 2), 2),
    (1, 8, 64, 64, 2500, torch.float32, None, (1, 2), 2),
]


@pytest.mark.parametrize("B,H,D,S,T,dtype,gdt,budget,waves", STEP_SHAPES)
def test_one_launch_step_shapes_and_dtypes(B, H, D, S, T, dtype, gdt, budget, waves):
    w = wl.Workload("step", B=B, H=H, D=D, T=T, S=S, budget_num=budget[0], budget_den=budget[1],
                    dtype=dtype, gate_dtype=gdt, seed=31 + T)
    heads = [(0, 0), (B - 1, H - 1), (0, H // 2), (B - 1, 1)]
    _, stats = run_case(w, T - 3, steps=3, heads=heads, path=waves, want_launches=1)
    assert stats["heads"] == 3 * len(set(heads))


@pytest.mark.parametrize("n_sink,n_local,K", [(0, 0, 1), (0, 0, 9), (1, 1, 2), (2, 3, 5), (2, 3, 40), (0, 2, 6), (3, 0, 7)])
def test_one_launch_step_forced_pages_and_budgets(n_sink, n_local, K):
    """First / newest pages inside the budget, also none at all (then the newest page competes with
    the score the update gives it) and budgets that hold nothing but forced pages."""
    w = wl.Workload("forced", B=2, H=8, D=128, T=1400, seed=5)
    run_case(w, 1398, steps=2, heads=[(0, 0), (1, 7), (1, 3)], n_sink=n_sink, n_local=n_local, budget=K, path=2,
             want_launches=1)


def test_one_launch_step_many_steps_alternate_counter_sets():
    """Forty consecutive steps (the per-head counters alternate between two sets, the newest page fills
    up and a new one opens), every step checked."""
    w = wl.Workload("multistep", B=2, H=8, D=128, T=1000, budget_den=8, seed=2, steps=40)
    _, stats = run_case(w, 1000, steps=40, heads=[(0, 0), (0, 5), (1, 1), (1, 7)], path=2, want_launches=1)
    assert stats["heads"] == 160


def planted_decode(U, H, waves, n_sink, n_local, Ks, D=64, S=16):
    """Scores planted through the keys (g = 0, channel 0 of every token of page p is U[h][p], q = e_0),
    the last token appended by the decode step itself; the list of the one-launch step must be the
    oracle's selection on the device's bounds, index for index."""
    U = np.asarray(U, dtype=np.float32)
    if U.ndim == 1:
        U = np.broadcast_to(U, (H, U.shape[0]))
    P = U.shape[1]
    T = P * S
    u = torch.from_numpy(np.ascontiguousarray(U)).to(DEV)                     # [H, P]
    k = torch.zeros(1, T, H, D, dtype=torch.float32, device=DEV)
    k[0, :, :, 0] = u.t().repeat_interleave(S, dim=0)
    z = torch.zeros_like(k)
    q = torch.zeros(1, H, D, dtype=torch.float32, device=DEV)
    q[:, :, 0] = 1.0
    for K in Ks:
        c = rq.Cache(1, H, D, S, T, torch.float32, n_sink_pages=n_sink, n_local_pages=n_local, max_budget_pages=P)
        c.handle.reserved[2] = waves
        rq.rq_build_cache(c.handle, k[:, :T - 1], z[:, :T - 1], z[:, :T - 1])
        assert rq.rq_decode_step_launches(c.handle, K) == 1
        o = torch.empty(1, H, D, dtype=torch.float32, device=DEV)
        idx = torch.full((1, H, K), -7, dtype=torch.int32, device=DEV)
        rq.rq_decode_step(c.handle, q, k[:, T - 1].contiguous(), z[:, T - 1].contiguous(), z[:, T - 1].contiguous(),
                          K, 0.0, o, idx)
        torch.cuda.synchronize()
        assert rq.rq_device_status(c.handle) == rq.RQ_OK
        for h in range(H):
            dev = parity.device_head_arrays(c, 0, h)
            Uo = oracle.page_scores(parity.f64(q[0, h]), dev["min"], dev["max"])
            assert np.array_equal(Uo, U[h].astype(np.float64))
            want, _ = oracle.select_pages(Uo, K, n_sink, n_local)
            got = idx[0, h].cpu().numpy().astype(np.int64)
            assert np.array_equal(got[:len(want)], want), f"head {h}, K {K}: pages differ from the oracle's"
            y = oracle.sparse_attention(parity.f64(q[0, h]), D ** -0.5, dev["k"], dev["v"], got, S)
            assert np.abs(parity.f64(o[0, h]) - y).max() <= 1e-4


def plateau_scores(P, levels, seed):
    rng = np.random.default_rng(seed)
    vals = rng.standard_normal(levels).astype(np.float32)
    return vals[rng.integers(0, levels, P)]


@pytest.mark.parametrize("forced", [(0, 0), (1, 1), (2, 3)])
def test_one_launch_step_long_runs_of_equal_scores(forced):
    """A few distinct scores over thousands of pages: the threshold bucket is too full to rank
    directly, the selecting warp goes through the radix passes and the ordered pass."""
    H, P = 8, 4100
    U = np.stack([plateau_scores(P, 2 + h % 4, seed=50 + h) for h in range(H)])
    planted_decode(U, H, 2, forced[0], forced[1], (3, P // 16, P // 3, P - 7))


def test_one_launch_step_distinct_and_duplicated_scores():
    """Distinct scores with a sprinkling of duplicates: the direct ranking of the threshold bucket,
    ties at the cut included; and one head whose scores are all equal."""
    H, P = 8, 3000
    rng = np.random.default_rng(77)
    U = rng.standard_normal((H, P)).astype(np.float32)
    for h in range(H):
        dup = rng.integers(0, P, 400)
        U[h, dup] = U[h, dup[0]]
    U[5] = np.float32(-0.75)
    planted_decode(U, H, 4, 1, 1, (2, 40, P // 8, P // 2 + 1))


def test_one_launch_step_degenerate_score_range():
    """Denormal scores: the a-priori range has no usable bucket width; everything lands in one bucket."""
    H, P = 8, 2000
    rng = np.random.default_rng(8)
    U = (rng.integers(0, 30, (H, P)).astype(np.float32) * np.float32(1.4e-45)).astype(np.float32)
    U[:, ::3] *= np.float32(-1.0)
    planted_decode(U, H, 2, 1, 1, (5, P // 10))


def test_one_launch_step_after_steps_as_separate_kernels():
    """Both paths keep the head's largest |stored key| up to date, so they can alternate on one cache."""
    w = wl.Workload("mixed", B=2, H=8, D=128, T=1200, budget_den=8, seed=12)
    cap = w.T + 8
    cache = rq.Cache(w.B, w.H, w.D, w.S, cap, w.dtype, max_budget_pages=w.pages(cap))
    k, v, g = wl.make_prefill(w, DEV, w.T - 6)
    rq.rq_build_cache(cache.handle, k, v, g)
    heads = [(0, 0), (1, 7)]
    ohs = {bh: parity.oracle_head(w, k, v, g, bh[0], bh[1], cap) for bh in heads}
    stats = {}
    for step, path in enumerate((1, 2, 2, 1, 2, 2)):
        cache.handle.reserved[2] = path
        q = wl.make_query(w, DEV, step)
        kt, vt, gt = wl.make_token(w, DEV, step)
        K = w.budget_pages(len(cache) + 1)
        o = torch.empty(w.B, w.H, w.D, dtype=w.dtype, device=DEV)
        idx = torch.full((w.B, w.H, K), -7, dtype=torch.int32, device=DEV)
        rq.rq_decode_step(cache.handle, q, kt, vt, gt, K, 0.0, o, idx)
        torch.cuda.synchronize()
        assert rq.rq_device_status(cache.handle) == rq.RQ_OK
        for (b, h), hd in ohs.items():
            hd.append(parity.f64(kt[b, h]), parity.f64(vt[b, h]), parity.f64(gt[b, h]))
            dev = parity.check_cache_level(cache, hd, b, h, w.dtype)
            parity.check_query_level(dev, hd, cache, b, h, q, K, w.D ** -0.5, o, idx, None, w.dtype, stats)
    assert stats["heads"] == 12
