"""GPU parity: the CUDA path, called through the C ABI, against the fp64 oracle
element by element on the same seeded inputs.  Sizes here are ones the oracle
finishes in seconds but that span several tiles and ragged tails."""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
import paper_2605_28640_b200 as rq
from paper_2605_28640_b200 import workloads as wl

import parity

pytestmark = pytest.mark.gpu
DEV = "cuda"


def run_case(w, T_prefill, steps=1, heads=None, n_sink=1, n_local=1, scale=0.0, chunks=None,
             budget=None, stats=None, path=0, want_launches=None):
    """Prefill T_prefill tokens (optionally in several rq_build_cache calls), then run decode
    steps, checking every level after the prefill and after every step for the sampled heads.
    path: rq_cache.reserved[2] (0: the library chooses how the step is launched, 1: separate
    kernels, 2 / 4 / 8: one launch with that many groups of heads)."""
    stats = {} if stats is None else stats
    cap = T_prefill + steps + 3
    maxK = max(w.pages(cap), budget or 1)
    cache = rq.Cache(w.B, w.H, w.D, w.S, cap, w.dtype, w.gdtype, n_sink, n_local, maxK)
    cache.handle.reserved[2] = path
    q0 = wl.make_query(w, DEV, 0)
    k, v, g = wl.make_prefill(w, DEV, T_prefill, q_for_needles=q0 if w.needles else None)
    bounds = [0, *(chunks or []), T_prefill]
    for a, b in zip(bounds[:-1], bounds[1:]):
        rq.rq_build_cache(cache.handle, k[:, a:b], v[:, a:b], g[:, a:b])
    assert len(cache) == T_prefill
    heads = heads or [(b, h) for b in range(w.B) for h in range(w.H)]
    ohs = {bh: parity.oracle_head(w, k, v, g, bh[0], bh[1], cap, n_sink, n_local) for bh in heads}
    if T_prefill > 0:
        for (b, h), hd in ohs.items():
            parity.check_cache_level(cache, hd, b, h, w.dtype)
    sc = scale if scale > 0 else w.D ** -0.5
    for step in range(steps):
        q = wl.make_query(w, DEV, step)
        kt, vt, gt = wl.make_token(w, DEV, step)
        T = T_prefill + step + 1
        K = budget if budget is not None else w.budget_pages(T)
        o = torch.empty(w.B, w.H, w.D, dtype=w.dtype, device=DEV)
        idx = torch.full((w.B, w.H, K), -7, dtype=torch.int32, device=DEV)
        if want_launches is not None:
            assert rq.rq_decode_step_launches(cache.handle, K) == want_launches
        rq.rq_decode_step(cache.handle, q, kt, vt, gt, K, scale, o, idx)
        assert len(cache) == T
        P = w.pages(T)
        scores = torch.empty(w.B, w.H, P, dtype=torch.float32, device=DEV)
        idx2 = torch.full((w.B, w.H, K), -7, dtype=torch.int32, device=DEV)
        rq.rq_select_pages(cache.handle, q, K, scores, idx2)
        torch.cuda.synchronize()
        assert torch.equal(idx, idx2), "stage export and decode step select different pages"
        assert rq.rq_device_status(cache.handle) == rq.RQ_OK
        for (b, h), hd in ohs.items():
            hd.append(parity.f64(kt[b, h]), parity.f64(vt[b, h]), parity.f64(gt[b, h]))
            dev = parity.check_cache_level(cache, hd, b, h, w.dtype)
            parity.check_query_level(dev, hd, cache, b, h, q, K, sc, o, idx, scores, w.dtype, stats)
    return cache, stats


def test_config0_tiny_fp32_full_chain():
    """Config 0: batch 1, 4 heads, D 64, context 1024, page 16, budget 1/4, fp32."""
    w = wl.CONFIGS[0]
    _, stats = run_case(w, w.T - 1, steps=1)
    assert stats["heads"] == 4 and stats.get("near_tie_mismatch", 0) <= stats.get("near_tie", 0)


SHAPES = [
    # B  H  D    S   T    dtype           gate dtype       budget (num, den)
    (2, 3, 128, 16, 333, torch.bfloat16, None, (1, 4)),
    (2, 3, 128, 16, 1000, torch.bfloat16, torch.float32, (1, 8)),
    (1, 2, 64, 16, 517, torch.bfloat16, None, (1, 4)),
    (1, 2, 64, 16, 700, torch.float32, torch.bfloat16, (1, 4)),
    (1, 2, 128, 16, 450, torch.float32, None, (1, 2)),
    (2, 2, 128, 64, 1111, torch.bfloat16, None, (1, 4)),
    (1, 3, 64, 64, 900, torch.bfloat16, torch.float32, (1, 2)),
    (1, 2, 128, 64, 400, torch.float32, None, (1, 2)),
    (1, 2, 64, 64, 260, torch.float32, None, (1, 2)),
]


@pytest.mark.parametrize("B,H,D,S,T,dtype,gdt,budget", SHAPES)
def test_shapes_and_dtypes(B, H, D, S, T, dtype, gdt, budget):
    w = wl.Workload("shape", B=B, H=H, D=D, T=T, S=S, budget_num=budget[0], budget_den=budget[1],
                    dtype=dtype, gate_dtype=gdt, seed=11 + T)
    run_case(w, T - 2, steps=2)


@pytest.mark.parametrize("T", [0, 1, 2, 15, 16, 17, 31, 32, 33, 63, 64, 65, 127, 128, 129, 255, 257])
def test_ragged_lengths(T):
    """Every alignment of the context against pages, slices and chunks, including an empty prefill."""
    w = wl.Workload("ragged", B=1, H=2, D=128, T=T + 1, budget_num=1, budget_den=2, seed=100 + T)
    run_case(w, T, steps=1)


@pytest.mark.parametrize("n_sink,n_local,K", [(0, 0, 1), (0, 0, 5), (1, 1, 2), (1, 1, 1), (2, 3, 4), (2, 3, 9),
                                              (0, 2, 6), (1, 1, 1000), (3, 0, 7)])
def test_forced_pages_and_budgets(n_sink, n_local, K):
    w = wl.Workload("forced", B=1, H=4, D=128, T=600, seed=5)
    run_case(w, 599, steps=1, n_sink=n_sink, n_local=n_local, budget=K)


def test_chunked_prefill_matches_oracle():
    """rq_build_cache may be called repeatedly; cuts at arbitrary (unaligned) positions."""
    w = wl.Workload("chunked", B=2, H=2, D=128, T=1200, budget_den=4, seed=21)
    run_case(w, 1199, steps=1, chunks=[1, 130, 131, 500, 777])
    w = wl.Workload("chunked64", B=1, H=2, D=64, T=900, S=64, budget_den=2, seed=22)
    run_case(w, 899, steps=1, chunks=[70, 128, 640])


def test_prefill_decode_equivalence():
    """build(T) + decode step must see the same cache as build(T+1)."""
    w = wl.Workload("equiv", B=1, H=4, D=128, T=800, budget_den=4, seed=31)
    for T in (799, 800, 815):     # new token lands mid-page, opens a page, closes a page
        k, v, g = wl.make_prefill(w, DEV, T + 1)
        q = wl.make_query(w, DEV, 0)
        K = w.budget_pages(T + 1)
        a = rq.Cache(w.B, w.H, w.D, w.S, T + 8, w.dtype)
        rq.rq_build_cache(a.handle, k[:, :T], v[:, :T], g[:, :T])
        oa = torch.empty(w.B, w.H, w.D, dtype=w.dtype, device=DEV)
        ia = torch.empty(w.B, w.H, K, dtype=torch.int32, device=DEV)
        rq.rq_decode_step(a.handle, q, k[:, T].contiguous(), v[:, T].contiguous(), g[:, T].contiguous(),
                          K, 0.0, oa, ia)
        b = rq.Cache(w.B, w.H, w.D, w.S, T + 8, w.dtype)
        rq.rq_build_cache(b.handle, k, v, g)
        ib = torch.empty_like(ia)
        ob = torch.empty_like(oa)
        rq.rq_select_pages(b.handle, q, K, None, ib)
        rq.rq_attend_pages(b.handle, q, ib, K, 0.0, ob)
        torch.cuda.synchronize()
        P = w.pages(T + 1)
        # states agree to fp32 rounding of differently associated sums; stored values to 1 ulp
        np.testing.assert_allclose(parity.f64(a.state_view()), parity.f64(b.state_view()), rtol=1e-4, atol=1e-6)
        ka, kb = parity.f64(a.kv_view()[:, :, :P]), parity.f64(b.kv_view()[:, :, :P])
        assert (ka != kb).mean() < 1e-3
        if torch.equal(ia, ib):
            assert (oa.float() - ob.float()).abs().max().item() <= 2e-2


def test_multistep_decode_batched():
    """A small version of the batched multi-step workload: every step checked."""
    w = wl.Workload("multistep", B=2, H=4, D=128, T=500, budget_den=8, seed=2, steps=40)
    _, stats = run_case(w, 500, steps=40, heads=[(0, 0), (0, 3), (1, 1), (1, 3)])
    assert stats["heads"] == 160


def test_config1_all_heads():
    """Config 1: batch 1, 32 heads, D 128, context 16384, budget 1/16 (64 pages), bf16."""
    w = wl.CONFIGS[1]
    _, stats = run_case(w, w.T - 1, steps=1, want_launches=3)     # 32 heads: separate kernels
    assert stats["heads"] == 32
    assert stats["e2e_overlap"] / stats["heads"] >= 0.99


def test_all_equal_scores_take_lowest_pages():
    """q = 0 makes every score equal: ties go to the lower page index, forced pages stay."""
    w = wl.Workload("ties", B=1, H=2, D=128, T=640, seed=41)
    k, v, g = wl.make_prefill(w, DEV)
    c = rq.Cache(w.B, w.H, w.D, w.S, w.T, w.dtype)
    rq.rq_build_cache(c.handle, k, v, g)
    q = torch.zeros(w.B, w.H, w.D, dtype=w.dtype, device=DEV)
    idx = torch.empty(w.B, w.H, 6, dtype=torch.int32, device=DEV)
    rq.rq_select_pages(c.handle, q, 6, None, idx)
    assert idx.cpu().tolist() == [[[0, 1, 2, 3, 4, 39]] * 2]
    # negative zero scores must tie with positive zero
    q[0, 0, 0] = -0.0
    rq.rq_select_pages(c.handle, q, 6, None, idx)
    assert idx.cpu().tolist() == [[[0, 1, 2, 3, 4, 39]] * 2]


def test_duplicated_scores_split_by_index():
    """Pages with identical bounds have identical scores; selection must be the oracle's exactly."""
    w = wl.Workload("dups", B=1, H=1, D=64, T=16 * 48, dtype=torch.float32, seed=43)
    k, v, g = wl.make_prefill(w, DEV)
    g.zero_()                                   # cache = raw keys
    k[:, 16 * 8:] = k[:, :16 * 8].repeat(1, 5, 1, 1)   # 48 pages = 6 copies of 8 pages
    c = rq.Cache(w.B, w.H, w.D, w.S, w.T, w.dtype, n_sink_pages=0, n_local_pages=0)
    rq.rq_build_cache(c.handle, k, v, g)
    q = wl.make_query(w, DEV)
    for K in (1, 3, 6, 7, 13, 20):
        idx = torch.empty(1, 1, K, dtype=torch.int32, device=DEV)
        sc = torch.empty(1, 1, 48, dtype=torch.float32, device=DEV)
        rq.rq_select_pages(c.handle, q, K, sc, idx)
        U = parity.f64(sc[0, 0])
        assert np.array_equal(U[:8], U[8:16]) and np.array_equal(U[:8], U[40:])
        want, _ = oracle.select_pages(U, K, 0, 0)
        assert idx[0, 0].cpu().tolist() == want.tolist()


def test_zero_gate_stores_raw_kv():
    """g = 0 (Eq. 2's standard-attention baseline): the cache holds k and v themselves."""
    w = wl.Workload("g0", B=1, H=2, D=128, T=300, seed=51)
    k, v, g = wl.make_prefill(w, DEV)
    g.zero_()
    c = rq.Cache(w.B, w.H, w.D, w.S, w.T, w.dtype)
    rq.rq_build_cache(c.handle, k, v, g)
    kv = c.kv_view()
    P = w.pages()
    got_k = kv[:, :, :P, 0].reshape(w.B, w.H, P * w.S, w.D)[:, :, :w.T].permute(0, 2, 1, 3)
    got_v = kv[:, :, :P, 1].reshape(w.B, w.H, P * w.S, w.D)[:, :, :w.T].permute(0, 2, 1, 3)
    assert torch.equal(got_k, k) and torch.equal(got_v, v)
    # dense budget: textbook attention on raw k, v
    q = wl.make_query(w, DEV)
    o = torch.empty(w.B, w.H, w.D, dtype=w.dtype, device=DEV)
    idx = torch.arange(P, dtype=torch.int32, device=DEV).repeat(w.B, w.H, 1)
    rq.rq_attend_pages(c.handle, q, idx, P, 0.0, o)
    ref = torch.nn.functional.scaled_dot_product_attention(
        q.double().cpu()[:, :, None, :], k.double().cpu().permute(0, 2, 1, 3), v.double().cpu().permute(0, 2, 1, 3))
    assert (o.double().cpu() - ref[:, :, 0]).abs().max().item() <= 2e-2


def test_attend_pages_with_caller_indices():
    """Random selector hook: duplicates are attended twice, -1 is skipped, out-of-range is reported."""
    w = wl.Workload("attend", B=2, H=2, D=128, T=1000, seed=61)
    k, v, g = wl.make_prefill(w, DEV)
    c = rq.Cache(w.B, w.H, w.D, w.S, w.T, w.dtype)
    rq.rq_build_cache(c.handle, k, v, g)
    q = wl.make_query(w, DEV)
    P = w.pages()
    gen = torch.Generator().manual_seed(0)
    idx = torch.randint(0, P, (w.B, w.H, 12), generator=gen, dtype=torch.int32)
    idx[:, :, 3] = -1
    idx[:, :, 5] = idx[:, :, 4]
    idx[0, 0, 7] = P - 1                      # ragged last page (1000 = 62*16 + 8)
    o = torch.empty(w.B, w.H, w.D, dtype=w.dtype, device=DEV)
    rq.rq_attend_pages(c.handle, q, idx.to(DEV), 12, 0.25, o)
    assert rq.rq_device_status(c.handle) == rq.RQ_OK
    for b in range(w.B):
        for h in range(w.H):
            dev = parity.device_head_arrays(c, b, h)
            use = np.array([p for p in idx[b, h].tolist() if p >= 0])
            # the oracle attends a repeated page once per occurrence as well
            y = oracle.sparse_attention(parity.f64(q[b, h]), 0.25, dev["k"], dev["v"], use, w.S)
            assert np.abs(parity.f64(o[b, h]) - y).max() <= 2e-2
    idx[1, 1, 0] = P
    rq.rq_attend_pages(c.handle, q, idx.to(DEV), 12, 0.25, o)
    assert rq.rq_device_status(c.handle) == rq.RQ_ERR_INVALID_ARG
    assert rq.rq_device_status(c.handle) == rq.RQ_OK      # reading clears it


def test_decode_step_host_buffers():
    """The host-buffer entry point gives the same result as the device-buffer one."""
    w = wl.Workload("host", B=2, H=4, D=128, T=700, budget_den=4, seed=71)
    k, v, g = wl.make_prefill(w, DEV, 699)
    q = wl.make_query(w, DEV)
    kt, vt, gt = wl.make_token(w, DEV)
    K = w.budget_pages()
    outs = []
    for host in (False, "pinned", "pageable"):       # pinned inputs are gathered by a kernel, pageable ones copied
        c = rq.Cache(w.B, w.H, w.D, w.S, w.T, w.dtype)
        rq.rq_build_cache(c.handle, k, v, g)
        if host:
            pin = (lambda t: t.pin_memory()) if host == "pinned" else (lambda t: t)
            hq, hk, hv, hg = (pin(t.cpu()) for t in (q, kt, vt, gt))
            o = pin(torch.empty(w.B, w.H, w.D, dtype=w.dtype))
            idx = pin(torch.empty(w.B, w.H, K, dtype=torch.int32))
            rq.rq_decode_step_host(c.handle, hq, hk, hv, hg, K, 0.0, o, idx)
        else:
            o = torch.empty(w.B, w.H, w.D, dtype=w.dtype, device=DEV)
            idx = torch.empty(w.B, w.H, K, dtype=torch.int32, device=DEV)
            rq.rq_decode_step(c.handle, q, kt, vt, gt, K, 0.0, o, idx)
        torch.cuda.synchronize()
        outs.append((o.cpu(), idx.cpu(), c.state_view().cpu()))
    for other in outs[1:]:
        assert torch.equal(outs[0][0], other[0]) and torch.equal(outs[0][1], other[1]) and torch.equal(outs[0][2], other[2])


def test_capacity_errors_leave_cache_unchanged():
    w = wl.Workload("cap", B=1, H=2, D=128, T=64, seed=81)
    k, v, g = wl.make_prefill(w, DEV)
    c = rq.Cache(w.B, w.H, w.D, w.S, 64, w.dtype, max_budget_pages=2)
    rq.rq_build_cache(c.handle, k, v, g)
    with pytest.raises(rq.RqError) as e:
        rq.rq_build_cache(c.handle, k[:, :1], v[:, :1], g[:, :1])
    assert e.value.status == rq.RQ_ERR_CAPACITY and len(c) == 64
    q = wl.make_query(w, DEV)
    kt, vt, gt = wl.make_token(w, DEV)
    o = torch.empty(w.B, w.H, w.D, dtype=w.dtype, device=DEV)
    with pytest.raises(rq.RqError) as e:
        rq.rq_decode_step(c.handle, q, kt, vt, gt, 2, 0.0, o)
    assert e.value.status == rq.RQ_ERR_CAPACITY and len(c) == 64
    idx = torch.empty(w.B, w.H, 3, dtype=torch.int32, device=DEV)
    with pytest.raises(rq.RqError) as e:
        rq.rq_select_pages(c.handle, q, 3, None, idx)       # beyond max_budget_pages
    assert e.value.status == rq.RQ_ERR_CAPACITY
    rq.rq_cache_reset(c.handle)
    assert len(c) == 0
    rq.rq_build_cache(c.handle, k[:, :10], v[:, :10], g[:, :10])
    torch.cuda.synchronize()
    assert len(c) == 10


def test_split_counts_give_same_result():
    """Different batch sizes change the split-K factor; the same head must give the same pages
    and (to fp32 re-association) the same output."""
    base = wl.Workload("splits", B=1, H=2, D=128, T=4000, budget_den=4, seed=91)
    outs = []
    for B in (1, 16, 64):
        w = dataclasses.replace(base, B=B)
        k, v, g = wl.make_prefill(base, DEV)
        q = wl.make_query(base, DEV)
        c = rq.Cache(B, w.H, w.D, w.S, w.T, w.dtype)
        rq.rq_build_cache(c.handle, k.expand(B, -1, -1, -1).contiguous(), v.expand(B, -1, -1, -1).contiguous(),
                          g.expand(B, -1, -1, -1).contiguous())
        K = w.budget_pages()
        idx = torch.empty(B, w.H, K, dtype=torch.int32, device=DEV)
        o = torch.empty(B, w.H, w.D, dtype=w.dtype, device=DEV)
        qq = q.expand(B, -1, -1).contiguous()
        rq.rq_select_pages(c.handle, qq, K, None, idx)
        rq.rq_attend_pages(c.handle, qq, idx, K, 0.0, o)
        torch.cuda.synchronize()
        assert torch.equal(idx[0], idx[-1]) and torch.equal(o[0], o[-1])
        outs.append((idx[0].cpu(), o[0].float().cpu()))
    for i, o in outs[1:]:
        assert torch.equal(i, outs[0][0])
        assert (o - outs[0][1]).abs().max().item() <= 4e-3
