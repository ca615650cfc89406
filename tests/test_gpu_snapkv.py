"""GPU parity of the SnapKV-style cache reduction on the decayed states (App. A.1, SnapKV paragraph)
against the fp64 oracle, level by level:

  importance : the device's fp32 importances vs the oracle's on the device's stored keys and the
               same query bits, within 2e-5 of the head's largest importance (fp32 dot products of
               D terms, exponentials and a sum over at most 64 queries); every query's weights sum
               to one, so a head's importances sum to the window length
  selection  : the oracle's selection run on the DEVICE's importances must give the same positions,
               index for index (ascending; equal importance to the lower position), except where
               the oracle flags a near-tie at the cut, which is counted
  compaction : the new cache holds exactly the selected rows of the old one (bit for bit), zeros in
               the unused slots of its last page, page bounds equal to min/max of its own rows, and
               the old cache's recurrence state
  decoding   : decode steps on the reduced cache with a budget that covers all its pages equal the
               oracle's attention over the retained tokens plus the tokens appended since, with the
               recurrence continuing from the prompt's end
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2605_28640_b200 as rq
from paper_2605_28640_b200 import workloads as wl

import parity

pytestmark = pytest.mark.gpu
DEV = "cuda"


def sample_heads(B, H, n):
    flat = sorted({int(round(x)) for x in np.linspace(0, B * H - 1, n)})
    return [(i // H, i % H) for i in flat]


def window_queries(w, W, seed):
    g = torch.Generator(device=DEV)
    g.manual_seed(seed)
    return torch.randn(w.B, W, w.H, w.D, generator=g, device=DEV, dtype=torch.float32).to(w.dtype)


def snap_select(cache, qw, W, keep, scale=0.0, want_importance=True):
    c = cache.cfg
    T = len(cache)
    idx = torch.full((c.batch, c.heads, keep), -7, dtype=torch.int32, device=DEV)
    imp = torch.empty(c.batch, c.heads, T, dtype=torch.float32, device=DEV) if want_importance else None
    scratch = torch.empty(rq.rq_snapkv_scratch_bytes(cache.handle), dtype=torch.uint8, device=DEV)
    assert scratch.data_ptr() % 256 == 0
    rq.rq_snapkv_select(cache.handle, qw, W, keep, scale, idx, imp, scratch)
    torch.cuda.synchronize()
    return idx, imp


def check_head_selection(cache, b, h, qw, W, keep, idx, imp, scale):
    """Importance and selection levels for one head.  Returns the device arrays of the head."""
    T = len(cache)
    dev = parity.device_head_arrays(cache, b, h)
    gi = parity.f64(imp[b, h])
    ref = oracle.snapkv_importance(parity.f64(qw[b, :, h, :]), scale, dev["k"])
    tol = 2e-5 * ref.max() + 1e-7
    err = np.abs(gi - ref).max()
    parity.note_max("snapkv_importance_err_over_max", err / ref.max())
    assert err <= tol, f"importance[{b},{h}]: max err {err:.3e} > {tol:.3e}"
    assert abs(gi.sum() - W) <= 1e-3 * W, f"importance[{b},{h}] sums to {gi.sum()}, not {W}"
    want, near = oracle.snapkv_select(gi, W, keep)
    got = idx[b, h].cpu().numpy().astype(np.int64)
    n = len(want)
    assert n == min(keep, T)
    assert (got[n:] == -1).all()
    assert (np.diff(got[:n]) > 0).all(), "retained positions are not strictly ascending"
    assert (got[n - min(W, n):n] == np.arange(T - min(W, n), T)).all(), "the window is not retained"
    parity.note_count("snapkv_heads_checked")
    if not np.array_equal(got[:n], want):
        assert near, f"head ({b},{h}), keep {keep}: positions differ from the oracle's without a near-tie at the cut"
        parity.note_count("snapkv_near_tie_heads")
        # all but the entries at the cut agree
        assert len(np.setdiff1d(got[:n], want)) <= 2
    return dev


def check_compaction(src_dev, dst, b, h, sel, src_state):
    """Compaction level for one head: rows, tail, bounds, state."""
    d = parity.device_head_arrays(dst, b, h)
    assert np.array_equal(d["k"], src_dev["k"][sel]), "compacted keys are not the selected rows"
    assert np.array_equal(d["v"], src_dev["v"][sel]), "compacted values are not the selected rows"
    assert not d["k_tail"].any() and not d["v_tail"].any()
    mn, mx = oracle.page_bounds(d["k"], dst.cfg.page_size)
    assert np.array_equal(mn, d["min"]) and np.array_equal(mx, d["max"])
    assert np.array_equal(d["state_k"], src_state[0]) and np.array_equal(d["state_v"], src_state[1])
    return d


def run_snapkv(w, W, keep, heads, steps=2, seed=11, scale=0.0):
    """Prefill, select, compact, decode `steps` tokens on the reduced cache; every level checked
    for the sampled heads."""
    T = w.T
    cache = rq.Cache(w.B, w.H, w.D, w.S, T, w.dtype, w.gdtype)
    k, v, g = wl.make_prefill(w, DEV, T)
    rq.rq_build_cache(cache.handle, k, v, g)
    del k, v, g
    qw = window_queries(w, W, seed)
    sc = scale if scale > 0 else w.D ** -0.5
    idx, imp = snap_select(cache, qw, W, keep, scale)
    n = min(keep, T)
    small = rq.Cache(w.B, w.H, w.D, w.S, n + steps, w.dtype, w.gdtype, n_sink_pages=1, n_local_pages=1)
    rq.rq_snapkv_compact(cache.handle, idx, n, small.handle)
    torch.cuda.synchronize()
    assert len(small) == n
    assert rq.rq_device_status(small.handle) == rq.RQ_OK
    heads_dev = {}
    for (b, h) in heads:
        src = check_head_selection(cache, b, h, qw, W, keep, idx, imp, sc)
        sel = idx[b, h, :n].cpu().numpy().astype(np.int64)
        st = parity.f64(cache.state_view()[b, h])
        check_compaction(src, small, b, h, sel, st)
        heads_dev[(b, h)] = (src, sel, st)
    # decoding on the reduced cache: all pages fit the budget, so attention covers every retained
    # entry and every appended token
    odt = parity.ODT[w.dtype]
    appended = {bh: ([], []) for bh in heads}
    state = {bh: (heads_dev[bh][2][0].copy(), heads_dev[bh][2][1].copy()) for bh in heads}
    for step in range(steps):
        q = wl.make_query(w, DEV, step)
        kt, vt, gt = wl.make_token(w, DEV, step)
        o = torch.empty(w.B, w.H, w.D, dtype=w.dtype, device=DEV)
        P = (len(small) + 1 + w.S - 1) // w.S
        rq.rq_decode_step(small.handle, q, kt, vt, gt, P, scale, o)
        torch.cuda.synchronize()
        assert rq.rq_device_status(small.handle) == rq.RQ_OK
        assert len(small) == n + step + 1
        for (b, h) in heads:
            src, sel, _ = heads_dev[(b, h)]
            sk, sv = state[(b, h)]
            gk = parity.f64(gt[b, h])
            kk, vv = oracle.recurrence(parity.f64(kt[b, h])[None], parity.f64(vt[b, h])[None], gk[None], sk, sv)
            state[(b, h)] = (kk[0], vv[0])
            appended[(b, h)][0].append(oracle.round_storage(kk[0], odt))
            appended[(b, h)][1].append(oracle.round_storage(vv[0], odt))
            kst = np.concatenate([src["k"][sel], np.stack(appended[(b, h)][0])])
            vst = np.concatenate([src["v"][sel], np.stack(appended[(b, h)][1])])
            y = oracle.token_attention(parity.f64(q[b, h]), sc, kst, vst, np.arange(len(kst)))
            got = parity.f64(o[b, h])
            mx_tol, mean_tol = parity.ATT_TOL[w.dtype]
            e = np.abs(got - y)
            parity.note_max(f"snapkv_attention_max_err_{'bf16' if w.dtype == torch.bfloat16 else 'f32'}", e.max())
            assert e.max() <= mx_tol and e.mean() <= mean_tol, f"decode on the reduced cache, head ({b},{h}), step {step}: {e.max():.3e}"
    return cache, small, idx, imp


@pytest.mark.parametrize("keep", [1024, 512, 256])
def test_paper_budgets_on_4k_prompts(keep):
    """The paper's setting: prompts of 4096 tokens, window of 64 queries, 1024 / 512 / 256 retained
    entries (tests/golden/snapkv_budgets.txt)."""
    w = wl.Workload("snapkv-4k", B=2, H=8, D=128, T=4096, seed=21)
    run_snapkv(w, 64, keep, sample_heads(w.B, w.H, 6))


@pytest.mark.parametrize("B,H,D,T,W,keep,dtype", [
    (1, 2, 64, 777, 64, 200, torch.float32),       # ragged last tile and page
    (2, 3, 128, 1000, 17, 129, torch.bfloat16),    # short window, odd sizes
    (1, 4, 64, 130, 64, 64, torch.bfloat16),       # nothing but the window
    (1, 4, 128, 130, 64, 40, torch.float32),       # fewer entries than the window: its newest part
    (1, 2, 64, 300, 1, 50, torch.float32),         # a window of one query
    (1, 2, 128, 260, 32, 260, torch.bfloat16),     # everything is kept
    (1, 1, 128, 64, 64, 10, torch.bfloat16),       # the prompt is the window
    (3, 5, 64, 2049, 64, 1025, torch.bfloat16),    # one position past a tile boundary
])
def test_shapes_windows_and_ragged_sizes(B, H, D, T, W, keep, dtype):
    w = wl.Workload("snapkv-small", B=B, H=H, D=D, T=T, dtype=dtype, seed=T + W)
    run_snapkv(w, W, keep, [(b, h) for b in range(B) for h in range(H)][:8], steps=3)


def test_keep_beyond_the_cache_length_pads_with_minus_one():
    w = wl.Workload("snapkv-pad", B=1, H=2, D=64, T=100, dtype=torch.float32, seed=4)
    cache = rq.Cache(w.B, w.H, w.D, w.S, w.T, w.dtype, w.gdtype)
    k, v, g = wl.make_prefill(w, DEV, w.T)
    rq.rq_build_cache(cache.handle, k, v, g)
    qw = window_queries(w, 16, 1)
    idx, _ = snap_select(cache, qw, 16, 128)
    got = idx.cpu().numpy()
    assert (got[:, :, :100] == np.arange(100)).all() and (got[:, :, 100:] == -1).all()


def test_equal_keys_give_the_lowest_positions():
    """All keys equal: every position seen by all window queries has the same importance, so the
    retained entries before the window are the lowest positions (ties go to the lower position)."""
    B, H, D, S, T, W, keep = 1, 2, 64, 16, 3000, 8, 500
    cache = rq.Cache(B, H, D, S, T, torch.float32)
    k = torch.ones(B, T, H, D, dtype=torch.float32, device=DEV) * 0.25
    g = torch.zeros_like(k)                          # zero gate: the cache holds k itself
    rq.rq_build_cache(cache.handle, k, k, g)
    qw = torch.randn(B, W, H, D, device=DEV, dtype=torch.float32)
    idx, imp = snap_select(cache, qw, W, keep)
    got = idx.cpu().numpy()
    want = np.concatenate([np.arange(keep - W), np.arange(T - W, T)])
    for h in range(H):
        i = imp[0, h].cpu().numpy()
        assert (i[:T - W] == i[0]).all(), "equal keys seen by every query must have bit-equal importance"
        assert np.array_equal(got[0, h], want)


def test_argument_checks():
    w = wl.Workload("snapkv-args", B=1, H=2, D=64, T=200, dtype=torch.float32, seed=4)
    cache = rq.Cache(w.B, w.H, w.D, w.S, w.T, w.dtype, w.gdtype)
    k, v, g = wl.make_prefill(w, DEV, w.T)
    rq.rq_build_cache(cache.handle, k, v, g)
    qw = window_queries(w, 64, 1)
    idx = torch.empty(1, 2, 32, dtype=torch.int32, device=DEV)
    scratch = torch.empty(rq.rq_snapkv_scratch_bytes(cache.handle), dtype=torch.uint8, device=DEV)
    for W, keep in ((0, 32), (65, 32), (64, 0), (201, 32)):
        with pytest.raises(rq.RqError) as e:
            rq.rq_snapkv_select(cache.handle, qw, W, keep, 0.0, idx, None, scratch)
        assert e.value.status == rq.RQ_ERR_INVALID_ARG
    other = rq.Cache(1, 2, 128, w.S, 64, w.dtype, w.gdtype)
    with pytest.raises(rq.RqError) as e:
        rq.rq_snapkv_compact(cache.handle, idx, 32, other.handle)
    assert e.value.status == rq.RQ_ERR_INVALID_ARG
    tiny = rq.Cache(1, 2, 64, w.S, 16, w.dtype, w.gdtype)
    with pytest.raises(rq.RqError) as e:
        rq.rq_snapkv_compact(cache.handle, idx, 32, tiny.handle)
    assert e.value.status == rq.RQ_ERR_CAPACITY
    with pytest.raises(rq.RqError) as e:
        rq.rq_snapkv_compact(cache.handle, idx, 32, cache.handle)
    assert e.value.status == rq.RQ_ERR_INVALID_ARG


def test_128k_prompt_sampled_heads():
    """A 128K-token prompt of 32 heads reduced to 8192 entries: sampled heads through the importance
    and selection levels, all heads through the properties that hold at any size."""
    w = wl.Workload("snapkv-128k", B=1, H=32, D=128, T=131072, seed=33)
    W, keep = 64, 8192
    cache = rq.Cache(w.B, w.H, w.D, w.S, w.T, w.dtype, w.gdtype)
    k, v, g = wl.make_prefill(w, DEV, w.T)
    rq.rq_build_cache(cache.handle, k, v, g)
    del k, v, g
    qw = window_queries(w, W, 2)
    idx, imp = snap_select(cache, qw, W, keep)
    sums = imp.sum(dim=-1, dtype=torch.float64).cpu().numpy()
    assert np.abs(sums - W).max() <= 1e-3 * W
    got = idx.cpu().numpy()
    assert (np.diff(got, axis=-1) > 0).all()
    assert (got[:, :, -W:] == np.arange(w.T - W, w.T)).all()
    # the smallest retained importance before the window is at least the largest one left out
    ic = imp[:, :, :w.T - W]
    kept = torch.zeros_like(ic, dtype=torch.bool)
    kept.scatter_(2, idx[:, :, :keep - W].long(), True)
    lo_kept = torch.where(kept, ic, torch.full_like(ic, float("inf"))).amin(dim=-1)
    hi_left = torch.where(kept, torch.full_like(ic, -1.0), ic).amax(dim=-1)
    assert (lo_kept >= hi_left).all()
    small = rq.Cache(w.B, w.H, w.D, w.S, keep + 16, w.dtype, w.gdtype)
    rq.rq_snapkv_compact(cache.handle, idx, keep, small.handle)
    torch.cuda.synchronize()
    for (b, h) in sample_heads(w.B, w.H, 3):
        src = check_head_selection(cache, b, h, qw, W, keep, idx, imp, w.D ** -0.5)
        sel = got[b, h].astype(np.int64)
        check_compaction(src, small, b, h, sel, parity.f64(cache.state_view()[b, h]))


def test_unused_cache_memory_full_of_nans_does_not_leak():
    """A cache much larger than the prompt whose memory holds NaN bit patterns everywhere the prefill did not write: the
    tile copies of the last tiles read some of it; importances and the selection must not pick any of it up."""
    w = wl.Workload("snapkv-nan", B=1, H=2, D=128, T=1000, seed=19)
    cache = rq.Cache(w.B, w.H, w.D, w.S, 4096, w.dtype, w.gdtype)
    cache.kv.fill_(0xFF)
    cache.meta.fill_(0xFF)
    k, v, g = wl.make_prefill(w, DEV, w.T)
    rq.rq_build_cache(cache.handle, k, v, g)
    W, keep = 64, 200
    qw = window_queries(w, W, 5)
    idx, imp = snap_select(cache, qw, W, keep)
    assert torch.isfinite(imp).all()
    for h in range(w.H):
        check_head_selection(cache, 0, h, qw, W, keep, idx, imp, w.D ** -0.5)
