"""Staged comparison of the CUDA path with the fp64 oracle for one (batch, head).

Levels (tolerances are the ones the benchmark definition states):
  1. state     : fp32 running state vs the oracle's fp64 state, 1e-4 relative
                 (with an absolute floor of 1e-5 of the state's rms for channels
                 that are near zero by cancellation)
  2. cache     : bf16 storage: stored k~, v~ equal to the oracle's stored values
                 or one storage-ulp apart, at least 99.9 % exactly equal (the
                 fp32 state error is far below a bf16 ulp, so only values next
                 to a rounding boundary can differ); fp32 storage: the stored
                 value IS the fp32 state, so the state tolerance applies;
                 page bounds bit-exact against min/max of the device's own cache
  3. selection : scores within 2e-6 of the sum of the products' magnitudes;
                 the oracle's scoring + top-k run on the DEVICE's bounds and q
                 bits must give the same pages, except where the oracle flags a
                 near-tie (1e-5 relative) at the cut — those are counted
  4. attention : the oracle's attention over the device's pages and stored
                 cache vs the device output: 2e-2 max-abs / 5e-3 mean-abs for
                 bf16, 1e-4 / 1e-5 for fp32; and the oracle's own end-to-end
                 chain wherever its page set equals the device's
"""
from __future__ import annotations

import numpy as np
import torch

import oracle

ODT = {torch.float32: oracle.F32, torch.bfloat16: oracle.BF16}

# Worst values and counts seen by the checks of this process; a test run prints them at its end
# (tests/conftest.py) and the benchmark puts them into its `parity` block.
OBSERVED = {}


def note_max(name, value):
    OBSERVED[name] = max(OBSERVED.get(name, 0.0), float(value))


def note_count(name, n=1):
    OBSERVED[name] = OBSERVED.get(name, 0) + n
ATT_TOL = {torch.bfloat16: (2e-2, 5e-3), torch.float32: (1e-4, 1e-5)}


def f64(t):
    return t.detach().to(torch.float64).cpu().numpy()


# Absolute floor of the state comparison, in units of the state's rms: a channel that cancels to
# near zero carries the rounding error of its terms, not of its value.  fp32 rounding of the
# recurrence leaves about eps/(1-g) relative to the terms' size; the largest error observed over
# the whole GPU suite (tests/conftest.py prints it) is well below this floor.
STATE_FLOOR = 1e-5


def storage_ulp(x, dtype):
    """Spacing of the storage format at |x| (normal range)."""
    ax = np.maximum(np.abs(x), 1e-30)
    e = np.floor(np.log2(ax))
    return 2.0 ** (e - (7 if dtype == torch.bfloat16 else 23))


def assert_state_close(gpu, ref, what):
    rms = float(np.sqrt(np.mean(ref ** 2))) or 1.0
    err = np.abs(gpu - ref)
    note_max("state_abs_err_over_rms", err.max() / rms)
    big = np.abs(ref) >= 0.05 * rms
    if big.any():
        note_max("state_rel_err_where_ref_ge_0.05rms", (err[big] / np.abs(ref[big])).max())
    tol = 1e-4 * np.abs(ref) + STATE_FLOOR * rms
    assert (err <= tol).all(), f"{what}: max excess {(err - tol).max():.3e} (rms {rms:.3e})"


def oracle_head(w, k, v, g, b, h, capacity, n_sink=1, n_local=1):
    """Oracle cache of head (b, h) prefilled with the same input bits."""
    hd = oracle.Head(w.D, w.S, capacity, ODT[w.dtype], n_sink, n_local)
    if k is not None and k.shape[1] > 0:
        hd.append(f64(k[b, :, h, :]), f64(v[b, :, h, :]), f64(g[b, :, h, :]))
    return hd


def device_head_arrays(cache, b, h):
    """The device's stored cache, bounds and state for head (b, h) as float64."""
    T = len(cache)
    S, D = cache.cfg.page_size, cache.cfg.head_dim
    P = (T + S - 1) // S
    kv = cache.kv_view()[b, h, :P]                     # [P, 2, S, D]
    k = f64(kv[:, 0]).reshape(P * S, D)[:T]
    v = f64(kv[:, 1]).reshape(P * S, D)[:T]
    meta = f64(cache.meta_view()[b, h, :P])            # [P, 2, D]
    st = f64(cache.state_view()[b, h])
    return {"k": k, "v": v, "min": meta[:, 0], "max": meta[:, 1], "state_k": st[0], "state_v": st[1],
            "k_tail": f64(kv[:, 0]).reshape(P * S, D)[T:], "v_tail": f64(kv[:, 1]).reshape(P * S, D)[T:]}


def check_cache_level(cache, hd, b, h, dtype):
    """Levels 1 and 2.  Returns the device arrays for later levels."""
    dev = device_head_arrays(cache, b, h)
    ex = hd.export()
    assert dev["k"].shape == ex["k"].shape
    assert_state_close(dev["state_k"], ex["state_k"], f"state_k[{b},{h}]")
    assert_state_close(dev["state_v"], ex["state_v"], f"state_v[{b},{h}]")
    for name in ("k", "v"):
        a, r = dev[name], ex[name]
        if dtype == torch.float32:
            # fp32 storage keeps the fp32 state itself: the state tolerance applies
            if a.size:
                assert_state_close(a, r, f"stored {name}[{b},{h}]")
            continue
        ne = a != r
        frac = ne.mean() if a.size else 0.0
        note_max("stored_fraction_one_step_off", frac)
        assert frac <= 1e-3, f"{name}[{b},{h}]: {frac:.2e} of stored values differ"
        if ne.any():
            # one rounding step apart, or (for values that are near zero by cancellation, where
            # an ulp is far below the fp32 state's absolute error) within the state tolerance
            gap = np.abs(a - r)[ne]
            ulp = storage_ulp(np.maximum(np.abs(a), np.abs(r)), dtype)[ne]
            rms = float(np.sqrt(np.mean(r ** 2)))
            slack = (1e-4 * np.abs(r) + STATE_FLOOR * rms)[ne]
            bad = gap > np.maximum(ulp * 1.0000001, slack)
            assert not bad.any(), (f"{name}[{b},{h}]: {bad.sum()} stored values are more than one "
                                   f"rounding step off (worst gap {gap[bad].max():.3e})")
    # unused slots of the last page are defined (zero)
    assert not dev["k_tail"].any() and not dev["v_tail"].any()
    mn, mx = oracle.page_bounds(dev["k"], cache.cfg.page_size)
    assert np.array_equal(mn, dev["min"]), f"min bounds [{b},{h}] differ from min of the device cache"
    assert np.array_equal(mx, dev["max"]), f"max bounds [{b},{h}] differ from max of the device cache"
    return dev


def check_query_level(dev, hd, cache, b, h, q, K, scale, o, idx, scores, dtype, stats):
    """Levels 3 and 4 for one head.  idx: device [B,H,K] int32; scores: device [B,H,P] or None."""
    S = cache.cfg.page_size
    n_sink, n_local = cache.cfg.n_sink_pages, cache.cfg.n_local_pages
    q64 = f64(q[b, h])
    U = oracle.page_scores(q64, dev["min"], dev["max"])
    if scores is not None:
        gU = f64(scores[b, h])
        assert gU.shape == U.shape
        # fp32 summation of the 2*D products (tree over the lanes, then sequential inside a lane):
        # the error is bounded by about 13 * 2^-24 of the sum of the products' magnitudes, which
        # is what matters when positive and negative terms cancel; allow 2e-6 of that sum
        mag = np.maximum(np.abs(q64 * dev["min"]), np.abs(q64 * dev["max"])).sum(axis=1)
        excess = np.abs(gU - U) - 2e-6 * mag
        assert excess.max() <= 0, f"scores[{b},{h}] off by {np.abs(gU - U).max():.2e} (allowed {2e-6 * mag.max():.2e})"
    want, near = oracle.select_pages(U, K, n_sink, n_local)
    got = idx[b, h].cpu().numpy().astype(np.int64)
    n = len(want)
    assert (got[n:] == -1).all(), "unused tail of the index list must be -1"
    got = got[:n]
    assert (np.diff(got) > 0).all(), "page list must be strictly ascending"
    stats["heads"] = stats.get("heads", 0) + 1
    note_count("heads_checked")
    if near:
        note_count("near_tie_heads")
    if not np.array_equal(got, want):
        note_count("near_tie_mismatches")
        assert near, f"pages [{b},{h}] differ from the oracle's with no near-tie at the cut"
        # whatever was swapped must sit within 1e-5 relative of the cut
        sel_o = set(want.tolist())
        sel_g = set(got.tolist())
        forced = set(range(min(n_sink, len(U)))) | set(range(max(len(U) - n_local, 0), len(U)))
        cut = min(U[p] for p in sel_o - forced)
        for p in sel_o ^ sel_g:
            assert abs(U[p] - cut) <= 2e-5 * abs(cut), f"page {p} swapped far from the cut"
        stats["near_tie_mismatch"] = stats.get("near_tie_mismatch", 0) + 1
    if near:
        stats["near_tie"] = stats.get("near_tie", 0) + 1
    # level 4: attention over the device's own pages and stored cache
    y = oracle.sparse_attention(q64, scale, dev["k"], dev["v"], got, S)
    go = f64(o[b, h])
    mx_tol, mean_tol = ATT_TOL[dtype]
    err = np.abs(go - y)
    assert err.max() <= mx_tol and err.mean() <= mean_tol, \
        f"attention[{b},{h}]: max {err.max():.3e} mean {err.mean():.3e}"
    stats["att_max"] = max(stats.get("att_max", 0.0), float(err.max()))
    stats["att_mean"] = max(stats.get("att_mean", 0.0), float(err.mean()))
    note_max("attention_max_abs_err_" + str(dtype).replace("torch.", ""), err.max())
    note_max("attention_mean_abs_err_" + str(dtype).replace("torch.", ""), err.mean())
    # end to end: the oracle's own chain from the raw inputs
    e2e = hd.query(q64, K, scale)
    if np.array_equal(e2e["idx"], got):
        err2 = np.abs(go - e2e["y"])
        assert err2.max() <= mx_tol and err2.mean() <= mean_tol, \
            f"end-to-end attention[{b},{h}]: max {err2.max():.3e} mean {err2.mean():.3e}"
        stats["e2e_same_pages"] = stats.get("e2e_same_pages", 0) + 1
    stats["e2e_overlap"] = stats.get("e2e_overlap", 0.0) + len(set(e2e["idx"].tolist()) & set(got.tolist())) / max(n, 1)
    return stats
