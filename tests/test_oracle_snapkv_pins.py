"""CPU pins of the SnapKV part of the oracle (oracle/rqo_snapkv.c) against what the paper and the
mathematics fix: closed forms, brute force in numpy, textbook softmax attention, and the budget
arithmetic the paper prints.  A dropped causal mask, a window aligned to the wrong end, importance
taken as a maximum instead of a sum, a tie rule the wrong way round or a window left out of the
retained set each fail one of these."""
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def rng(seed):
    return np.random.default_rng(seed)


def brute_importance(qw, kst, scale):
    """Row-by-row causal softmax in numpy, written independently of the C code."""
    W, T = qw.shape[0], kst.shape[0]
    imp = np.zeros(T)
    for i in range(W):
        t = T - W + i
        s = scale * kst[: t + 1] @ qw[i]
        w = np.exp(s - s.max())
        imp[: t + 1] += w / w.sum()
    return imp


@pytest.mark.parametrize("T,W,D", [(40, 8, 4), (64, 64, 8), (19, 1, 3), (100, 16, 16)])
def test_importance_matches_brute_force_and_sums_to_window(T, W, D):
    r = rng(T + W)
    qw, kst = r.normal(size=(W, D)), r.normal(size=(T, D))
    imp = oracle.snapkv_importance(qw, 0.7, kst)
    np.testing.assert_allclose(imp, brute_importance(qw, kst, 0.7), rtol=1e-12, atol=1e-15)
    # every query's weights sum to one
    assert abs(imp.sum() - W) < 1e-10
    assert (imp >= 0).all()


def test_causal_mask_and_window_alignment():
    """The query of position t must not see positions after t: the last position gets weight from
    the last query only, and position T-W+i from the queries i .. W-1."""
    T, W, D = 12, 4, 2
    qw = np.zeros((W, D))                       # zero queries: uniform weights over what each one sees
    kst = rng(1).normal(size=(T, D))
    imp = oracle.snapkv_importance(qw, 1.0, kst)
    expect = np.zeros(T)
    for i in range(W):
        t = T - W + i
        expect[: t + 1] += 1.0 / (t + 1)
    np.testing.assert_allclose(imp, expect, rtol=1e-13)
    assert imp[T - 1] == pytest.approx(1.0 / T)
    # a huge key at the last position draws only the last query
    kst2 = np.zeros((T, D)); kst2[T - 1, 0] = 50.0
    qw2 = np.zeros((W, D)); qw2[:, 0] = 1.0
    imp2 = oracle.snapkv_importance(qw2, 1.0, kst2)
    assert imp2[T - 1] == pytest.approx(1.0, abs=1e-12)
    assert imp2[: T - 1].sum() == pytest.approx(W - 1.0, abs=1e-9)


def test_window_of_one_query_is_top_k_of_one_softmax_row():
    T, D, keep = 50, 6, 9
    r = rng(5)
    q, kst = r.normal(size=(1, D)), r.normal(size=(T, D))
    imp = oracle.snapkv_importance(q, 1.0, kst)
    s = kst @ q[0]
    w = np.exp(s - s.max()); w /= w.sum()
    np.testing.assert_allclose(imp, w, rtol=1e-12)
    idx, _ = oracle.snapkv_select(imp, 1, keep)
    # brute force: the window (last position) + the keep-1 largest of the rest
    order = sorted(range(T - 1), key=lambda j: (-w[j], j))[: keep - 1]
    assert idx.tolist() == sorted(order + [T - 1])


def test_selection_against_full_sort_with_ties_and_window_always_kept():
    r = rng(9)
    T, W = 300, 16
    imp = r.integers(0, 6, T).astype(np.float64)       # heavy ties
    for keep in (W, W + 1, 40, 150, 299):
        idx, _ = oracle.snapkv_select(imp, W, keep)
        assert len(idx) == keep and (np.diff(idx) > 0).all()
        assert set(range(T - W, T)) <= set(idx.tolist())
        order = sorted(range(T - W), key=lambda j: (-imp[j], j))[: keep - W]
        assert idx.tolist() == sorted(order + list(range(T - W, T)))
    # keep >= T keeps everything; keep below the window keeps the newest positions
    assert oracle.snapkv_select(imp, W, T)[0].tolist() == list(range(T))
    assert oracle.snapkv_select(imp, W, T + 5)[0].tolist() == list(range(T))
    assert oracle.snapkv_select(imp, W, 5)[0].tolist() == list(range(T - 5, T))


def test_equal_keys_keep_the_lowest_positions():
    """All keys equal: every query spreads its weight evenly, positions before the window all get the
    same importance, so the lowest positions are retained besides the window."""
    T, W, D = 80, 8, 4
    kst = np.ones((T, D))
    qw = rng(2).normal(size=(W, D))
    imp = oracle.snapkv_importance(qw, 1.0, kst)
    assert np.ptp(imp[: T - W]) < 1e-15
    idx, near = oracle.snapkv_select(imp, W, 20)
    assert idx.tolist() == list(range(12)) + list(range(T - W, T))
    assert near is True


def test_near_tie_flag():
    imp = np.array([5.0, 1.0, 1.0 + 5e-6, 0.5, 9.0, 9.0])
    idx, near = oracle.snapkv_select(imp, 2, 4)         # window = positions 4, 5; want two of 0..3
    assert idx.tolist() == [0, 2, 4, 5] and near is True
    imp[1] = 0.9
    assert oracle.snapkv_select(imp, 2, 4)[1] is False


def test_token_attention_is_textbook_softmax_and_matches_page_attention():
    r = rng(3)
    T, D, S = 70, 8, 16
    k, v, q = r.normal(size=(T, D)), r.normal(size=(T, D)), r.normal(size=D)
    s = (k @ q) * 0.35
    w = np.exp(s - s.max())
    dense = (w[:, None] * v).sum(0) / w.sum()
    np.testing.assert_allclose(oracle.token_attention(q, 0.35, k, v, np.arange(T)), dense, rtol=1e-12)
    # a subset of whole pages gives what the page-list attention gives
    pages = np.array([0, 2, 4])
    tok = np.concatenate([np.arange(p * S, min((p + 1) * S, T)) for p in pages])
    np.testing.assert_allclose(oracle.token_attention(q, 0.35, k, v, tok),
                               oracle.sparse_attention(q, 0.35, k, v, pages, S), rtol=1e-12)
    # one token: its value row
    np.testing.assert_allclose(oracle.token_attention(q, 0.35, k, v, np.array([17])), v[17], rtol=1e-14)


def test_budget_arithmetic_from_the_paper():
    for line in open(os.path.join(GOLDEN, "snapkv_budgets.txt")):
        if line.startswith("#") or not line.strip():
            continue
        ctx, window, K, num, den = map(int, line.split())
        assert K * den == ctx * num
        r = rng(K)
        imp = oracle.snapkv_importance(r.normal(size=(window, 8)), 1.0, r.normal(size=(ctx, 8)))
        idx, _ = oracle.snapkv_select(imp, window, K)
        assert len(idx) == K and set(range(ctx - window, ctx)) <= set(idx.tolist())
