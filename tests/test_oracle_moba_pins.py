"""CPU pins of the MoBA part of the oracle (oracle/rqo_moba.c and the chain in oracle/__init__.py) against
what the paper and the mathematics fix.  A mean taken over the wrong rows, candidates that include the
query's own or later blocks, a missing causal mask inside the own block, a forced block left out of the
budget or a tie rule the wrong way round each fail one of these."""
import os

import numpy as np
import pytest
import torch

import oracle

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def rng(seed):
    return np.random.default_rng(seed)


def dense_causal(q_all, kst, vst, scale):
    """Textbook causal softmax attention in fp64 (torch's routine)."""
    q = torch.from_numpy(q_all)[None, None]
    k = torch.from_numpy(kst)[None, None]
    v = torch.from_numpy(vst)[None, None]
    return torch.nn.functional.scaled_dot_product_attention(q, k, v, is_causal=True, scale=scale)[0, 0].numpy()


@pytest.mark.parametrize("T,B", [(64, 8), (100, 16), (37, 5)])
def test_means_of_constant_and_linear_blocks(T, B):
    """A block of equal keys has that key as its mean; keys that grow linearly inside a block have the
    block's midpoint; the ragged last block averages its valid tokens only."""
    D = 3
    nb = (T + B - 1) // B
    r = rng(T)
    centre = r.normal(size=(nb, D))
    kst = np.repeat(centre, B, axis=0)[:T]
    np.testing.assert_allclose(oracle.block_means(kst, B), centre, rtol=1e-14)
    ramp = np.arange(T, dtype=np.float64)[:, None] * np.ones((1, D))
    m = oracle.block_means(ramp, B)
    for j in range(nb):
        lo, hi = j * B, min((j + 1) * B, T)
        assert m[j, 0] == pytest.approx((lo + hi - 1) / 2.0)


def test_one_token_blocks_route_like_a_token_top_k():
    """Blocks of one position: the representative is the key itself, so the routing is the arg-top-K of
    q . k over the positions before t (brute force with numpy), plus position 0 and position t."""
    T, D, K = 50, 6, 9
    r = rng(3)
    kst, q = r.normal(size=(T, D)), r.normal(size=D)
    means = oracle.block_means(kst, 1)
    np.testing.assert_array_equal(means, kst)
    t = 41
    got, _ = oracle.moba_route(q, means, t, 1, K)
    s = kst[:t] @ q
    order = [int(j) for j in np.argsort(-s[1:], kind="stable") + 1]      # candidates 1 .. t-1, best first
    want = sorted([0, t] + order[:K - 2])
    assert list(got) == want


@pytest.mark.parametrize("T,B,D", [(96, 16, 8), (130, 32, 4)])
def test_full_budget_is_dense_causal_attention(T, B, D):
    """With a budget that covers every block, MoBA is plain causal softmax attention."""
    r = rng(T + B)
    kst, vst, q_all = r.normal(size=(T, D)), r.normal(size=(T, D)), r.normal(size=(T, D))
    means = oracle.block_means(kst, B)
    ref = dense_causal(q_all, kst, vst, 0.3)
    nb = (T + B - 1) // B
    for t in (0, 1, B - 1, B, T // 2, T - 1):
        blocks, _ = oracle.moba_route(q_all[t], means, t, B, nb)
        assert list(blocks) == list(range(t // B + 1))
        y = oracle.moba_attention(q_all[t], 0.3, kst, vst, blocks, t, B)
        np.testing.assert_allclose(y, ref[t], rtol=1e-10, atol=1e-12)


def test_forced_blocks_causality_and_budget_count():
    T, B, D, K = 256, 16, 8, 5
    r = rng(11)
    kst, vst = r.normal(size=(T, D)), r.normal(size=(T, D))
    means = oracle.block_means(kst, B)
    for t in (17, 100, 255):
        q = r.normal(size=D)
        blocks, _ = oracle.moba_route(q, means, t, B, K)
        bt = t // B
        assert len(blocks) == min(K, bt + 1)
        assert blocks[0] == 0 and blocks[-1] == bt and (np.diff(blocks) > 0).all()
        # nothing after the query is attended: changing later keys and values changes nothing
        k2, v2 = kst.copy(), vst.copy()
        k2[t + 1:] += 100.0
        v2[t + 1:] -= 100.0
        y1 = oracle.moba_attention(q, 0.5, kst, vst, blocks, t, B)
        y2 = oracle.moba_attention(q, 0.5, k2, v2, blocks, t, B)
        np.testing.assert_array_equal(y1, y2)
        # the own block is cut at t: a huge value inside the own block but after t does not leak
        if (t + 1) % B:
            assert np.isfinite(y2).all()


def test_planted_block_is_selected_and_ties_go_to_the_lower_block():
    T, B, D, K = 512, 32, 16, 4
    r = rng(5)
    kst = 0.1 * r.normal(size=(T, D))
    q = r.normal(size=D)
    planted = 7
    kst[planted * B:(planted + 1) * B] += 2.0 * q / np.linalg.norm(q)
    means = oracle.block_means(kst, B)
    blocks, _ = oracle.moba_route(q, means, T - 1, B, K)
    assert planted in blocks
    # equal representatives: the lower blocks win
    same = np.tile(r.normal(size=(1, D)), (T, 1))
    means2 = oracle.block_means(same, B)
    blocks2, _ = oracle.moba_route(q, means2, T - 1, B, K)
    assert list(blocks2) == [0, 1, 2, T // B - 1]


def test_paper_budget_arithmetic():
    """K blocks per query at the 4K context are the budgets the paper names."""
    rows = [l.split() for l in open(os.path.join(GOLDEN, "moba_budgets.txt")) if l.strip() and not l.startswith("#")]
    assert len(rows) == 5
    for ctx, blk, K, num, den in (map(int, r) for r in rows):
        nb = ctx // blk
        assert K * den == nb * num
        # the last query of the prompt attends exactly K blocks, first and own included
        r = rng(K + blk)
        kst = r.normal(size=(ctx, 4))
        means = oracle.block_means(kst, blk)
        blocks, _ = oracle.moba_route(r.normal(size=4), means, ctx - 1, blk, K)
        assert len(blocks) == K and blocks[0] == 0 and blocks[-1] == nb - 1
