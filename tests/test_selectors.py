"""CPU tests of the selection instrumentation (random selector, strict head-level hit rate)."""
import math

import torch

from paper_2605_28640_b200 import selectors


def test_random_pages_are_uniform_k_subsets():
    B, H, P, K = 2, 3, 40, 7
    a = selectors.random_pages(B, H, P, K, seed=1)
    assert a.shape == (B, H, K) and a.dtype == torch.int32
    assert (a[..., 1:] > a[..., :-1]).all() and a.min() >= 0 and a.max() < P      # ascending, distinct, in range
    assert torch.equal(a, selectors.random_pages(B, H, P, K, seed=1))             # a seed names one draw
    assert not torch.equal(a, selectors.random_pages(B, H, P, K, seed=2))
    # every page is chosen with probability K / P: chi-square over many draws stays small
    n = 4000
    counts = torch.zeros(P)
    for s in range(n // (B * H)):
        counts += torch.bincount(selectors.random_pages(B, H, P, K, seed=100 + s).flatten().long(), minlength=P)
    draws = (n // (B * H)) * B * H
    expect = draws * K / P
    chi2 = ((counts - expect) ** 2 / expect).sum().item()
    assert chi2 < 2.0 * P, chi2                                                   # mean P - 1, sd about sqrt(2 P)
    assert torch.equal(selectors.random_pages(1, 1, 5, 9, seed=0)[0, 0], torch.arange(5, dtype=torch.int32))


def test_head_hits_is_strict_over_steps():
    # two heads, three steps; head 0 always holds page 4, head 1 misses page 9 at the second step
    steps = [torch.tensor([[[1, 4, 7], [2, 9, -1]]]), torch.tensor([[[4, 5, 6], [2, 3, 8]]]),
             torch.tensor([[[0, 4, -1], [9, 10, 11]]])]
    gold = torch.tensor([[4, 9]])
    hits = selectors.head_hits(steps, gold)
    assert hits.tolist() == [[True, False]]
    assert selectors.hit_rate(steps, gold) == 0.5
    # several golden pages per head: all of them, at every step
    gold2 = torch.tensor([[[4, 7], [2, 9]]])
    assert selectors.head_hits(steps[:1], gold2).tolist() == [[True, True]]
    assert selectors.head_hits(steps[:2], gold2).tolist() == [[False, False]]


def test_random_selector_hit_probability_matches_closed_form():
    """A uniform K-subset of P pages holds a given page with probability K / P, so a head is hit
    over t independent steps with probability (K / P)^t."""
    B, H, P, K, t = 4, 64, 32, 8, 2
    gold = torch.randint(0, P, (B, H), generator=torch.Generator().manual_seed(3))
    rates = []
    for rep in range(40):
        steps = [selectors.random_pages(B, H, P, K, seed=1000 * rep + s) for s in range(t)]
        rates.append(selectors.hit_rate(steps, gold))
    mean = sum(rates) / len(rates)
    p = (K / P) ** t
    sd = math.sqrt(p * (1 - p) / (B * H * len(rates)))
    assert abs(mean - p) < 5 * sd, (mean, p)
