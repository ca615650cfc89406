"""Host-side instrumentation for the paper's two hypotheses about query-aware selection
(Sec. 2.3): the strict head-level hit rate and the random selector.

Nothing here computes attention: a random page list goes to `rq_attend_pages`, which takes
caller-chosen pages, and hit rates are counted from the page lists `rq_decode_step` returns.
"""
import torch


def random_pages(B, H, P, K, seed, device="cpu"):
    """Random selector (Sec. 2.3, H2): for every (batch, head) a uniform K-subset of the P pages,
    ascending, as int32 [B, H, K]; K >= P gives every page.  Seeds are independent draws."""
    K = min(K, P)
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    out = torch.empty(B, H, K, dtype=torch.int32)
    for b in range(B):
        for h in range(H):
            out[b, h] = torch.randperm(P, generator=g)[:K].sort().values.to(torch.int32)
    return out.to(device)


def head_hits(selected_steps, golden_pages):
    """Strict head-level hit (Sec. 2.3, H1): Hit_h = 1 iff at EVERY decode step the golden page of
    head h is among the pages selected for it.

    selected_steps: list over decode steps of int tensors [B, H, K] (unused entries -1)
    golden_pages:   int tensor [B, H] (one golden page per head) or [B, H, n] (all n must be hit)
    returns a bool tensor [B, H]
    """
    gold = golden_pages if golden_pages.dim() == 3 else golden_pages[..., None]
    gold = gold.to("cpu", torch.int64)
    hit = torch.ones(gold.shape[:2], dtype=torch.bool)
    for sel in selected_steps:
        sel = sel.to("cpu", torch.int64)
        present = (sel[:, :, None, :] == gold[:, :, :, None]).any(dim=-1)      # [B, H, n]
        hit &= present.all(dim=-1)
    return hit


def hit_rate(selected_steps, golden_pages):
    """Fraction of heads with Hit_h = 1."""
    return head_hits(selected_steps, golden_pages).float().mean().item()
