"""The workspace-free attention entry point against the ordinary one.

`rq_attend_pages_noalloc` is for callers that must not allocate device memory (for instance a
plug-in in an engine that owns the whole GPU): it keeps the kernel's partial results and
counters in a fixed array inside the library instead of a caller-provided workspace.  Here it
is called twice in a row through the C ABI on the same inputs as `rq_attend_pages`; the array
keeps the first call's contents, so the second call also shows that what must start at zero is
cleared.  This file sorts after the other test files on purpose: a run that stops at the first
failure has then already run everything else.
"""
import pytest
import torch

import paper_2605_28640_b200 as rq
from paper_2605_28640_b200 import workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.mark.parametrize("B,H,D,S,T,dtype,den", [
    (1, 32, 128, 16, 20000, torch.bfloat16, 16),     # one CTA group per head
    (4, 8, 64, 16, 500, torch.float32, 16),          # fewer CTAs than heads: warps sweep over the heads
])
def test_noalloc_matches_workspace_version(B, H, D, S, T, dtype, den):
    w = wl.Workload("noalloc", B=B, H=H, D=D, T=T, S=S, budget_den=den, dtype=dtype, seed=123)
    k, v, g = wl.make_prefill(w, DEV)
    cache = rq.Cache(w.B, w.H, w.D, w.S, w.T, w.dtype)
    rq.rq_build_cache(cache.handle, k, v, g)
    q = wl.make_query(w, DEV)
    K = w.budget_pages()
    idx = torch.empty(w.B, w.H, K, dtype=torch.int32, device=DEV)
    rq.rq_select_pages(cache.handle, q, K, None, idx)
    ref = torch.empty(w.B, w.H, w.D, dtype=w.dtype, device=DEV)
    rq.rq_attend_pages(cache.handle, q, idx, K, 0.0, ref)
    torch.cuda.synchronize()
    tol = 2e-2 if dtype == torch.bfloat16 else 1e-4
    for call in range(2):
        out = torch.full_like(ref, float("nan"))
        rq.rq_attend_pages_noalloc(cache.cfg, cache.kv, len(cache), q, idx, K, 0.0, out)
        torch.cuda.synchronize()
        err = (out.float() - ref.float()).abs().max().item()
        assert err <= tol, f"call {call}: max difference {err:.3e}"


def test_noalloc_refuses_shapes_beyond_its_scratch():
    """Many heads with few tiles each need one partial record per warp and head: too much for 4 MiB.
    The refusal comes from the host before anything is enqueued, so dummy pointers are enough."""
    cfg = rq.rq_config(64, 64, 128, 16, 4096, rq.RQ_BF16, rq.RQ_BF16, 1, 1, 256, 0)
    buf = torch.zeros(1024, dtype=torch.uint8, device=DEV)
    with pytest.raises(rq.RqError) as e:
        rq.rq_attend_pages_noalloc(cfg, buf, 4096, buf, buf, 64, 0.0, buf)
    assert e.value.status == rq.RQ_ERR_CAPACITY
    with pytest.raises(rq.RqError) as e:
        rq.rq_attend_pages_noalloc(cfg, buf, 0, buf, buf, 64, 0.0, buf)
    assert e.value.status == rq.RQ_ERR_INVALID_ARG
