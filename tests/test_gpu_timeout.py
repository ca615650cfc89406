"""The bounded device-side waits, made to run out without faulting or hanging anything.

Every wait of the kernels for an asynchronous copy is a bounded number of polls.  With the testing
aid rq_cache.reserved[1] < 0 that number is zero, so the first wait of every warp gives up although
its copy is on its way: the warp records RQ_ERR_TIMEOUT, lets every copy it has in flight land (with
the usual bound), takes no more work and the kernel returns.  The host then reads the status once,
finds it cleared afterwards, and after rq_cache_reset the same cache works again."""
import pytest
import torch

import paper_2605_28640_b200 as rq
from paper_2605_28640_b200 import workloads as wl

import parity

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.mark.parametrize("path", [1, 2])        # separate kernels; the whole step as one launch
def test_wait_that_runs_out_is_reported_and_the_cache_recovers(path):
    w = wl.Workload("timeout", B=2, H=8, D=128, T=1300, budget_den=8, seed=3)
    cap = w.T + 8
    cache = rq.Cache(w.B, w.H, w.D, w.S, cap, w.dtype, max_budget_pages=w.pages(cap))
    cache.handle.reserved[2] = path
    k, v, g = wl.make_prefill(w, DEV, w.T - 1)
    q = wl.make_query(w, DEV)
    kt, vt, gt = wl.make_token(w, DEV)
    K = w.budget_pages()
    o = torch.zeros(w.B, w.H, w.D, dtype=w.dtype, device=DEV)

    rq.rq_build_cache(cache.handle, k, v, g)
    cache.handle.reserved[1] = -1                     # no poll at all: every first wait gives up
    rq.rq_decode_step(cache.handle, q, kt, vt, gt, K, 0.0, o)
    torch.cuda.synchronize()                          # the call returns and the kernels end
    assert rq.rq_device_status(cache.handle) == rq.RQ_ERR_TIMEOUT
    assert rq.rq_device_status(cache.handle) == rq.RQ_OK          # reading cleared it
    assert rq.rq_status_string(rq.RQ_ERR_TIMEOUT) == "device-side wait timed out"

    # back to the built-in limit: after a reset the cache is as good as new
    cache.handle.reserved[1] = 0
    rq.rq_cache_reset(cache.handle)
    rq.rq_build_cache(cache.handle, k, v, g)
    idx = torch.full((w.B, w.H, K), -7, dtype=torch.int32, device=DEV)
    rq.rq_decode_step(cache.handle, q, kt, vt, gt, K, 0.0, o, idx)
    torch.cuda.synchronize()
    assert rq.rq_device_status(cache.handle) == rq.RQ_OK
    stats = {}
    for (b, h) in [(0, 0), (1, 7)]:
        hd = parity.oracle_head(w, k, v, g, b, h, cap)
        hd.append(parity.f64(kt[b, h]), parity.f64(vt[b, h]), parity.f64(gt[b, h]))
        dev = parity.check_cache_level(cache, hd, b, h, w.dtype)
        parity.check_query_level(dev, hd, cache, b, h, q, K, w.D ** -0.5, o, idx, None, w.dtype, stats)
    assert stats["heads"] == 2
