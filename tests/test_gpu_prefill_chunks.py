"""GPU parity of the prefill's time-chunked form (Eq. 1 over a long prompt of few heads: the sequence of a channel
group is cut into chunks that run on different SMs, every chunk entering with the state that the chunks before it
leave) against the fp64 oracle: final state, stored cache and page bounds of every head, and that a cache built in
two calls, the second one long enough to be chunked, equals the oracle's as well."""
import numpy as np
import pytest
import torch

import paper_2605_28640_b200 as rq
from paper_2605_28640_b200 import workloads as wl

import parity

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.mark.parametrize("B,H,D,T,S,dtype,resets", [
    (1, 2, 64, 40000, 16, torch.bfloat16, False),     # 4 channel groups
    (1, 1, 128, 33000, 16, torch.bfloat16, True),     # state resets inside chunks
    (2, 2, 128, 20011, 64, torch.bfloat16, False),    # pages of 64, ragged end
    (1, 3, 64, 25000, 16, torch.float32, False),      # fp32 storage: the stored value is the state itself
])
def test_long_prompt_of_few_heads(B, H, D, T, S, dtype, resets):
    w = wl.Workload("chunks", B=B, H=H, D=D, T=T, S=S, dtype=dtype, seed=T % 97, resets=resets)
    cache = rq.Cache(B, H, D, S, T + 8, dtype, w.gdtype)
    k, v, g = wl.make_prefill(w, DEV, T)
    rq.rq_build_cache(cache.handle, k, v, g)
    torch.cuda.synchronize()
    assert rq.rq_device_status(cache.handle) == rq.RQ_OK and len(cache) == T
    for b in range(B):
        for h in range(H):
            hd = parity.oracle_head(w, k, v, g, b, h, T + 8)
            parity.check_cache_level(cache, hd, b, h, dtype)
    # decoding continues from the chunked prefill's state
    q = wl.make_query(w, DEV, 0)
    kt, vt, gt = wl.make_token(w, DEV, 0)
    K = w.pages(T + 1) // 8
    o = torch.empty(B, H, D, dtype=dtype, device=DEV)
    idx = torch.empty(B, H, K, dtype=torch.int32, device=DEV)
    rq.rq_decode_step(cache.handle, q, kt, vt, gt, K, 0.0, o, idx)
    torch.cuda.synchronize()
    hd = parity.oracle_head(w, k, v, g, 0, 0, T + 8)
    hd.append(parity.f64(kt[0, 0]), parity.f64(vt[0, 0]), parity.f64(gt[0, 0]))
    dev = parity.check_cache_level(cache, hd, 0, 0, dtype)
    stats = {}
    parity.check_query_level(dev, hd, cache, 0, 0, q, K, D ** -0.5, o, idx, None, dtype, stats)


def test_second_call_is_chunked_and_starts_inside_a_page():
    """5003 tokens first (one chunk), then 30000 more (chunked, starting inside a page and a tile)."""
    w = wl.Workload("chunks2", B=1, H=2, D=64, T=35003, seed=13)
    cache = rq.Cache(1, 2, 64, 16, w.T, w.dtype, w.gdtype)
    k, v, g = wl.make_prefill(w, DEV, w.T)
    rq.rq_build_cache(cache.handle, k[:, :5003], v[:, :5003], g[:, :5003])
    rq.rq_build_cache(cache.handle, k[:, 5003:], v[:, 5003:], g[:, 5003:])
    torch.cuda.synchronize()
    assert len(cache) == w.T
    for h in range(2):
        hd = parity.oracle_head(w, k, v, g, 0, h, w.T)
        parity.check_cache_level(cache, hd, 0, h, w.dtype)


def test_chunked_build_is_reproducible():
    w = wl.Workload("chunks3", B=1, H=2, D=128, T=30000, seed=3)
    k, v, g = wl.make_prefill(w, DEV, w.T)
    outs = []
    for _ in range(2):
        cache = rq.Cache(1, 2, 128, 16, w.T, w.dtype, w.gdtype)
        rq.rq_build_cache(cache.handle, k, v, g)
        torch.cuda.synchronize()
        outs.append((cache.kv_view().clone(), cache.meta_view().clone(), cache.state_view().clone()))
    for a, b in zip(*outs):
        assert torch.equal(a, b)
