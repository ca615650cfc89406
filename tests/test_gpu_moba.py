"""GPU parity of the MoBA-style block-sparse prefill attention on the decayed states (App. A.1, MoBA
paragraph; Sec. 2.2) against the fp64 oracle, level by level, for sampled (head, position) pairs:

  representatives : the device's fp32 block means vs the oracle's on the device's stored keys, within 1e-5
                    of the head's largest |mean| (an fp32 sum of at most 128 stored values)
  routing         : the oracle's scores and TopK run on the DEVICE's means and the same query bits must give
                    the same blocks, index for index (ascending; equal scores to the lower block), except where
                    the oracle flags a near-tie at the cut, which is counted
  attention       : the oracle's attention over the device's blocks and stored cache vs the device output,
                    within the attention tolerance of the decode path
and, with a budget that covers every block, against textbook causal softmax attention for every position.
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


def prompt_queries(w, T, seed):
    g = torch.Generator(device=DEV)
    g.manual_seed(seed)
    return torch.randn(w.B, T, w.H, w.D, generator=g, device=DEV, dtype=torch.float32).to(w.dtype)


def run_moba(w, block, K, scale=0.0, q=None, kvg=None):
    T = w.T
    cache = rq.Cache(w.B, w.H, w.D, w.S, T, w.dtype, w.gdtype)
    k, v, g = kvg if kvg is not None else wl.make_prefill(w, DEV, T)
    rq.rq_build_cache(cache.handle, k, v, g)
    q = prompt_queries(w, T, w.seed + 5) if q is None else q
    nb = (T + block - 1) // block
    o = torch.full((w.B, T, w.H, w.D), float("nan"), dtype=w.dtype, device=DEV)
    blocks = torch.full((w.B, w.H, T, K), -7, dtype=torch.int32, device=DEV)
    means = torch.empty(w.B, w.H, nb, w.D, dtype=torch.float32, device=DEV)
    scratch = torch.empty(rq.rq_moba_scratch_bytes(cache.handle, block, K), dtype=torch.uint8, device=DEV)
    rq.rq_moba_prefill(cache.handle, q, block, K, scale, o, blocks, means, scratch)
    torch.cuda.synchronize()
    assert rq.rq_device_status(cache.handle) == rq.RQ_OK
    return cache, q, o, blocks, means


def sample_positions(T, block, n, seed):
    edge = {0, 1, block - 1, block, block + 1, 2 * block - 1, 2 * block, T - 1, T - 2, (T - 1) // block * block}
    r = np.random.default_rng(seed)
    pos = sorted({p for p in edge if 0 <= p < T} | set(int(x) for x in r.integers(0, T, n)))
    return pos


def check_head(w, cache, q, o, blocks, means, b, h, block, K, scale, positions):
    dev = parity.device_head_arrays(cache, b, h)
    T = len(cache)
    m_dev = parity.f64(means[b, h])
    m_ref = oracle.block_means(dev["k"], block)
    tol = 1e-5 * np.abs(m_ref).max() + 1e-7
    err = np.abs(m_dev - m_ref).max()
    parity.note_max("moba_means_err_over_max", err / np.abs(m_ref).max())
    assert err <= tol, f"means[{b},{h}]: {err:.3e} > {tol:.3e}"
    mx_tol, mean_tol = parity.ATT_TOL[w.dtype]
    for t in positions:
        qt = parity.f64(q[b, t, h])
        got = blocks[b, h, t].cpu().numpy().astype(np.int64)
        want, near = oracle.moba_route(qt, m_dev, t, block, K)
        n = len(want)
        assert n == min(K, t // block + 1)
        assert (got[n:] == -1).all() and (np.diff(got[:n]) > 0).all()
        assert got[0] == 0 and got[n - 1] == t // block, "the first block and the query's own block are always attended"
        parity.note_count("moba_queries_checked")
        if not np.array_equal(got[:n], want):
            assert near, f"head ({b},{h}), position {t}: blocks differ from the oracle's without a near-tie at the cut"
            parity.note_count("moba_near_tie_queries")
            assert len(np.setdiff1d(got[:n], want)) <= 2
        y = oracle.moba_attention(qt, scale, dev["k"], dev["v"], got[:n], t, block)
        e = np.abs(parity.f64(o[b, t, h]) - y)
        parity.note_max(f"moba_attention_max_err_{'bf16' if w.dtype == torch.bfloat16 else 'f32'}", e.max())
        assert e.max() <= mx_tol and e.mean() <= mean_tol, f"head ({b},{h}), position {t}: attention error {e.max():.3e}"


@pytest.mark.parametrize("block,K", [(64, 16), (64, 8), (64, 4), (128, 8), (128, 4)])
def test_paper_settings_on_4k_prompts(block, K):
    """The paper's settings: prompts of 4096 tokens, block 64 with 16 / 8 / 4 blocks per query, block 128 with
    8 / 4 (tests/golden/moba_budgets.txt)."""
    w = wl.Workload("moba-4k", B=1, H=8, D=128, T=4096, seed=31)
    cache, q, o, blocks, means = run_moba(w, block, K)
    assert not torch.isnan(o.float()).any()
    for h in (0, 3, 7):
        check_head(w, cache, q, o, blocks, means, 0, h, block, K, w.D ** -0.5, sample_positions(w.T, block, 14, h))


@pytest.mark.parametrize("B,H,D,T,S,block,K,dtype", [
    (1, 2, 64, 1000, 16, 64, 5, torch.float32),       # ragged last block, narrow heads
    (2, 3, 128, 777, 16, 64, 3, torch.bfloat16),      # odd sizes, two batch items
    (1, 2, 128, 640, 64, 128, 2, torch.bfloat16),     # pages of 64, the smallest budget: first and own block only
    (1, 2, 64, 2049, 64, 64, 6, torch.bfloat16),      # one position into a new block
    (1, 1, 128, 50, 16, 64, 4, torch.float32),        # a prompt shorter than one block
    (1, 2, 128, 1500, 16, 256, 3, torch.bfloat16),    # blocks of 256
    (1, 2, 64, 12000, 16, 64, 9, torch.bfloat16),     # 188 blocks: representatives read from global memory, arg-max rounds
    (1, 1, 128, 9000, 16, 64, 20, torch.float32),     # the same on an fp32 cache
    (1, 2, 128, 65536, 16, 64, 64, torch.bfloat16),   # 1024 blocks, 64 per query: a long prompt at budget 1/16
    (1, 1, 64, 131072, 64, 128, 16, torch.bfloat16),  # 1024 blocks of 128 on pages of 64
])
def test_shapes_blocks_and_ragged_sizes(B, H, D, T, S, block, K, dtype):
    w = wl.Workload("moba-small", B=B, H=H, D=D, T=T, S=S, dtype=dtype, seed=T + K)
    cache, q, o, blocks, means = run_moba(w, block, K, scale=0.21)
    assert not torch.isnan(o.float()).any()
    for b in range(B):
        for h in range(H):
            check_head(w, cache, q, o, blocks, means, b, h, block, K, 0.21, sample_positions(T, block, 10, b * 7 + h))


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_full_budget_is_dense_causal_attention(dtype):
    """A budget that covers every block: every position attends everything before it; compared with torch's causal
    softmax attention in fp64 on the device's stored cache, for all positions."""
    w = wl.Workload("moba-dense", B=1, H=2, D=64, T=900, dtype=dtype, seed=8)
    block = 64
    nb = (w.T + block - 1) // block
    cache, q, o, blocks, means = run_moba(w, block, nb)
    mx_tol, mean_tol = parity.ATT_TOL[dtype]
    for h in range(w.H):
        dev = parity.device_head_arrays(cache, 0, h)
        qq = torch.from_numpy(parity.f64(q[0, :, h]))[None, None]
        kk = torch.from_numpy(dev["k"])[None, None]
        vv = torch.from_numpy(dev["v"])[None, None]
        ref = torch.nn.functional.scaled_dot_product_attention(qq, kk, vv, is_causal=True)[0, 0].numpy()
        e = np.abs(parity.f64(o[0, :, h]) - ref)
        assert e.max() <= mx_tol and e.mean() <= mean_tol, f"head {h}: {e.max():.3e}"
        got = blocks[0, h].cpu().numpy()
        for t in (0, 63, 64, 500, 899):
            n = t // block + 1
            assert (got[t, :n] == np.arange(n)).all() and (got[t, n:] == -1).all()


def test_planted_blocks_are_routed_to():
    """Keys of a few blocks carry a component along a later query: those blocks are among the chosen ones."""
    w = wl.Workload("moba-planted", B=1, H=4, D=128, T=4096, seed=12, gate_zero=True)   # zero gate: the cache holds k itself
    block, K = 64, 4
    k, v, g = wl.make_prefill(w, DEV, w.T)
    q = prompt_queries(w, w.T, 77)
    t = w.T - 1
    planted = {0: [5, 40], 1: [17, 33], 2: [2, 61], 3: [9, 10]}
    kf = k.float()
    for h, js in planted.items():
        qn = q[0, t, h].float()
        qn = qn / qn.norm()
        for j in js:
            kf[0, j * block:(j + 1) * block, h, :] += 1.5 * qn
    k = kf.to(w.dtype)
    cache, q, o, blocks, means = run_moba(w, block, K, q=q, kvg=(k, v, g))
    for h, js in planted.items():
        got = blocks[0, h, t].cpu().numpy().tolist()
        assert got[0] == 0 and got[-1] == t // block
        assert set(js) <= set(got), f"head {h}: planted blocks {js} not among {got}"


def test_argument_checks():
    w = wl.Workload("moba-args", B=1, H=2, D=64, T=300, dtype=torch.float32, seed=4)
    cache = rq.Cache(w.B, w.H, w.D, w.S, w.T, w.dtype, w.gdtype)
    k, v, g = wl.make_prefill(w, DEV, w.T)
    rq.rq_build_cache(cache.handle, k, v, g)
    q = prompt_queries(w, w.T, 1)
    o = torch.empty_like(q)
    scratch = torch.empty(rq.rq_moba_scratch_bytes(cache.handle, 64, 4), dtype=torch.uint8, device=DEV)
    for block, K in ((32, 4), (96, 4), (64, 1), (64, 0)):
        with pytest.raises(rq.RqError) as e:
            rq.rq_moba_prefill(cache.handle, q, block, K, 0.0, o, None, None, scratch)
        assert e.value.status == rq.RQ_ERR_INVALID_ARG
    empty = rq.Cache(w.B, w.H, w.D, w.S, w.T, w.dtype, w.gdtype)
    with pytest.raises(rq.RqError) as e:
        rq.rq_moba_prefill(empty.handle, q, 64, 4, 0.0, o, None, None, scratch)
    assert e.value.status == rq.RQ_ERR_INVALID_ARG


def test_unused_cache_memory_full_of_nans_does_not_leak():
    """A cache much larger than the prompt whose memory holds NaN bit patterns everywhere the prefill did not write:
    copies of whole chunks read some of it (the pages after the prompt's end); neither the routing nor the attention may
    pick any of it up."""
    w = wl.Workload("moba-nan", B=1, H=2, D=128, T=1000, seed=17)
    block, K = 64, 4
    cache = rq.Cache(w.B, w.H, w.D, w.S, 4096, w.dtype, w.gdtype)
    cache.kv.fill_(0xFF)
    cache.meta.fill_(0xFF)
    k, v, g = wl.make_prefill(w, DEV, w.T)
    rq.rq_build_cache(cache.handle, k, v, g)
    q = prompt_queries(w, w.T, 3)
    o = torch.full((w.B, w.T, w.H, w.D), float("nan"), dtype=w.dtype, device=DEV)
    blocks = torch.empty(w.B, w.H, w.T, K, dtype=torch.int32, device=DEV)
    means = torch.empty(w.B, w.H, (w.T + block - 1) // block, w.D, dtype=torch.float32, device=DEV)
    scratch = torch.empty(rq.rq_moba_scratch_bytes(cache.handle, block, K), dtype=torch.uint8, device=DEV)
    rq.rq_moba_prefill(cache.handle, q, block, K, 0.0, o, blocks, means, scratch)
    torch.cuda.synchronize()
    assert torch.isfinite(o.float()).all() and torch.isfinite(means).all()
    for h in range(w.H):
        check_head(w, cache, q, o, blocks, means, 0, h, block, K, w.D ** -0.5, sample_positions(w.T, block, 8, h))
