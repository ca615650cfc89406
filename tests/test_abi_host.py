"""CPU-only checks of the C-ABI library: it loads, exports every function the
header declares, and its host-side argument validation answers before any
CUDA call (no compute is launched here)."""
import ctypes as C
import os
import re

import pytest

import paper_2605_28640_b200 as rq
from paper_2605_28640_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build_library()
    return binding.lib()


def declared_functions():
    names = []
    for fn in sorted(os.listdir(os.path.join(ROOT, "include"))):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            names += re.findall(r"^RQ_API\s+[\w\s\*]+?\b(rq_\w+)\s*\(", text, flags=re.M)
    return names


def test_every_declared_symbol_is_exported_and_bound(lib):
    names = declared_functions()
    assert len(names) >= 12
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in include/ but not exported"
    assert set(names) == set(binding.SIGNATURES), "binding and header disagree on the function list"


def test_version_and_status_strings(lib):
    assert rq.rq_version() == 1
    assert rq.rq_status_string(rq.RQ_OK) == "ok"
    seen = {rq.rq_status_string(s) for s in range(6)}
    assert len(seen) == 6 and rq.rq_status_string(99) == "unknown status"


def cfg(**kw):
    base = dict(batch=1, heads=32, head_dim=128, page_size=16, capacity_tokens=131072, dtype=rq.RQ_BF16,
                gate_dtype=rq.RQ_BF16, n_sink_pages=1, n_local_pages=1, max_budget_pages=512, reserved=0)
    base.update(kw)
    return rq.rq_config(**base)


def test_sizes_follow_the_documented_layouts(lib):
    kv, meta, st, ws = rq.rq_sizes(cfg())
    assert kv == 32 * 8192 * 2 * 16 * 128 * 2          # [B][H][P][2][S][D] bf16 = 2 GiB
    assert meta == 32 * 8192 * 2 * 128 * 2             # [B][H][P][2][D]    bf16 = 128 MiB
    assert st == 32 * 2 * 128 * 4
    assert ws % 256 == 0 and ws > 32 * 8192 * 4
    kv32, meta32, _, _ = rq.rq_sizes(cfg(dtype=rq.RQ_F32, head_dim=64, page_size=64, capacity_tokens=1000))
    assert kv32 == 32 * 16 * 2 * 64 * 64 * 4 and meta32 == 32 * 16 * 2 * 64 * 4


@pytest.mark.parametrize("kw,status", [
    (dict(batch=0), rq.RQ_ERR_INVALID_ARG), (dict(heads=-1), rq.RQ_ERR_INVALID_ARG),
    (dict(capacity_tokens=0), rq.RQ_ERR_INVALID_ARG), (dict(dtype=7), rq.RQ_ERR_INVALID_ARG),
    (dict(gate_dtype=-1), rq.RQ_ERR_INVALID_ARG), (dict(n_sink_pages=-1), rq.RQ_ERR_INVALID_ARG),
    (dict(max_budget_pages=0), rq.RQ_ERR_INVALID_ARG), (dict(reserved=1), rq.RQ_ERR_INVALID_ARG),
    (dict(head_dim=96), rq.RQ_ERR_UNSUPPORTED), (dict(page_size=32), rq.RQ_ERR_UNSUPPORTED),
    (dict(capacity_tokens=16 * 32768 + 1), rq.RQ_ERR_UNSUPPORTED),
])
def test_bad_configs_are_rejected(lib, kw, status):
    with pytest.raises(rq.RqError) as e:
        rq.rq_sizes(cfg(**kw))
    assert e.value.status == status


def test_null_and_misaligned_arguments_are_rejected_on_the_host(lib):
    c = cfg()
    cache = rq.rq_cache()
    f = lib.rq_cache_init
    assert lib.rq_sizes(None, None, None, None, None) == rq.RQ_ERR_INVALID_ARG
    assert f(None, C.byref(c), 256, 256, 256, 256, None) == rq.RQ_ERR_INVALID_ARG
    assert f(C.byref(cache), None, 256, 256, 256, 256, None) == rq.RQ_ERR_INVALID_ARG
    assert f(C.byref(cache), C.byref(c), None, 256, 256, 256, None) == rq.RQ_ERR_INVALID_ARG
    assert f(C.byref(cache), C.byref(c), 256, 256, 256, 264, None) == rq.RQ_ERR_INVALID_ARG   # misaligned
    # a handle that was never initialised is refused by every entry point
    empty = rq.rq_cache()
    assert lib.rq_cache_reset(C.byref(empty), None) == rq.RQ_ERR_INVALID_ARG
    assert lib.rq_build_cache(C.byref(empty), 256, 256, 256, 1, 0, 0, 0, None) == rq.RQ_ERR_INVALID_ARG
    assert lib.rq_decode_step(C.byref(empty), 256, 256, 256, 256, 1, 0.0, 256, None, None) == rq.RQ_ERR_INVALID_ARG
    assert lib.rq_decode_step_host(C.byref(empty), 256, 256, 256, 256, 1, 0.0, 256, None, None) == rq.RQ_ERR_INVALID_ARG
    assert lib.rq_select_pages(C.byref(empty), 256, 1, None, 256, None) == rq.RQ_ERR_INVALID_ARG
    assert lib.rq_attend_pages(C.byref(empty), 256, 256, 1, 0.0, 256, None) == rq.RQ_ERR_INVALID_ARG
    assert lib.rq_cache_len(None) == -1
    out = C.c_int32(0)
    assert lib.rq_device_status(C.byref(empty), C.byref(out), None) == rq.RQ_ERR_INVALID_ARG


def test_argument_checks_on_a_filled_in_handle(lib):
    """Fill the handle by hand (no device involved): the checks that come before any launch."""
    c = cfg(capacity_tokens=64, max_budget_pages=2)
    cache = rq.rq_cache()
    cache.cfg = c
    cache.kv = cache.meta = cache.state = cache.workspace = 4096
    cache.page_capacity = 4
    cache.len = 64
    assert lib.rq_build_cache(C.byref(cache), 256, 256, 256, -1, 0, 0, 0, None) == rq.RQ_ERR_INVALID_ARG
    assert lib.rq_build_cache(C.byref(cache), 256, 256, 256, 0, 0, 0, 0, None) == rq.RQ_OK       # no-op
    assert lib.rq_build_cache(C.byref(cache), None, 256, 256, 1, 0, 0, 0, None) == rq.RQ_ERR_INVALID_ARG
    assert lib.rq_build_cache(C.byref(cache), 256, 256, 264, 1, 0, 0, 0, None) == rq.RQ_ERR_INVALID_ARG
    assert lib.rq_build_cache(C.byref(cache), 256, 256, 256, 1, 4096, 4100, 128, None) == rq.RQ_ERR_INVALID_ARG
    assert lib.rq_build_cache(C.byref(cache), 256, 256, 256, 1, 4096, 4096, 128, None) == rq.RQ_ERR_CAPACITY
    assert lib.rq_decode_step(C.byref(cache), 256, 256, 256, 256, 0, 0.0, 256, None, None) == rq.RQ_ERR_INVALID_ARG
    assert lib.rq_decode_step(C.byref(cache), 256, 256, 256, 256, 3, 0.0, 256, None, None) == rq.RQ_ERR_CAPACITY
    assert lib.rq_decode_step(C.byref(cache), 256, 256, 256, 256, 2, 0.0, 256, None, None) == rq.RQ_ERR_CAPACITY
    assert lib.rq_decode_step_host(C.byref(cache), 256, 256, 256, 256, 2, 0.0, 256, None, None) == rq.RQ_ERR_CAPACITY
    assert lib.rq_select_pages(C.byref(cache), 256, 3, None, 256, None) == rq.RQ_ERR_CAPACITY
    assert lib.rq_select_pages(C.byref(cache), 256, 1, None, None, None) == rq.RQ_ERR_INVALID_ARG
    assert lib.rq_attend_pages(C.byref(cache), 256, 256, 3, 0.0, 256, None) == rq.RQ_ERR_CAPACITY
    assert lib.rq_attend_pages(C.byref(cache), 256, None, 1, 0.0, 256, None) == rq.RQ_ERR_INVALID_ARG
    assert lib.rq_cache_len(C.byref(cache)) == 64
    cache.len = 0
    assert lib.rq_select_pages(C.byref(cache), 256, 1, None, 256, None) == rq.RQ_ERR_INVALID_ARG   # empty cache


def test_argument_checks_of_the_widened_rows(lib):
    """SnapKV and MoBA entry points: everything that is decided on the host before a launch."""
    c = cfg(capacity_tokens=8192, max_budget_pages=8)
    cache = rq.rq_cache()
    cache.cfg = c
    cache.kv = cache.meta = cache.state = cache.workspace = 4096
    cache.page_capacity = 8192 // c.page_size
    cache.len = 5000
    n = C.c_size_t()
    BH = c.batch * c.heads
    # SnapKV scratch: importance [BH][len] fp32 + statistics per 128-key tile and final, each rounded to 256 bytes
    assert lib.rq_snapkv_scratch_bytes(C.byref(cache), C.byref(n)) == rq.RQ_OK
    tiles = -(-5000 // 128)
    r256 = lambda x: -(-x // 256) * 256
    assert n.value == r256(BH * 5000 * 4) + r256(BH * tiles * 64 * 8) + r256(BH * 64 * 8)
    assert lib.rq_snapkv_scratch_bytes(C.byref(cache), None) == rq.RQ_ERR_INVALID_ARG
    for window, keep in ((0, 16), (65, 16), (64, 0), (5001, 16)):
        assert lib.rq_snapkv_select(C.byref(cache), 256, window, keep, 0.0, 256, None, 256, None) == rq.RQ_ERR_INVALID_ARG
    assert lib.rq_snapkv_select(C.byref(cache), None, 64, 16, 0.0, 256, None, 256, None) == rq.RQ_ERR_INVALID_ARG
    assert lib.rq_snapkv_select(C.byref(cache), 256, 64, 16, 0.0, 256, None, 260, None) == rq.RQ_ERR_INVALID_ARG   # scratch alignment
    other = rq.rq_cache()
    other.cfg = cfg(capacity_tokens=64, max_budget_pages=2)
    other.kv = other.meta = other.state = other.workspace = 8192
    other.page_capacity = 4
    assert lib.rq_snapkv_compact(C.byref(cache), 256, 65, C.byref(other), None) == rq.RQ_ERR_CAPACITY
    assert lib.rq_snapkv_compact(C.byref(cache), 256, 0, C.byref(other), None) == rq.RQ_ERR_INVALID_ARG
    assert lib.rq_snapkv_compact(C.byref(cache), 256, 5001, C.byref(other), None) == rq.RQ_ERR_INVALID_ARG
    assert lib.rq_snapkv_compact(C.byref(cache), None, 16, C.byref(other), None) == rq.RQ_ERR_INVALID_ARG
    other.kv = 4096                                                   # the same buffer as the source
    assert lib.rq_snapkv_compact(C.byref(cache), 256, 16, C.byref(other), None) == rq.RQ_ERR_INVALID_ARG
    # MoBA scratch: representatives [BH][blocks][D] fp32 + chosen blocks [BH][len][K] int32
    assert lib.rq_moba_scratch_bytes(C.byref(cache), 64, 4, C.byref(n)) == rq.RQ_OK
    nb = -(-5000 // 64)
    assert n.value == r256(BH * nb * c.head_dim * 4) + r256(BH * 5000 * 4 * 4)
    for block, K in ((32, 4), (96, 4), (64, 1), (72, 4)):
        assert lib.rq_moba_scratch_bytes(C.byref(cache), block, K, C.byref(n)) == rq.RQ_ERR_INVALID_ARG
        assert lib.rq_moba_prefill(C.byref(cache), 256, block, K, 0.0, 256, None, None, 256, None) == rq.RQ_ERR_INVALID_ARG
    assert lib.rq_moba_prefill(C.byref(cache), None, 64, 4, 0.0, 256, None, None, 256, None) == rq.RQ_ERR_INVALID_ARG
    assert lib.rq_moba_prefill(C.byref(cache), 256, 64, 4, 0.0, 256, None, None, 260, None) == rq.RQ_ERR_INVALID_ARG
    cache.len = 0
    assert lib.rq_moba_scratch_bytes(C.byref(cache), 64, 4, C.byref(n)) == rq.RQ_ERR_INVALID_ARG


def _no_gpu():
    import torch
    return not torch.cuda.is_available()


@pytest.mark.skipif(not _no_gpu(), reason="drives the launch code with made-up pointers: only where no launch can succeed")
def test_failed_launch_leaves_length_and_step_count_unchanged(lib):
    """Without a device every CUDA call fails: the step must return RQ_ERR_CUDA and roll nothing forward."""
    c = cfg(capacity_tokens=1 << 16, max_budget_pages=64)
    cache = rq.rq_cache()
    cache.cfg = c
    cache.kv = cache.meta = cache.state = cache.workspace = 4096
    cache.page_capacity = (1 << 16) // 16
    cache.len = 20000
    cache.reserved[0] = 7
    for path in (0, 1, 2):
        cache.reserved[2] = path
        assert lib.rq_decode_step(C.byref(cache), 256, 256, 256, 256, 64, 0.0, 256, None, None) == rq.RQ_ERR_CUDA
        assert cache.len == 20000 and cache.reserved[0] == 7
    assert lib.rq_build_cache(C.byref(cache), 256, 256, 256, 16, 1 << 20, 4096, 128, None) == rq.RQ_ERR_CUDA
    assert cache.len == 20000
    assert lib.rq_decode_step_launches(C.byref(cache), 64) == 3       # no device: nothing to plan a single launch with
    assert lib.rq_decode_step_launches(None, 64) == -1


def test_workload_generators_are_seeded_and_shaped():
    import torch
    from paper_2605_28640_b200 import workloads as wl
    w = wl.Workload("t", B=2, H=3, D=64, T=100, seed=9, resets=True)
    k1, v1, g1 = wl.make_prefill(w, "cpu")
    k2, v2, g2 = wl.make_prefill(w, "cpu")
    assert torch.equal(k1, k2) and torch.equal(v1, v2) and torch.equal(g1, g2)
    assert k1.shape == (2, 100, 3, 64) and k1.dtype == torch.bfloat16
    assert 0.9 < g1.float().mean() < 0.995
    w2 = wl.Workload("n", B=1, H=2, D=64, T=160, seed=9, needles=3)
    pages = wl.needle_pages(w2)
    assert pages.shape == (1, 2, 3) and pages.min() >= 1 and pages.max() <= 8
    q = wl.make_query(w2, "cpu")
    kn, _, _ = wl.make_prefill(w2, "cpu", q_for_needles=q)
    k0, _, _ = wl.make_prefill(wl.Workload("n", B=1, H=2, D=64, T=160, seed=9), "cpu")
    diff = (kn.float() - k0.float()).abs().sum(-1)       # [B, T, H]
    for h in range(2):
        touched = sorted(set((diff[0, :, h].nonzero().flatten() // 16).tolist()))
        assert touched == sorted(pages[0, h].tolist())
    assert wl.CONFIGS[2].budget_pages(32769) == 257 and wl.CONFIGS[1].budget_pages() == 64
    assert wl.METRIC.budget_pages() == 512 and wl.CONFIGS[0].budget_pages() == 16
