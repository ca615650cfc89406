"""ctypes binding of ``librq.so`` (the C ABI declared in ``include/rq.h``).

The functions here have the ABI's names and do argument marshalling only:
every step of the path runs in the library's CUDA kernels.  PyTorch supplies
device memory and streams.  There is no CPU fallback: if the library cannot be
loaded, importing a compute entry point fails with the loader's error.
"""
from __future__ import annotations

import ctypes as C
import os

RQ_OK, RQ_ERR_INVALID_ARG, RQ_ERR_UNSUPPORTED, RQ_ERR_CAPACITY, RQ_ERR_CUDA, RQ_ERR_TIMEOUT = range(6)
RQ_F32, RQ_BF16 = 0, 1

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "librq.so")


class rq_config(C.Structure):
    _fields_ = [("batch", C.c_int32), ("heads", C.c_int32), ("head_dim", C.c_int32),
                ("page_size", C.c_int32), ("capacity_tokens", C.c_int64), ("dtype", C.c_int32),
                ("gate_dtype", C.c_int32), ("n_sink_pages", C.c_int32), ("n_local_pages", C.c_int32),
                ("max_budget_pages", C.c_int32), ("reserved", C.c_int32)]


class rq_cache(C.Structure):
    _fields_ = [("cfg", rq_config), ("kv", C.c_void_p), ("meta", C.c_void_p), ("state", C.c_void_p),
                ("workspace", C.c_void_p), ("len", C.c_int64), ("page_capacity", C.c_int64),
                ("reserved", C.c_int64 * 4)]


_vp, _i32, _i64, _f = C.c_void_p, C.c_int32, C.c_int64, C.c_float
_szp = C.POINTER(C.c_size_t)
_cfgp, _cachep = C.POINTER(rq_config), C.POINTER(rq_cache)

# name -> (restype, argtypes); one entry per function declared in rq.h
SIGNATURES = {
    "rq_sizes": (C.c_int, [_cfgp, _szp, _szp, _szp, _szp]),
    "rq_cache_init": (C.c_int, [_cachep, _cfgp, _vp, _vp, _vp, _vp, _vp]),
    "rq_cache_reset": (C.c_int, [_cachep, _vp]),
    "rq_build_cache": (C.c_int, [_cachep, _vp, _vp, _vp, _i64, _i64, _i64, _i64, _vp]),
    "rq_decode_step": (C.c_int, [_cachep, _vp, _vp, _vp, _vp, _i32, _f, _vp, _vp, _vp]),
    "rq_decode_step_host": (C.c_int, [_cachep, _vp, _vp, _vp, _vp, _i32, _f, _vp, _vp, _vp]),
    "rq_decode_step_profiled": (C.c_int, [_cachep, _vp, _vp, _vp, _vp, _i32, _f, _vp, _vp,
                                          C.POINTER(C.c_float), _vp]),
    "rq_profile_slot_name": (C.c_char_p, [C.c_int]),
    "rq_select_pages": (C.c_int, [_cachep, _vp, _i32, _vp, _vp, _vp]),
    "rq_attend_pages": (C.c_int, [_cachep, _vp, _vp, _i32, _f, _vp, _vp]),
    "rq_attend_pages_noalloc": (C.c_int, [_cfgp, _vp, _i64, _vp, _vp, _i32, _f, _vp, _vp]),
    "rq_probe_read": (C.c_int, [_vp, C.c_size_t, _vp, _vp]),
    "rq_snapkv_scratch_bytes": (C.c_int, [_cachep, _szp]),
    "rq_snapkv_select": (C.c_int, [_cachep, _vp, _i32, _i32, _f, _vp, _vp, _vp, _vp]),
    "rq_snapkv_compact": (C.c_int, [_cachep, _vp, _i32, _cachep, _vp]),
    "rq_moba_scratch_bytes": (C.c_int, [_cachep, _i32, _i32, _szp]),
    "rq_moba_prefill": (C.c_int, [_cachep, _vp, _i32, _i32, _f, _vp, _vp, _vp, _vp, _vp]),
    "rq_cache_len": (C.c_int64, [_cachep]),
    "rq_decode_step_launches": (C.c_int, [_cachep, _i32]),
    "rq_device_status": (C.c_int, [_cachep, C.POINTER(C.c_int32), _vp]),
    "rq_status_string": (C.c_char_p, [C.c_int]),
    "rq_version": (C.c_int, []),
}

_lib = None


def lib():
    """Load the shared library (once).  Raises OSError if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise OSError(f"{LIB_PATH} is missing: run paper_2605_28640_b200.build.build_library() "
                          "(there is no fallback path)")
        L = C.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(L, name)
            fn.restype, fn.argtypes = res, args
        _lib = L
    return _lib


class RqError(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        super().__init__(f"{where}: {lib().rq_status_string(status).decode()} (status {status})")


def _check(status, where):
    if status != RQ_OK:
        raise RqError(status, where)


def _ptr(t):
    """Device (or host) address of a torch tensor, or None."""
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream):
    import torch
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


# ---------------------------------------------------------------- ABI-named calls
def rq_sizes(cfg: rq_config):
    kv, meta, st, ws = C.c_size_t(), C.c_size_t(), C.c_size_t(), C.c_size_t()
    _check(lib().rq_sizes(C.byref(cfg), C.byref(kv), C.byref(meta), C.byref(st), C.byref(ws)), "rq_sizes")
    return kv.value, meta.value, st.value, ws.value


def rq_cache_init(cfg: rq_config, kv, meta, state, workspace, stream=None) -> rq_cache:
    cache = rq_cache()
    _check(lib().rq_cache_init(C.byref(cache), C.byref(cfg), _ptr(kv), _ptr(meta), _ptr(state),
                               _ptr(workspace), _stream(stream)), "rq_cache_init")
    return cache


def rq_cache_reset(cache: rq_cache, stream=None):
    _check(lib().rq_cache_reset(C.byref(cache), _stream(stream)), "rq_cache_reset")


def rq_build_cache(cache: rq_cache, k, v, g, stream=None):
    """k, v, g: torch tensors [B, T, H, D] (any strides with d contiguous; g uses k's strides)."""
    assert k.dim() == 4 and k.stride(3) == 1 and v.stride() == k.stride() and g.stride() == k.stride()
    _check(lib().rq_build_cache(C.byref(cache), _ptr(k), _ptr(v), _ptr(g), k.shape[1], k.stride(0),
                                k.stride(1), k.stride(2), _stream(stream)), "rq_build_cache")


def rq_decode_step(cache: rq_cache, q, k_t, v_t, g_t, budget_pages, scale, o, sel_idx_out=None, stream=None):
    _check(lib().rq_decode_step(C.byref(cache), _ptr(q), _ptr(k_t), _ptr(v_t), _ptr(g_t), budget_pages,
                                scale, _ptr(o), _ptr(sel_idx_out), _stream(stream)), "rq_decode_step")


def rq_decode_step_host(cache: rq_cache, q, k_t, v_t, g_t, budget_pages, scale, o, sel_idx_out=None,
                        stream=None):
    """Same as rq_decode_step with HOST tensors (pinned for asynchronous copies)."""
    _check(lib().rq_decode_step_host(C.byref(cache), _ptr(q), _ptr(k_t), _ptr(v_t), _ptr(g_t), budget_pages,
                                     scale, _ptr(o), _ptr(sel_idx_out), _stream(stream)),
           "rq_decode_step_host")


RQ_PROFILE_SLOTS = 3


def rq_decode_step_profiled(cache: rq_cache, q, k_t, v_t, g_t, budget_pages, scale, o, sel_idx_out=None,
                            stream=None):
    """rq_decode_step with per-kernel timing; synchronises; returns {kernel name: microseconds}."""
    us = (C.c_float * RQ_PROFILE_SLOTS)()
    _check(lib().rq_decode_step_profiled(C.byref(cache), _ptr(q), _ptr(k_t), _ptr(v_t), _ptr(g_t),
                                         budget_pages, scale, _ptr(o), _ptr(sel_idx_out), us,
                                         _stream(stream)), "rq_decode_step_profiled")
    return {lib().rq_profile_slot_name(i).decode(): us[i] for i in range(RQ_PROFILE_SLOTS)}


def rq_select_pages(cache: rq_cache, q, budget_pages, scores_out, idx_out, stream=None):
    _check(lib().rq_select_pages(C.byref(cache), _ptr(q), budget_pages, _ptr(scores_out), _ptr(idx_out),
                                 _stream(stream)), "rq_select_pages")


def rq_attend_pages(cache: rq_cache, q, idx, n_idx, scale, o, stream=None):
    _check(lib().rq_attend_pages(C.byref(cache), _ptr(q), _ptr(idx), n_idx, scale, _ptr(o),
                                 _stream(stream)), "rq_attend_pages")


def rq_attend_pages_noalloc(cfg: rq_config, kv, length, q, idx, n_idx, scale, o, stream=None):
    """rq_attend_pages without a workspace, for callers that may not allocate device memory: the
    kernel's scratch is a fixed array inside the library (shapes beyond its 4 MiB are refused)."""
    _check(lib().rq_attend_pages_noalloc(C.byref(cfg), _ptr(kv), length, _ptr(q), _ptr(idx), n_idx, scale,
                                         _ptr(o), _stream(stream)), "rq_attend_pages_noalloc")


def rq_probe_read(buf, nbytes, sink, stream=None):
    """One launch that reads nbytes of the device tensor `buf` once (benchmarking aid)."""
    _check(lib().rq_probe_read(_ptr(buf), nbytes, _ptr(sink), _stream(stream)), "rq_probe_read")


def rq_snapkv_scratch_bytes(cache: rq_cache) -> int:
    n = C.c_size_t()
    _check(lib().rq_snapkv_scratch_bytes(C.byref(cache), C.byref(n)), "rq_snapkv_scratch_bytes")
    return n.value


def rq_snapkv_select(cache: rq_cache, q_window, window, keep, scale, idx_out, importance_out, scratch, stream=None):
    _check(lib().rq_snapkv_select(C.byref(cache), _ptr(q_window), window, keep, scale, _ptr(idx_out),
                                  _ptr(importance_out), _ptr(scratch), _stream(stream)), "rq_snapkv_select")


def rq_snapkv_compact(src: rq_cache, idx, keep, dst: rq_cache, stream=None):
    _check(lib().rq_snapkv_compact(C.byref(src), _ptr(idx), keep, C.byref(dst), _stream(stream)), "rq_snapkv_compact")


def rq_moba_scratch_bytes(cache: rq_cache, block, budget_blocks) -> int:
    n = C.c_size_t()
    _check(lib().rq_moba_scratch_bytes(C.byref(cache), block, budget_blocks, C.byref(n)), "rq_moba_scratch_bytes")
    return n.value


def rq_moba_prefill(cache: rq_cache, q, block, budget_blocks, scale, o, blocks_out, means_out, scratch, stream=None):
    _check(lib().rq_moba_prefill(C.byref(cache), _ptr(q), block, budget_blocks, scale, _ptr(o), _ptr(blocks_out),
                                 _ptr(means_out), _ptr(scratch), _stream(stream)), "rq_moba_prefill")


def rq_cache_len(cache: rq_cache) -> int:
    return lib().rq_cache_len(C.byref(cache))


def rq_decode_step_launches(cache: rq_cache, budget_pages: int) -> int:
    return lib().rq_decode_step_launches(C.byref(cache), budget_pages)


def rq_device_status(cache: rq_cache, stream=None) -> int:
    out = C.c_int32(0)
    _check(lib().rq_device_status(C.byref(cache), C.byref(out), _stream(stream)), "rq_device_status")
    return out.value


def rq_status_string(status: int) -> str:
    return lib().rq_status_string(status).decode()


def rq_version() -> int:
    return lib().rq_version()


# ---------------------------------------------------------------- allocation helper
class Cache:
    """Allocates the four device buffers with torch and adopts them with rq_cache_init.
    Holds the tensors so that they outlive the handle."""

    def __init__(self, batch, heads, head_dim, page_size, capacity_tokens, dtype, gate_dtype=None,
                 n_sink_pages=1, n_local_pages=1, max_budget_pages=None, device="cuda", stream=None):
        import torch
        self.torch_dtype = dtype
        rq_dt = {torch.float32: RQ_F32, torch.bfloat16: RQ_BF16}
        gate_dtype = gate_dtype or dtype
        pc = (capacity_tokens + page_size - 1) // page_size
        self.cfg = rq_config(batch, heads, head_dim, page_size, capacity_tokens, rq_dt[dtype],
                             rq_dt[gate_dtype], n_sink_pages, n_local_pages,
                             max_budget_pages or pc, 0)
        kvb, mb, sb, wb = rq_sizes(self.cfg)
        self.kv = torch.empty(kvb, dtype=torch.uint8, device=device)
        self.meta = torch.empty(mb, dtype=torch.uint8, device=device)
        self.state = torch.empty(sb, dtype=torch.uint8, device=device)
        self.workspace = torch.empty(wb, dtype=torch.uint8, device=device)
        self.page_capacity = pc
        self.handle = rq_cache_init(self.cfg, self.kv, self.meta, self.state, self.workspace, stream)

    def __len__(self):
        return rq_cache_len(self.handle)

    # typed views of the caller-owned buffers (layouts of rq.h)
    def kv_view(self):
        c = self.cfg
        return self.kv.view(self.torch_dtype).view(c.batch, c.heads, self.page_capacity, 2, c.page_size, c.head_dim)

    def meta_view(self):
        c = self.cfg
        return self.meta.view(self.torch_dtype).view(c.batch, c.heads, self.page_capacity, 2, c.head_dim)

    def state_view(self):
        import torch
        c = self.cfg
        return self.state.view(torch.float32).view(c.batch, c.heads, 2, c.head_dim)
