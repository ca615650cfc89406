"""ctypes front end of the fp64 CPU oracle in ``rqo.c``.

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, by the smoke check and by the
benchmark's CPU-baseline leg.  The CUDA library and its Python binding never
import this package, and this package never imports them.

Every wrapper works on one (batch, head) pair with float64 numpy arrays.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

F32 = 0
BF16 = 1

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "rqo.c")
_LIB = os.path.join(_HERE, "librqo.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile ``rqo.c`` into ``librqo.so`` next to it (gcc, -O2, strict IEEE)."""
    srcs = [_SRC, os.path.join(_HERE, "rqo_snapkv.c"), os.path.join(_HERE, "rqo_moba.c")]
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < max(os.path.getmtime(f) for f in srcs):
        cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-ffp-contract=off",
               "-fno-fast-math", "-o", _LIB, *srcs, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


_dp = C.POINTER(C.c_double)
_ip = C.POINTER(C.c_int64)


def _d(a):
    return None if a is None else a.ctypes.data_as(_dp)


def _f64(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.float64)


def lib():
    global _lib
    if _lib is None:
        build()
        L = C.CDLL(_LIB)
        L.rqo_recurrence.argtypes = [C.c_int64, C.c_int, _dp, _dp, _dp, _dp, _dp, _dp, _dp]
        L.rqo_recurrence.restype = None
        L.rqo_round_bf16.argtypes = [C.c_double]
        L.rqo_round_bf16.restype = C.c_double
        L.rqo_round_f32.argtypes = [C.c_double]
        L.rqo_round_f32.restype = C.c_double
        L.rqo_round_storage.argtypes = [C.c_int64, _dp, C.c_int, _dp]
        L.rqo_round_storage.restype = None
        L.rqo_page_bounds.argtypes = [C.c_int64, C.c_int, C.c_int, _dp, _dp, _dp]
        L.rqo_page_bounds.restype = None
        L.rqo_page_scores.argtypes = [C.c_int64, C.c_int, _dp, _dp, _dp, _dp]
        L.rqo_page_scores.restype = None
        L.rqo_select_pages.argtypes = [C.c_int64, _dp, C.c_int64, C.c_int64, C.c_int64, _ip,
                                       C.POINTER(C.c_int)]
        L.rqo_select_pages.restype = C.c_int64
        L.rqo_sparse_attention.argtypes = [C.c_int64, C.c_int, C.c_int, _dp, C.c_double, _dp, _dp,
                                           _ip, C.c_int64, _dp]
        L.rqo_sparse_attention.restype = None
        L.rqo_head_new.argtypes = [C.c_int, C.c_int, C.c_int64, C.c_int, C.c_int64, C.c_int64]
        L.rqo_head_new.restype = C.c_void_p
        L.rqo_head_free.argtypes = [C.c_void_p]
        L.rqo_head_free.restype = None
        L.rqo_head_len.argtypes = [C.c_void_p]
        L.rqo_head_len.restype = C.c_int64
        L.rqo_head_append.argtypes = [C.c_void_p, C.c_int64, _dp, _dp, _dp]
        L.rqo_head_append.restype = C.c_int
        L.rqo_head_query.argtypes = [C.c_void_p, _dp, C.c_int64, C.c_double, _dp, _ip, _ip, _dp,
                                     C.POINTER(C.c_int)]
        L.rqo_head_query.restype = None
        L.rqo_head_export.argtypes = [C.c_void_p, _dp, _dp, _dp, _dp, _dp, _dp]
        L.rqo_head_export.restype = None
        L.rqo_head_load.argtypes = [C.c_void_p, C.c_int64, _dp, _dp, _dp, _dp]
        L.rqo_head_load.restype = C.c_int
        L.rqo_snapkv_importance.argtypes = [C.c_int64, C.c_int, C.c_int, _dp, C.c_double, _dp, _dp]
        L.rqo_snapkv_importance.restype = None
        L.rqo_snapkv_select.argtypes = [C.c_int64, C.c_int, _dp, C.c_int64, _ip, C.POINTER(C.c_int)]
        L.rqo_snapkv_select.restype = C.c_int64
        L.rqo_token_attention.argtypes = [C.c_int64, _ip, C.c_int, _dp, C.c_double, _dp, _dp, _dp]
        L.rqo_token_attention.restype = None
        L.rqo_block_means.argtypes = [C.c_int64, C.c_int, C.c_int64, _dp, _dp]
        L.rqo_block_means.restype = None
        L.rqo_moba_scores.argtypes = [C.c_int64, C.c_int, _dp, _dp, _dp]
        L.rqo_moba_scores.restype = None
        _lib = L
    return _lib


# ---------------------------------------------------------------- stage calls
def recurrence(k, v, g, k_init=None, v_init=None):
    """Eq. 1 over [T, D] inputs; returns all states (k~, v~) as [T, D] float64."""
    k, v, g = _f64(k), _f64(v), _f64(g)
    T, D = k.shape
    kt = np.empty((T, D), np.float64)
    vt = np.empty((T, D), np.float64)
    ki, vi = _f64(k_init), _f64(v_init)
    lib().rqo_recurrence(T, D, _d(k), _d(v), _d(g), _d(ki), _d(vi), _d(kt), _d(vt))
    return kt, vt


def round_storage(x, dtype):
    """Value the cache holds for state x (bf16 or fp32, round-to-nearest-even)."""
    x = _f64(x)
    out = np.empty_like(x)
    lib().rqo_round_storage(x.size, _d(x), dtype, _d(out))
    return out


def page_bounds(kst, S):
    """Per page, per channel min and max of stored keys [T, D] -> ([P, D], [P, D])."""
    kst = _f64(kst)
    T, D = kst.shape
    P = (T + S - 1) // S
    mn = np.empty((P, D), np.float64)
    mx = np.empty((P, D), np.float64)
    lib().rqo_page_bounds(T, D, S, _d(kst), _d(mn), _d(mx))
    return mn, mx


def page_scores(q, mn, mx):
    """U_p = sum_i max(q_i*min_p[i], q_i*max_p[i]) for every page -> [P]."""
    q, mn, mx = _f64(q), _f64(mn), _f64(mx)
    P, D = mn.shape
    U = np.empty(P, np.float64)
    lib().rqo_page_scores(P, D, _d(q), _d(mn), _d(mx), _d(U))
    return U


def select_pages(U, K, n_sink=1, n_local=1):
    """Top-K pages with forced first/local pages; returns (ascending idx, near_tie)."""
    U = _f64(U)
    P = U.shape[0]
    idx = np.empty(max(min(K, P), 1), np.int64)
    nt = C.c_int(0)
    n = lib().rqo_select_pages(P, _d(U), K, n_sink, n_local, idx.ctypes.data_as(_ip), C.byref(nt))
    return idx[:n].copy(), bool(nt.value)


def sparse_attention(q, scale, kst, vst, idx, S):
    """Eq. 4: softmax attention over the valid tokens of the pages in idx -> [D]."""
    q, kst, vst = _f64(q), _f64(kst), _f64(vst)
    T, D = kst.shape
    idx = np.ascontiguousarray(idx, dtype=np.int64)
    y = np.empty(D, np.float64)
    lib().rqo_sparse_attention(T, D, S, _d(q), float(scale), _d(kst), _d(vst),
                               idx.ctypes.data_as(_ip), idx.shape[0], _d(y))
    return y


# ---------------------------------------------------------------- head object
def snapkv_importance(qw, scale, kst):
    """App. A.1 (SnapKV): importance of every position under the window's queries.  qw [W, D], kst [T, D]."""
    qw, kst = _f64(qw), _f64(kst)
    W, D = qw.shape
    T = kst.shape[0]
    imp = np.empty(T, np.float64)
    lib().rqo_snapkv_importance(T, W, D, _d(qw), float(scale), _d(kst), _d(imp))
    return imp


def snapkv_select(imp, W, keep):
    """Retained positions (ascending) and the near-tie flag."""
    imp = _f64(imp)
    T = imp.shape[0]
    idx = np.empty(max(min(keep, T), 1), np.int64)
    near = C.c_int(0)
    n = lib().rqo_snapkv_select(T, W, _d(imp), keep, idx.ctypes.data_as(_ip), C.byref(near))
    return idx[:n].copy(), bool(near.value)


def token_attention(q, scale, kst, vst, tok):
    """Eq. 4 over an explicit token list."""
    q, kst, vst = _f64(q), _f64(kst), _f64(vst)
    tok = np.ascontiguousarray(tok, dtype=np.int64)
    y = np.empty(q.shape[0], np.float64)
    lib().rqo_token_attention(len(tok), tok.ctypes.data_as(_ip), q.shape[0], _d(q), float(scale), _d(kst), _d(vst), _d(y))
    return y


def block_means(kst, block):
    """App. A.1 (MoBA): mean-pooled representative of every block of `block` positions.  kst [T, D]."""
    kst = _f64(kst)
    T, D = kst.shape
    means = np.empty(((T + block - 1) // block, D), np.float64)
    lib().rqo_block_means(T, D, block, _d(kst), _d(means))
    return means


def moba_scores(q, means, n):
    """Eq. 3's score of the first n blocks under query q: q . mean."""
    q, means = _f64(q), _f64(means)
    U = np.empty(n, np.float64)
    lib().rqo_moba_scores(n, q.shape[0], _d(q), _d(means), _d(U))
    return U


def moba_route(q, means, t, block, K, n_sink=1, n_local=1):
    """Blocks the query of position t attends (ascending) and the near-tie flag: the TopK of Eq. 3 over the
    complete blocks before the query's own, the first block(s) and the own block always included, all inside K."""
    bt = t // block
    U = np.zeros(bt + 1)
    if bt > 0:
        U[:bt] = moba_scores(q, means, bt)
    # the own block is the newest `page`: forced whatever its score (n_local >= 1), ranked last otherwise
    U[bt] = -np.inf if n_local < 1 else 0.0
    return select_pages(U, K, n_sink, n_local)


def moba_attention(q, scale, kst, vst, blocks, t, block):
    """Eq. 4 for the query of position t over the listed blocks: their tokens up to position t."""
    tok = np.concatenate([np.arange(j * block, min((j + 1) * block, t + 1)) for j in blocks]) if len(blocks) else np.zeros(0, np.int64)
    return token_attention(q, scale, kst, vst, tok)


class Head:
    """fp64 cache of one (batch, head) pair: prefill = append(T tokens),
    decode step = append(1 token) then query."""

    def __init__(self, D, S, capacity, dtype, n_sink=1, n_local=1):
        self.D, self.S, self.cap, self.dtype = D, S, capacity, dtype
        self._h = lib().rqo_head_new(D, S, capacity, dtype, n_sink, n_local)

    def __del__(self):
        if getattr(self, "_h", None):
            lib().rqo_head_free(self._h)
            self._h = None

    def __len__(self):
        return lib().rqo_head_len(self._h)

    def append(self, k, v, g):
        k, v, g = _f64(k).reshape(-1, self.D), _f64(v).reshape(-1, self.D), _f64(g).reshape(-1, self.D)
        rc = lib().rqo_head_append(self._h, k.shape[0], _d(k), _d(v), _d(g))
        if rc != 0:
            raise ValueError("oracle cache capacity exceeded")

    def query(self, q, K, scale, want_scores=False):
        q = _f64(q)
        P = (len(self) + self.S - 1) // self.S
        idx = np.empty(max(min(K, P), 1), np.int64)
        n = C.c_int64(0)
        nt = C.c_int(0)
        y = np.empty(self.D, np.float64)
        U = np.empty(max(P, 1), np.float64) if want_scores else None
        lib().rqo_head_query(self._h, _d(q), K, float(scale), _d(y), idx.ctypes.data_as(_ip),
                             C.byref(n), _d(U), C.byref(nt))
        out = {"y": y, "idx": idx[: n.value].copy(), "near_tie": bool(nt.value)}
        if want_scores:
            out["U"] = U[:P]
        return out

    def export(self):
        T = len(self)
        P = (T + self.S - 1) // self.S
        D = self.D
        sk, sv = np.empty(D), np.empty(D)
        kst, vst = np.empty((T, D)), np.empty((T, D))
        mn, mx = np.empty((P, D)), np.empty((P, D))
        lib().rqo_head_export(self._h, _d(sk), _d(sv), _d(kst), _d(vst), _d(mn), _d(mx))
        return {"state_k": sk, "state_v": sv, "k": kst, "v": vst, "min": mn, "max": mx}

    def load(self, kst, vst, state_k=None, state_v=None):
        kst, vst = _f64(kst), _f64(vst)
        sk, sv = _f64(state_k), _f64(state_v)
        if lib().rqo_head_load(self._h, kst.shape[0], _d(kst), _d(vst), _d(sk), _d(sv)) != 0:
            raise ValueError("oracle cache capacity exceeded")
