"""GPU parity of the selection (the TopK of Eq. 3) on score vectors built to reach every branch of
the selection kernels: the direct ranking of the threshold bucket, the radix passes on the key bits
that finish a bucket holding more than 1024 keys (long runs of identical scores, with the cut inside
a run and at the end of a run), the radix passes taken when the score range is too narrow for a
float bucket width, heads whose keys live in registers and heads whose keys live in shared memory.

Scores are planted through the page bounds: with q = e_0 and min_p[0] = max_p[0] = u_p (all other
channels zero) the bound of Eq. 3 is exactly u_p, on the device and in the oracle alike, so the
oracle's selection on the device's bounds must be reproduced index for index (equal scores go to the
lower page)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2605_28640_b200 as rq

import parity

pytestmark = pytest.mark.gpu
DEV = "cuda"


def planted_cache(U, H=1, n_sink=1, n_local=1, D=64, S=16):
    """A cache of H heads whose page p has score U[h][p] for q = e_0 (fp32 storage)."""
    U = np.asarray(U, dtype=np.float32)
    if U.ndim == 1:
        U = np.broadcast_to(U, (H, U.shape[0]))
    P = U.shape[1]
    T = P * S
    c = rq.Cache(1, H, D, S, T, torch.float32, n_sink_pages=n_sink, n_local_pages=n_local, max_budget_pages=P)
    z = torch.zeros(1, T, H, D, dtype=torch.float32, device=DEV)
    rq.rq_build_cache(c.handle, z, z, z)
    torch.cuda.synchronize()
    meta = c.meta_view()
    assert not meta[0, :, :P].any()
    u = torch.from_numpy(np.ascontiguousarray(U)).to(DEV)
    meta[0, :, :P, 0, 0] = u
    meta[0, :, :P, 1, 0] = u
    q = torch.zeros(1, H, D, dtype=torch.float32, device=DEV)
    q[:, :, 0] = 1.0
    return c, q, U


def check_selection(c, q, U, K, n_sink, n_local):
    H, P = U.shape
    idx = torch.full((1, H, K), -7, dtype=torch.int32, device=DEV)
    sc = torch.empty(1, H, P, dtype=torch.float32, device=DEV)
    rq.rq_select_pages(c.handle, q, K, sc, idx)
    torch.cuda.synchronize()
    assert rq.rq_device_status(c.handle) == rq.RQ_OK
    for h in range(H):
        got_scores = sc[0, h].cpu().numpy()
        # the planted score is reproduced bit for bit (-0 and +0 count as equal)
        assert np.array_equal(got_scores, U[h]), "planted scores are not reproduced"
        dev = parity.device_head_arrays(c, 0, h)
        Uo = oracle.page_scores(parity.f64(q[0, h]), dev["min"], dev["max"])
        assert np.array_equal(Uo, U[h].astype(np.float64))
        want, _ = oracle.select_pages(Uo, K, n_sink, n_local)
        got = idx[0, h].cpu().numpy().astype(np.int64)
        assert np.array_equal(got[:len(want)], want), f"head {h}, K {K}: pages differ from the oracle's"
        assert (got[len(want):] == -1).all()


def plateau_scores(P, levels, seed, spread=1.0):
    """P scores drawn from a handful of distinct values: thousands of pages share each value."""
    rng = np.random.default_rng(seed)
    vals = (spread * rng.standard_normal(levels)).astype(np.float32)
    return vals[rng.integers(0, levels, P)]


@pytest.mark.parametrize("P,levels", [(8192, 3), (8192, 5), (5000, 2), (10240, 4), (2100, 2)])
@pytest.mark.parametrize("forced", [(0, 0), (1, 1), (2, 3)])
def test_long_runs_of_equal_scores_register_keys(P, levels, forced):
    """A few distinct scores over thousands of pages: the threshold bucket holds more than 1024 keys
    and the cut falls inside a run of equal scores; exactly the lowest pages of the run are taken."""
    n_sink, n_local = forced
    U = plateau_scores(P, levels, seed=P + levels)
    c, q, U = planted_cache(U, 1, n_sink, n_local)
    counts = sorted(np.unique(U[0], return_counts=True)[1])
    assert counts[-1] > 1024
    for K in (1, 7, P // 16, P // 4 + 3, P // 2, P - 5):
        check_selection(c, q, U, K, n_sink, n_local)


def test_two_runs_in_one_bucket_cut_at_the_end_of_the_lower_run():
    """Two runs of 700 equal scores each inside one value bucket and a slightly lower score in the
    bucket below, budget ending exactly with the lower run.  The radix passes end early (the whole
    bin is wanted) with a threshold whose low bits are cleared, which lies BELOW the lower run and
    below the bucket's edge; the score between that value and the run must not be taken."""
    ulp = np.float32(2.0 ** -14)                     # spacing of fp32 in [512, 1024)
    v_lo = np.float32(0.125) + 2 * ulp               # smallest score; buckets are [v_lo + j, v_lo + j + 1)
    v_hi = v_lo + np.float32(2047.0)
    assert np.float32(v_hi - v_lo) == np.float32(2047.0)
    lower = np.float32(600.125) + 3 * ulp            # bucket 600; low key bits 011
    upper = lower + np.float32(0.5)                  # bucket 600 as well
    below = np.float32(600.125) + 1 * ulp            # bucket 599, above `lower` with its low 3 bits cleared
    assert int(np.float32(lower - v_lo)) == 600 and int(np.float32(upper - v_lo)) == 600
    assert int(np.float32(below - v_lo)) == 599
    rng = np.random.default_rng(5)
    P = 8192
    U = np.empty(P, dtype=np.float32)
    U[:] = rng.uniform(1.0, 500.0, P).astype(np.float32)      # filler well below
    above = rng.choice(P, 100, replace=False)
    U[above] = rng.uniform(700.0, 2000.0, 100).astype(np.float32)
    rest = np.setdiff1d(np.arange(P), above)
    rng.shuffle(rest)
    U[rest[:700]] = lower
    U[rest[700:1400]] = upper
    U[rest[1400:1440]] = below
    U[rest[1440]] = v_lo
    U[rest[1441]] = v_hi
    c, q, U2 = planted_cache(U, 1, 0, 0)
    n_above = int((U > upper).sum())
    for K in (n_above + 1400, n_above + 1399, n_above + 1401, n_above + 700, n_above + 701, n_above + 1420):
        check_selection(c, q, U2, K, 0, 0)


@pytest.mark.parametrize("P", [300, 8192, 20000])
def test_score_range_too_narrow_for_a_bucket_width(P):
    """Scores a few denormal steps apart: the bucket width underflows, the selection goes straight to
    the radix passes on the key bits."""
    rng = np.random.default_rng(P)
    tiny = np.float32(1.4e-45)                       # smallest positive fp32
    U = (rng.integers(0, 40, P).astype(np.float32) * tiny).astype(np.float32)
    U[rng.integers(0, P, P // 3)] *= np.float32(-1.0)
    assert 0 < float(U.max()) - float(U.min()) < 1e-40
    c, q, U = planted_cache(U, 1, 1, 1)
    for K in (3, P // 10, P // 2):
        check_selection(c, q, U, K, 1, 1)


@pytest.mark.parametrize("P", [16384 + 100, 32768])
def test_long_runs_of_equal_scores_shared_memory_keys(P):
    """Heads of more than 10240 pages keep their keys in shared memory; same cases."""
    U = plateau_scores(P, 4, seed=P)
    c, q, U = planted_cache(U, 1, 1, 2)
    for K in (5, P // 16, P // 3):
        check_selection(c, q, U, K, 1, 2)
    # and distinct scores with a few duplicates
    rng = np.random.default_rng(P + 1)
    V = rng.standard_normal(P).astype(np.float32)
    V[rng.integers(0, P, 2000)] = V[17]
    c, q, V = planted_cache(V, 1, 1, 2)
    for K in (P // 16, P // 2 + 1):
        check_selection(c, q, V, K, 1, 2)


def test_mid_sized_heads_with_shared_memory_keys():
    """10241 .. 16384 pages: the 16-row shared-memory variant."""
    P = 12000
    rng = np.random.default_rng(3)
    U = rng.standard_normal(P).astype(np.float32)
    U[rng.integers(0, P, 3000)] = np.float32(0.25)
    c, q, U = planted_cache(U, 1, 1, 1)
    for K in (1, 2, 750, 4000, 9000):
        check_selection(c, q, U, K, 1, 1)


def test_short_context_kernel_on_planted_scores():
    """At most 256 pages per head and at least 16 heads: scoring and selection share one launch."""
    H, P = 16, 256
    rng = np.random.default_rng(9)
    U = np.stack([plateau_scores(P, 2 + h % 3, seed=100 + h) for h in range(H)])
    U[3] = (rng.integers(0, 9, P).astype(np.float32) * np.float32(1.4e-45))      # degenerate range
    U[4] = np.float32(1.5)                                                       # all equal
    c, q, U = planted_cache(U, H, 1, 1)
    for K in (2, 16, 100, 255):
        check_selection(c, q, U, K, 1, 1)
