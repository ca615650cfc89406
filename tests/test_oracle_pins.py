"""Pins for the fp64 oracle: each stage is checked against something other than
itself — closed forms, brute force, textbook routines, invariants — chosen so
that a dropped term, a wrong sign or index, or a transposed operand fails.
CPU only."""
import os

import numpy as np
import pytest
import torch

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rng(seed):
    return np.random.default_rng(seed)


# ------------------------------------------------------------------ Eq. 1
def test_recurrence_closed_form():
    """x~_t = sum_s (1-g_s) prod_{r>s} g_r x_s with zero initial state."""
    r = rng(0)
    T, D = 37, 5
    k, v = r.normal(size=(T, D)), r.normal(size=(T, D))
    g = r.uniform(0.05, 0.999, size=(T, D))
    kt, vt = oracle.recurrence(k, v, g)
    for x, xt in ((k, kt), (v, vt)):
        for t in range(T):
            for i in range(D):
                acc = 0.0
                for s in range(t + 1):
                    w = 1.0 - g[s, i]
                    for rr in range(s + 1, t + 1):
                        w *= g[rr, i]
                    acc += w * x[s, i]
                assert abs(xt[t, i] - acc) <= 1e-13 * max(1.0, abs(acc))


def test_recurrence_constant_inputs():
    """Constant gate and input: x~_t = x (1 - g^t)."""
    T, D = 50, 3
    gv = np.array([0.9, 0.5, 0.984])
    xv = np.array([2.0, -3.0, 0.25])
    yv = np.array([-1.0, 4.0, 8.0])
    k = np.tile(xv, (T, 1))
    v = np.tile(yv, (T, 1))
    g = np.tile(gv, (T, 1))
    kt, vt = oracle.recurrence(k, v, g)
    t = np.arange(1, T + 1)[:, None]
    np.testing.assert_allclose(kt, xv * (1 - gv ** t), rtol=1e-12)
    np.testing.assert_allclose(vt, yv * (1 - gv ** t), rtol=1e-12)


def test_recurrence_gate_extremes_and_convexity():
    r = rng(1)
    T, D = 40, 4
    k, v = r.normal(size=(T, D)), r.normal(size=(T, D))
    kt, vt = oracle.recurrence(k, v, np.zeros((T, D)))      # g = 0: no memory (Eq. 2 baseline)
    assert np.array_equal(kt, k) and np.array_equal(vt, v)
    kt, vt = oracle.recurrence(k, v, np.ones((T, D)))       # g = 1: nothing is ever written
    assert not kt.any() and not vt.any()
    g = r.uniform(0, 1, size=(T, D))
    kt, vt = oracle.recurrence(k, v, g)
    for x, xt in ((k, kt), (v, vt)):
        lo = np.minimum(0, np.minimum.accumulate(x, axis=0))
        hi = np.maximum(0, np.maximum.accumulate(x, axis=0))
        assert (xt >= lo - 1e-15).all() and (xt <= hi + 1e-15).all()


def test_recurrence_restart_and_initial_state():
    """scan(T1) then continue(T2) from the final state equals scan(T1+T2);
    a non-zero initial state decays as prod g."""
    r = rng(2)
    T1, T2, D = 19, 23, 6
    k, v = r.normal(size=(T1 + T2, D)), r.normal(size=(T1 + T2, D))
    g = r.uniform(0.5, 1, size=(T1 + T2, D))
    ka, va = oracle.recurrence(k, v, g)
    k1, v1 = oracle.recurrence(k[:T1], v[:T1], g[:T1])
    k2, v2 = oracle.recurrence(k[T1:], v[T1:], g[T1:], k1[-1], v1[-1])
    np.testing.assert_allclose(np.vstack([k1, k2]), ka, rtol=0, atol=1e-15)
    np.testing.assert_allclose(np.vstack([v1, v2]), va, rtol=0, atol=1e-15)
    z = np.zeros((T2, D))
    kz, vz = oracle.recurrence(z, z, g[:T2], np.ones(D), 2 * np.ones(D))
    np.testing.assert_allclose(kz, np.cumprod(g[:T2], axis=0), rtol=1e-13)
    np.testing.assert_allclose(vz, 2 * np.cumprod(g[:T2], axis=0), rtol=1e-13)


def test_recurrence_k_and_v_do_not_mix():
    """A change of v alone must leave k~ alone and vice versa; channels are independent."""
    r = rng(3)
    T, D = 12, 4
    k, v, g = r.normal(size=(T, D)), r.normal(size=(T, D)), r.uniform(0, 1, size=(T, D))
    kt, vt = oracle.recurrence(k, v, g)
    v2 = v.copy()
    v2[3, 1] += 1.0
    kt2, vt2 = oracle.recurrence(k, v2, g)
    assert np.array_equal(kt, kt2)
    diff = vt2 - vt
    assert (diff[:3] == 0).all() and (np.delete(diff, 1, axis=1) == 0).all() and diff[3, 1] != 0


# ------------------------------------------------------------------ storage rounding
def _bf16_rne_bits(x64):
    """Independent bf16 rounding on the IEEE-754 bit pattern of a double
    (valid where the result is a normal bf16 number)."""
    b = np.asarray(x64, np.float64).view(np.uint64).astype(object)
    out = []
    for bits in b.ravel():
        bits = int(bits)
        rem = bits & ((1 << 45) - 1)
        trunc = bits - rem
        half = 1 << 44
        if rem > half or (rem == half and (trunc >> 45) & 1):
            trunc += 1 << 45
        out.append(trunc)
    return np.array(out, dtype=np.uint64).view(np.float64).reshape(np.shape(x64))


def test_round_bf16_against_bit_manipulation():
    r = rng(4)
    x = np.concatenate([r.normal(size=4000), r.normal(size=2000) * 1e-3, r.normal(size=2000) * 1e4,
                        np.float64(np.float32(r.normal(size=2000)))])
    got = oracle.round_storage(x, oracle.BF16)
    assert np.array_equal(got, _bf16_rne_bits(x))
    # results are bf16 numbers: the low 16 bits of their fp32 pattern are zero
    assert (np.float32(got).view(np.uint32) & 0xFFFF == 0).all()
    assert np.array_equal(np.float64(np.float32(got)), got)


def test_round_bf16_ties_to_even_and_edges():
    # 1 + 2^-8 is exactly between 1 and 1 + 2^-7: ties to even -> 1
    assert oracle.round_storage([1 + 2.0 ** -8], oracle.BF16)[0] == 1.0
    # 1 + 3*2^-8 is between 1+2^-7 (odd) and 1+2^-6 (even) -> 1 + 2^-6
    assert oracle.round_storage([1 + 3 * 2.0 ** -8], oracle.BF16)[0] == 1 + 2.0 ** -6
    # just above / below the tie
    assert oracle.round_storage([1 + 2.0 ** -8 + 2.0 ** -40], oracle.BF16)[0] == 1 + 2.0 ** -7
    assert oracle.round_storage([1 + 3 * 2.0 ** -8 - 2.0 ** -40], oracle.BF16)[0] == 1 + 2.0 ** -7
    # mantissa carry into the exponent
    assert oracle.round_storage([2 - 2.0 ** -9], oracle.BF16)[0] == 2.0
    # sign symmetry, zero, all bf16 values are fixed points
    allbf = (np.arange(0x0080, 0x7F80, dtype=np.uint32) << 16).view(np.float32).astype(np.float64)
    assert np.array_equal(oracle.round_storage(allbf, oracle.BF16), allbf)
    assert np.array_equal(oracle.round_storage(-allbf, oracle.BF16), -allbf)
    assert oracle.round_storage([0.0], oracle.BF16)[0] == 0.0
    # torch's fp32 -> bf16 conversion agrees on fp32 inputs
    x32 = torch.randn(20000, generator=torch.Generator().manual_seed(0))
    want = x32.to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(oracle.round_storage(x32.to(torch.float64).numpy(), oracle.BF16), want)


def test_round_f32_matches_ieee_cast():
    r = rng(5)
    x = np.concatenate([r.normal(size=5000), r.normal(size=1000) * 1e-30, r.normal(size=1000) * 1e30])
    assert np.array_equal(oracle.round_storage(x, oracle.F32), np.float64(np.float32(x)))


# ------------------------------------------------------------------ page bounds
@pytest.mark.parametrize("T,S", [(64, 16), (70, 16), (5, 16), (1, 16), (130, 64), (33, 16)])
def test_page_bounds_brute_force(T, S):
    r = rng(6)
    D = 7
    k = r.normal(size=(T, D))
    mn, mx = oracle.page_bounds(k, S)
    P = (T + S - 1) // S
    assert mn.shape == (P, D)
    for p in range(P):
        blk = k[p * S:(p + 1) * S]
        assert np.array_equal(mn[p], blk.min(axis=0)) and np.array_equal(mx[p], blk.max(axis=0))
        assert (blk >= mn[p]).all() and (blk <= mx[p]).all()
    if T % S == 1:                    # single-token last page: min == max == that key
        assert np.array_equal(mn[-1], k[-1]) and np.array_equal(mx[-1], k[-1])


# ------------------------------------------------------------------ scores
def test_scores_upper_bound_property():
    """U_p >= max over the page's tokens of q.k, with equality for one-token pages."""
    r = rng(7)
    T, D, S = 16 * 9 + 1, 16, 16
    k = r.normal(size=(T, D))
    mn, mx = oracle.page_bounds(k, S)
    for trial in range(20):
        q = r.normal(size=D)
        U = oracle.page_scores(q, mn, mx)
        for p in range(mn.shape[0]):
            true = (k[p * S:(p + 1) * S] @ q).max()
            assert U[p] >= true - 1e-12
        assert abs(U[-1] - k[-1] @ q) < 1e-12       # last page has one token
    # the bound is attained: a page whose tokens are the two opposite corners per sign of q
    q = r.normal(size=D)
    corner = np.where(q >= 0, 3.0, -2.0)
    other = np.where(q >= 0, -2.0, 3.0)
    mn2, mx2 = oracle.page_bounds(np.stack([corner, other]), 2)
    assert abs(oracle.page_scores(q, mn2, mx2)[0] - corner @ q) < 1e-12


def test_scores_homogeneity_permutation_and_sign():
    r = rng(8)
    P, D = 11, 9
    a, b = r.normal(size=(P, D)), r.normal(size=(P, D))
    mn, mx = np.minimum(a, b), np.maximum(a, b)
    q = r.normal(size=D)
    U = oracle.page_scores(q, mn, mx)
    np.testing.assert_allclose(oracle.page_scores(3.5 * q, mn, mx), 3.5 * U, rtol=1e-13)
    perm = r.permutation(D)
    np.testing.assert_allclose(oracle.page_scores(q[perm], mn[:, perm], mx[:, perm]), U, rtol=1e-13)
    # negating q swaps the roles of min and max
    np.testing.assert_allclose(oracle.page_scores(-q, mn, mx), oracle.page_scores(q, -mx, -mn), rtol=1e-13)
    # one-hot queries read out max (positive) or -min (negative) of that channel
    e = np.zeros(D)
    e[4] = 1.0
    assert np.array_equal(oracle.page_scores(e, mn, mx), mx[:, 4])
    assert np.array_equal(oracle.page_scores(-e, mn, mx), -mn[:, 4])


# ------------------------------------------------------------------ selection
def _select_brute(U, K, n_sink, n_local):
    P = len(U)
    if K >= P:
        return list(range(P))
    forced = []
    for p in range(min(n_sink, P)):
        forced.append(p)
    for p in range(P - 1, max(P - 1 - n_local, -1), -1):
        if p not in forced:
            forced.append(p)
    forced = forced[:K]
    rest = sorted((p for p in range(P) if p not in forced), key=lambda p: (-U[p], p))
    return sorted(forced + rest[:K - len(forced)])


@pytest.mark.parametrize("n_sink,n_local", [(1, 1), (0, 0), (2, 3), (0, 1), (4, 0)])
def test_select_against_full_sort(n_sink, n_local):
    r = rng(9)
    for P in (1, 2, 5, 17, 64):
        for K in (1, 2, 3, 4, 7, 16, 64, 100):
            U = np.round(r.normal(size=P), 1)        # rounding creates many exact ties
            idx, _ = oracle.select_pages(U, K, n_sink, n_local)
            assert list(idx) == _select_brute(U, K, n_sink, n_local), (P, K)


def test_select_special_cases():
    r = rng(10)
    U = r.normal(size=40)
    idx, _ = oracle.select_pages(U, 1, 0, 0)
    assert list(idx) == [int(np.argmax(U))]
    idx, _ = oracle.select_pages(U, 40, 1, 1)
    assert list(idx) == list(range(40))
    idx, _ = oracle.select_pages(U, 1000, 1, 1)
    assert list(idx) == list(range(40))
    for trial in range(10):                          # forced pages are there whatever the scores
        U = r.normal(size=40)
        U[0] = U[39] = -1e9
        idx, _ = oracle.select_pages(U, 5, 1, 1)
        assert idx[0] == 0 and idx[-1] == 39 and len(idx) == 5 and (np.diff(idx) > 0).all()
    # all equal: lower indices win
    idx, _ = oracle.select_pages(np.zeros(10), 4, 0, 0)
    assert list(idx) == [0, 1, 2, 3]
    idx, _ = oracle.select_pages(np.zeros(10), 4, 1, 1)
    assert list(idx) == [0, 1, 2, 9]


def test_select_near_tie_flag():
    U = np.array([5.0, 1.0, 3.0, 3.0 * (1 - 5e-6), 0.5, 0.1])
    idx, nt = oracle.select_pages(U, 3, 0, 0)       # cut between 3.0 and 3.0*(1-5e-6)
    assert list(idx) == [0, 2, 3] and nt is False   # takes 5, 3, 2.999985; next is 1.0: far
    idx, nt = oracle.select_pages(U, 2, 0, 0)       # cut falls between the two near-equal scores
    assert list(idx) == [0, 2] and nt is True
    U[3] = 3.0 * (1 - 5e-5)
    idx, nt = oracle.select_pages(U, 2, 0, 0)
    assert nt is False


def test_budget_arithmetic_from_paper_tables():
    """K blocks of the stated size at a 4K context equal the stated budget, so forced
    first/local blocks must count inside K: the selection returns exactly K pages."""
    for line in open(os.path.join(GOLDEN, "budget_arithmetic.txt")):
        if line.startswith("#") or not line.strip():
            continue
        ctx, block, K, num, den = map(int, line.split())
        P = ctx // block
        assert K * den == P * num
        idx, _ = oracle.select_pages(rng(K).normal(size=P), K, 1, 1)
        assert len(idx) == K and len(idx) * block * den == ctx * num


# ------------------------------------------------------------------ attention
def _dense_two_pass(q, K, V, scale):
    s = (K @ q) * scale
    w = np.exp(s - s.max())
    return (w[:, None] * V).sum(0) / w.sum()


@pytest.mark.parametrize("T", [48, 53, 7])
def test_attention_full_budget_is_dense_softmax(T):
    r = rng(11)
    D, S = 8, 16
    k, v, q = r.normal(size=(T, D)), r.normal(size=(T, D)), r.normal(size=D)
    P = (T + S - 1) // S
    y = oracle.sparse_attention(q, 0.3, k, v, np.arange(P), S)
    np.testing.assert_allclose(y, _dense_two_pass(q, k, v, 0.3), rtol=1e-12)
    tq = torch.from_numpy(q)[None, None, None, :]
    tk = torch.from_numpy(k)[None, None]
    tv = torch.from_numpy(v)[None, None]
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, scale=0.3)[0, 0, 0].numpy()
    np.testing.assert_allclose(y, ref, rtol=1e-10)


def test_attention_subset_convexity_single_token_and_shift():
    r = rng(12)
    T, D, S = 100, 6, 16
    k, v, q = r.normal(size=(T, D)), r.normal(size=(T, D)), r.normal(size=D)
    idx = np.array([0, 3, 6])                        # page 6 is ragged: tokens 96..99
    toks = np.r_[0:16, 48:64, 96:100]
    y = oracle.sparse_attention(q, 0.5, k, v, idx, S)
    np.testing.assert_allclose(y, _dense_two_pass(q, k[toks], v[toks], 0.5), rtol=1e-12)
    assert (y >= v[toks].min(0) - 1e-12).all() and (y <= v[toks].max(0) + 1e-12).all()
    # one selected token: the output is that value row
    y1 = oracle.sparse_attention(q, 0.5, k[:97], v[:97], np.array([6]), S)
    np.testing.assert_allclose(y1, v[96], rtol=1e-14)
    # adding one vector to every key shifts all logits equally: output unchanged
    u = r.normal(size=D)
    y2 = oracle.sparse_attention(q, 0.5, k + u, v, idx, S)
    np.testing.assert_allclose(y2, y, rtol=1e-10)
    # a huge logit dominates: output -> that token's value
    kk = k.copy()
    kk[50] = 100 * q / np.linalg.norm(q)
    y3 = oracle.sparse_attention(q, 1.0, kk, v, idx, S)
    np.testing.assert_allclose(y3, v[50], atol=1e-10)


# ------------------------------------------------------------------ chained object
def test_head_matches_stage_functions_and_prefill_decode_equivalence():
    r = rng(13)
    T, D, S = 77, 8, 16
    k, v = r.normal(size=(T + 1, D)), r.normal(size=(T + 1, D))
    g = 1 / (1 + np.exp(-r.normal(4.12, 0.5, size=(T + 1, D))))
    q = r.normal(size=D)
    for dtype in (oracle.BF16, oracle.F32):
        a = oracle.Head(D, S, 128, dtype)
        a.append(k[:T], v[:T], g[:T])
        a.append(k[T], v[T], g[T])                  # decode step appends one token
        b = oracle.Head(D, S, 128, dtype)
        b.append(k, v, g)                            # build(T+1)
        ea, eb = a.export(), b.export()
        for key in ea:
            assert np.array_equal(ea[key], eb[key]), key
        # against the stage functions
        kt, vt = oracle.recurrence(k, v, g)
        ks, vs = oracle.round_storage(kt, dtype), oracle.round_storage(vt, dtype)
        mn, mx = oracle.page_bounds(ks, S)
        assert np.array_equal(ea["k"], ks) and np.array_equal(ea["v"], vs)
        assert np.array_equal(ea["min"], mn) and np.array_equal(ea["max"], mx)
        np.testing.assert_allclose(ea["state_k"], kt[-1], rtol=0, atol=0)
        U = oracle.page_scores(q, mn, mx)
        idx, _ = oracle.select_pages(U, 3, 1, 1)
        y = oracle.sparse_attention(q, D ** -0.5, ks, vs, idx, S)
        out = a.query(q, 3, D ** -0.5, want_scores=True)
        assert np.array_equal(out["idx"], idx) and np.array_equal(out["U"], U)
        assert np.array_equal(out["y"], y)
        ob = b.query(q, 3, D ** -0.5)
        assert np.array_equal(ob["y"], y)


def test_zero_gate_reduces_to_plain_attention_on_raw_kv():
    """Eq. 2: with g = 0 the method is the same sparse method on the raw K, V;
    at full budget that is textbook attention."""
    r = rng(14)
    T, D, S = 40, 8, 16
    k = np.float64(np.float32(r.normal(size=(T, D))))
    v = np.float64(np.float32(r.normal(size=(T, D))))
    q = r.normal(size=D)
    h = oracle.Head(D, S, 64, oracle.F32)
    h.append(k, v, np.zeros((T, D)))
    out = h.query(q, 100, 0.4)
    np.testing.assert_allclose(out["y"], _dense_two_pass(q, k, v, 0.4), rtol=1e-12)
    e = h.export()
    assert np.array_equal(e["k"], k) and np.array_equal(e["v"], v)


def test_capacity_is_enforced():
    h = oracle.Head(4, 16, 8, oracle.F32)
    h.append(np.zeros((8, 4)), np.zeros((8, 4)), np.zeros((8, 4)))
    with pytest.raises(ValueError):
        h.append(np.zeros((1, 4)), np.zeros((1, 4)), np.zeros((1, 4)))
    assert len(h) == 8
