"""Pins for the CPU oracle: every check here is against something other than the oracle
itself -- a library routine on a special case, a closed form, an invariant, an identity,
brute force on tiny vocabularies, or a figure printed in the paper."""
import os

import numpy as np
import pytest
from scipy.special import softmax as sp_softmax

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rng(seed):
    return np.random.default_rng(seed)


def _order(l):
    """(logit desc, index asc) by a library sort."""
    return np.lexsort((np.arange(l.size), -l.astype(np.float64)))


# ---------------------------------------------------------------------------------------
# compress: Eq. (4) top-k, plus top-p / renormalisation
# ---------------------------------------------------------------------------------------

@pytest.mark.parametrize("V,k,T", [(50, 5, 0.7), (333, 32, 1.0), (17, 17, 1.3), (9, 20, 0.5)])
def test_topk_equals_library_topk_then_softmax(V, k, T):
    # closed form: with pure top-k the full normaliser cancels, so the renormalised sparse
    # row is the softmax over the k selected logits alone
    rng = _rng(V * 1000 + k)
    l = rng.normal(0, 3, size=(2, 3, V)).astype(np.float32)
    Ts = np.array([T, T * 1.5], np.float32)
    qi, qp, qc, _ = oracle.compress(l, Ts, top_k=k, top_p=1.0, k_max=k)
    n = min(k, V)
    for b in range(2):
        for i in range(3):
            sel = _order(l[b, i])[:n]
            ref = sp_softmax(l[b, i, sel].astype(np.float64) / np.float64(Ts[b]))
            assert qc[b, i] == n
            assert np.array_equal(qi[b, i, :n], sel)
            assert np.all(qi[b, i, n:] == -1) and np.all(qp[b, i, n:] == 0)
            np.testing.assert_allclose(qp[b, i, :n], ref, rtol=2e-7, atol=0)


def test_topk_ties_take_lower_index_first():
    # integer logits force ties at the k-th value
    rng = _rng(7)
    l = rng.integers(-3, 4, size=(1, 4, 64)).astype(np.float32)
    qi, qp, qc, _ = oracle.compress(l, np.ones(1, np.float32), top_k=10, top_p=1.0, k_max=10)
    for i in range(4):
        assert np.array_equal(qi[0, i], _order(l[0, i])[:10])
    # all-equal logits: uniform over the first k indices
    l = np.full((1, 1, 40), 2.5, np.float32)
    qi, qp, qc, _ = oracle.compress(l, np.ones(1, np.float32), top_k=8, top_p=1.0, k_max=8)
    assert np.array_equal(qi[0, 0], np.arange(8))
    np.testing.assert_allclose(qp[0, 0], 1.0 / 8, rtol=1e-7)


@pytest.mark.parametrize("top_p,k_max,top_k", [(0.9, 64, 0), (0.5, 64, 0), (0.95, 8, 0), (0.9, 64, 4),
                                               (0.999, 200, 0)])
def test_top_p_invariants(top_p, k_max, top_k):
    rng = _rng(int(top_p * 1000) + k_max)
    V = 200
    ranks = rng.permuted(np.tile(np.arange(1, V + 1), (6, 1)), axis=1)
    l = (-1.2 * np.log(ranks) + rng.normal(0, 1.0, size=(6, V))).astype(np.float32).reshape(2, 3, V)
    T = np.array([0.8, 1.1], np.float32)
    tp = np.float32(top_p)
    qi, qp, qc, _ = oracle.compress(l, T, top_k=top_k, top_p=float(tp), k_max=k_max)
    for b in range(2):
        for i in range(3):
            q = sp_softmax(l[b, i].astype(np.float64) / np.float64(T[b]))
            order = _order(l[b, i])
            cum = np.cumsum(q[order])
            k_eff = min(top_k if top_k > 0 else k_max, k_max, V)
            n = qc[b, i]
            assert 1 <= n <= k_eff
            # support is exactly the first n of the sorted order
            assert np.array_equal(qi[b, i, :n], order[:n])
            assert np.all(qi[b, i, n:] == -1) and np.all(qp[b, i, n:] == 0)
            # nucleus rule: smallest prefix reaching top_p, capped at k_eff
            if n < k_eff:
                assert cum[n - 1] >= np.float64(tp)
            if n > 1:
                assert cum[n - 2] < np.float64(tp)
            # renormalised: sums to one, proportional to q on the support
            assert abs(qp[b, i, :n].astype(np.float64).sum() - 1.0) < 1e-6
            np.testing.assert_allclose(qp[b, i, :n], q[order[:n]] / cum[n - 1], rtol=3e-7)


def test_dense_limit_k_ge_V_gives_full_softmax():
    rng = _rng(3)
    V = 31
    l = rng.normal(0, 2, size=(1, 2, V)).astype(np.float32)
    T = np.array([0.9], np.float32)
    qi, qp, qc, _ = oracle.compress(l, T, top_k=0, top_p=1.0, k_max=V + 5)
    for i in range(2):
        assert qc[0, i] == V
        dense = np.zeros(V)
        dense[qi[0, i, :V]] = qp[0, i, :V]
        np.testing.assert_allclose(dense, sp_softmax(l[0, i].astype(np.float64) / np.float64(T[0])),
                                   rtol=2e-7)


def test_draft_token_draw_is_inverse_cdf_of_sparse_row():
    rng = _rng(11)
    V, k = 40, 6
    l = rng.normal(0, 2, size=(1, 1, V)).astype(np.float32)
    N = 4000
    ls = np.repeat(l, N, axis=0)
    u = ((np.arange(N) + 0.5) / N).astype(np.float32).reshape(N, 1)
    qi, qp, qc, tok = oracle.compress(ls, np.ones(N, np.float32), top_k=k, top_p=1.0, k_max=k, u_draft=u)
    # library inverse CDF
    cum = np.cumsum(qp[0, 0].astype(np.float64))
    ref = qi[0, 0][np.minimum(np.searchsorted(cum, u[:, 0].astype(np.float64) * cum[-1], side="right"), k - 1)]
    assert np.array_equal(tok[:, 0], ref)
    # empirical law of the draw equals the sparse row
    for j in range(k):
        assert abs(np.mean(tok[:, 0] == qi[0, 0, j]) - qp[0, 0, j]) < 2.0 / N + 1e-6


# ---------------------------------------------------------------------------------------
# verify: accept test, scan, residual mass
# ---------------------------------------------------------------------------------------

def test_q_equal_p_accepts_everything_and_residual_vanishes():
    rng = _rng(5)
    B, G, V = 6, 3, 23
    lt = rng.normal(0, 2, size=(B, G + 1, V)).astype(np.float32)
    T = rng.uniform(0.5, 1.5, size=B).astype(np.float32)
    qi, qp, qc, _ = oracle.compress(lt[:, :G], T, top_k=0, top_p=1.0, k_max=V)
    tok = rng.integers(0, V, size=(B, G)).astype(np.int32)
    for u_val in (0.0, 0.3, 0.999):
        u = np.full((B, G), u_val, np.float32)
        r = oracle.verify(lt, T, tok, qi, qp, qc, u, u_resample=np.full((B, 2), 0.5, np.float32))
        assert np.all(r["accept_len"] == G)
        assert np.all(np.abs(r["resid_mass"]) < 1e-6)


def test_scalar_q_reduces_to_textbook_speculative_test():
    # K = 1: the sparse row holds only the drafted token and the probability the drafter gave it
    # (the paper's uplink form); the decision is u < min(1, p(x)/q(x))
    rng = _rng(9)
    B, G, V = 400, 3, 12
    lt = rng.normal(0, 1.5, size=(B, G + 1, V)).astype(np.float32)
    T = np.full(B, 0.9, np.float32)
    tok = rng.integers(0, V, size=(B, G)).astype(np.int32)
    q = rng.uniform(0.02, 0.6, size=(B, G, 1)).astype(np.float32)
    qi = tok.reshape(B, G, 1).copy()
    qc = np.ones((B, G), np.int32)
    u = rng.uniform(0, 1, size=(B, G)).astype(np.float32)
    r = oracle.verify(lt, T, tok, qi, q, qc, u)
    p = sp_softmax(lt.astype(np.float64) / np.float64(T[0]), axis=-1)
    px = np.take_along_axis(p[:, :G], tok[..., None].astype(np.int64), axis=-1)[..., 0]
    acc = u.astype(np.float64) < np.minimum(1.0, px / q[..., 0].astype(np.float64))
    lead = np.where(acc.all(1), G, np.argmin(acc, axis=1))
    assert np.array_equal(r["accept_len"], lead)
    np.testing.assert_allclose(r["p_draft"], px, rtol=1e-12)
    # residual with a single-entry q: 1 - min(p(x), q(x))
    np.testing.assert_allclose(r["resid_mass"], 1.0 - np.minimum(px, q[..., 0]), rtol=1e-9)


def test_token_outside_support_is_accepted():
    rng = _rng(13)
    B, G, V = 3, 2, 30
    ld = rng.normal(0, 2, size=(B, G, V)).astype(np.float32)
    lt = rng.normal(0, 2, size=(B, G + 1, V)).astype(np.float32)
    T = np.ones(B, np.float32)
    qi, qp, qc, _ = oracle.compress(ld, T, top_k=4, top_p=1.0, k_max=4)
    tok = np.empty((B, G), np.int32)
    for b in range(B):
        for i in range(G):
            tok[b, i] = [v for v in range(V) if v not in qi[b, i]][0]
    r = oracle.verify(lt, T, tok, qi, qp, qc, np.full((B, G), 0.999, np.float32))
    assert np.all(r["accept_len"] == G)


def test_residual_mass_identity_and_accept_rate():
    # R = 1 - sum_{v in S} min(p_v, q~_v); the mean accept indicator over u tends to 1 - R when
    # the draft token is drawn from q~
    rng = _rng(17)
    G, V, k = 1, 64, 8
    ld = rng.normal(0, 2, size=(1, G, V)).astype(np.float32)
    lt = (0.6 * ld[0, 0] + rng.normal(0, 1.0, size=V)).astype(np.float32)
    lt = np.stack([lt, rng.normal(0, 1, size=V).astype(np.float32)])[None]
    T = np.array([0.8], np.float32)
    N = 200000
    u_d = rng.uniform(0, 1, size=(N, G)).astype(np.float32)
    qi, qp, qc, tok = oracle.compress(np.repeat(ld, N, 0), np.repeat(T, N), top_k=k, top_p=1.0,
                                      k_max=k, u_draft=u_d)
    u = rng.uniform(0, 1, size=(N, G)).astype(np.float32)
    r = oracle.verify(np.repeat(lt, N, 0), np.repeat(T, N), tok, qi, qp, qc, u, nthreads=4)
    p = sp_softmax(lt[0, 0].astype(np.float64) / np.float64(T[0]))
    R_id = 1.0 - np.minimum(p[qi[0, 0]], qp[0, 0].astype(np.float64)).sum()
    np.testing.assert_allclose(r["resid_mass"][:, 0], R_id, rtol=1e-10)
    rate = np.mean(r["accept_len"] == 1)
    assert abs(rate - (1.0 - R_id)) < 4 * np.sqrt(0.25 / N)


def test_borderline_count_only_counts_deciding_positions():
    # build ratios by hand: p(x)/q(x) known from a two-token vocabulary
    V, G = 2, 3
    lt = np.zeros((1, G + 1, V), np.float32)            # p = (0.5, 0.5) everywhere
    T = np.ones(1, np.float32)
    tok = np.zeros((1, G), np.int32)
    qi = np.zeros((1, G, 1), np.int32)
    qp = np.full((1, G, 1), 0.8, np.float32)            # ratio = 0.5 / 0.8 (fp32 0.8 widened)
    qc = np.ones((1, G), np.int32)
    ratio = 0.5 / np.float64(np.float32(0.8))
    near = np.float32(ratio)                            # within 6e-8 relative of the ratio
    far = np.float32(ratio * (1 - 1e-3))
    # position 0: far below -> accept, not borderline; position 1: near -> borderline, decides
    # either way; position 2: near, but only counted if position 1 accepted
    u = np.array([[far, near, near]], np.float32)
    r = oracle.verify(lt, T, tok, qi, qp, qc, u)
    acc1 = np.float64(near) < ratio
    assert r["accept_len"][0] == (3 if acc1 else 1)
    assert r["borderline_count"] == (2 if acc1 else 1)
    # a rejection far from the threshold stops the count
    u = np.array([[np.float32(0.9), near, near]], np.float32)
    r = oracle.verify(lt, T, tok, qi, qp, qc, u)
    assert r["accept_len"][0] == 0 and r["borderline_count"] == 0


# ---------------------------------------------------------------------------------------
# sampler: two-level inverse CDF and the residual distribution
# ---------------------------------------------------------------------------------------

def test_single_chunk_sampler_is_library_inverse_cdf():
    rng = _rng(19)
    V, N = 37, 3000
    lt = rng.normal(0, 2, size=(1, 1, V)).astype(np.float32)
    T = np.ones(N, np.float32)
    u = rng.uniform(0, 1, size=(N, 2)).astype(np.float32)
    tokens, mass = oracle.residual_sample(np.repeat(lt, N, 0), T, np.zeros(N, np.int32),
                                          np.zeros((N, 0, 1), np.int32), np.zeros((N, 0, 1), np.float32),
                                          np.zeros((N, 0), np.int32), u)
    p = sp_softmax(lt[0, 0].astype(np.float64))
    cum = np.cumsum(p)
    ref = np.searchsorted(cum, u[:, 1].astype(np.float64) * cum[-1], side="right")
    assert np.array_equal(tokens, np.minimum(ref, V - 1))
    np.testing.assert_allclose(mass, 1.0, rtol=1e-12)


@pytest.mark.parametrize("V,chunk,k", [(16, 4, 3), (13, 4, 5), (10, 3, 2)])
def test_two_level_sampler_law_on_grid(V, chunk, k):
    # brute force over a fine (u1, u2) grid: the area mapped to each token is r_v / R with
    # r = max(0, p - q~) written straight from the paper's definition
    rng = _rng(V * 7 + chunk)
    ld = rng.normal(0, 1.5, size=(1, 1, V)).astype(np.float32)
    lt = np.stack([(0.5 * ld[0, 0] + rng.normal(0, 1.2, size=V)).astype(np.float32),
                   rng.normal(0, 1, size=V).astype(np.float32)])[None]
    T = np.array([0.9], np.float32)
    qi, qp, qc, _ = oracle.compress(ld, T, top_k=k, top_p=1.0, k_max=k)
    n = 400
    g = (np.arange(n) + 0.5) / n
    u = np.stack(np.meshgrid(g, g, indexing="ij"), -1).reshape(-1, 2).astype(np.float32)
    N = u.shape[0]
    p = sp_softmax(lt[0].astype(np.float64) / np.float64(T[0]), axis=-1)
    for pos in (0, 1):
        tokens, mass = oracle.residual_sample(np.repeat(lt, N, 0), np.repeat(T, N),
                                              np.full(N, pos, np.int32), np.repeat(qi, N, 0),
                                              np.repeat(qp, N, 0), np.repeat(qc, N, 0), u,
                                              chunk=chunk, nthreads=4)
        if pos == 0:
            qd = np.zeros(V)
            qd[qi[0, 0, :k]] = qp[0, 0, :k]
            r = np.maximum(0.0, p[0] - qd)
        else:
            r = p[1]
        law = np.bincount(tokens, minlength=V) / N
        np.testing.assert_allclose(law, r / r.sum(), atol=3.0 / n)
        np.testing.assert_allclose(mass, r.sum(), rtol=1e-12)
        # zero residual weight is never drawn
        assert np.all(law[r == 0] == 0)


def test_zero_residual_falls_back_to_p():
    rng = _rng(23)
    V = 20
    lt = rng.normal(0, 2, size=(1, 2, V)).astype(np.float32)
    T = np.ones(1, np.float32)
    qi, qp, qc, _ = oracle.compress(lt[:, :1], T, top_k=0, top_p=1.0, k_max=V)
    # make q~ >= p everywhere: scale the stored probabilities up slightly
    qp = (qp * np.float32(1.001)).astype(np.float32)
    u = np.array([[0.3, 0.7]], np.float32)
    t_res, _ = oracle.residual_sample(lt, T, np.zeros(1, np.int32), qi, qp, qc, u)
    empty = (np.zeros((1, 1, 1), np.int32), np.zeros((1, 1, 1), np.float32), np.zeros((1, 1), np.int32))
    t_p, _ = oracle.residual_sample(lt, T, np.zeros(1, np.int32), *empty, u)
    assert t_res[0] == t_p[0]


def test_residual_counts_as_vanished_up_to_1e_12_of_the_row():
    # Sec. 3.3's norm(max(0, P - Q)) is undefined for a vanishing residual; the reading is: total
    # residual mass <= 1e-12 of the row -> draw from P itself.  Three entries: q~ = (0.5, 0.5) covers
    # the first two (each p there is a little below 0.5), so the residual is p_2 alone.
    T = np.ones(1, np.float32)
    qi = np.array([[[0, 1]]], np.int32)
    qp = np.array([[[0.5, 0.5]]], np.float32)
    qc = np.array([[2]], np.int32)
    pos = np.zeros(1, np.int32)
    u = np.array([[0.2, 0.3]], np.float32)
    for gap, vanished in ((23.0, False), (32.0, True)):
        lt = np.zeros((1, 2, 3), np.float32)
        lt[0, 0, 2] = -gap
        p2 = np.exp(-gap) / (2.0 + np.exp(-gap))
        assert (p2 <= 1e-12) == vanished and p2 > 0
        tok, mass = oracle.residual_sample(lt, T, pos, qi, qp, qc, u)
        if vanished:
            # the draw is from p: u1 = 0.2 lands in the single chunk, u2 = 0.3 < p_0 picks entry 0
            assert tok[0] == 0 and abs(mass[0] - 1.0) < 1e-12
        else:
            # the only entry with residual weight, whatever the uniforms
            assert tok[0] == 2 and abs(mass[0] / p2 - 1.0) < 1e-9


# ---------------------------------------------------------------------------------------
# whole method: output law equals the target distribution (Sec. 2.1 / Sec. 3.3 claim)
# ---------------------------------------------------------------------------------------

@pytest.mark.parametrize("V,k,top_p,chunk", [(16, 5, 1.0, 4), (12, 12, 0.8, 5), (8, 3, 1.0, 1024)])
def test_output_law_equals_target_per_position(V, k, top_p, chunk):
    # Monte Carlo over all uniforms with the draft token drawn from q~: conditional on reaching
    # position i, the emitted token at i follows p_i
    rng = _rng(V + k)
    G, N = 3, 400000
    ld = rng.normal(0, 1.5, size=(1, G, V)).astype(np.float32)
    lt = np.concatenate([(0.7 * ld[0] + rng.normal(0, 0.9, size=(G, V))).astype(np.float32),
                         rng.normal(0, 1, size=(1, V)).astype(np.float32)])[None]
    T = np.array([0.85], np.float32)
    Ts = np.repeat(T, N)
    qi, qp, qc, tok = oracle.compress(np.repeat(ld, N, 0), Ts, top_k=k, top_p=top_p, k_max=k,
                                      u_draft=rng.uniform(0, 1, size=(N, G)).astype(np.float32),
                                      nthreads=4)
    r = oracle.verify(np.repeat(lt, N, 0), Ts, tok, qi, qp, qc,
                      rng.uniform(0, 1, size=(N, G)).astype(np.float32),
                      u_resample=rng.uniform(0, 1, size=(N, 2)).astype(np.float32),
                      chunk=chunk, nthreads=4)
    p = sp_softmax(lt[0].astype(np.float64) / np.float64(T[0]), axis=-1)
    a = r["accept_len"]
    for i in range(G + 1):
        reach = a >= i
        emitted = np.where(a[reach] > i, tok[reach, min(i, G - 1)], r["token"][reach])
        n_i = reach.sum()
        assert n_i > 5000
        law = np.bincount(emitted, minlength=V) / n_i
        sigma = np.sqrt(p[i] * (1 - p[i]) / n_i)
        assert np.all(np.abs(law - p[i]) < 4.5 * sigma + 1e-9), (i, np.abs(law - p[i]).max())


def test_exact_law_by_enumeration_tiny():
    # V = 4, gamma = 1: enumerate the draft token over the support and integrate the uniforms
    # on a grid fine enough that the discretisation error is below the tolerance
    rng = _rng(29)
    V, k = 4, 2
    ld = rng.normal(0, 1, size=(1, 1, V)).astype(np.float32)
    lt = rng.normal(0, 1, size=(1, 2, V)).astype(np.float32)
    T = np.ones(1, np.float32)
    qi, qp, qc, _ = oracle.compress(ld, T, top_k=k, top_p=1.0, k_max=k)
    p = sp_softmax(lt[0, 0].astype(np.float64))
    n = 160
    g = ((np.arange(n) + 0.5) / n).astype(np.float32)
    ua, u1, u2 = [x.reshape(-1) for x in np.meshgrid(g, g, g, indexing="ij")]
    N = ua.size
    law = np.zeros(V)
    for j in range(k):
        tok = np.full((N, 1), qi[0, 0, j], np.int32)
        r = oracle.verify(np.repeat(lt, N, 0), np.ones(N, np.float32), tok, np.repeat(qi, N, 0),
                          np.repeat(qp, N, 0), np.repeat(qc, N, 0), ua.reshape(N, 1),
                          u_resample=np.stack([u1, u2], -1), chunk=2, nthreads=4)
        out = np.where(r["accept_len"] == 1, tok[:, 0], r["token"])
        law += float(qp[0, 0, j]) * np.bincount(out, minlength=V) / N
    np.testing.assert_allclose(law, p, atol=2.5 / n)


def test_expected_length_matches_eq5():
    rows = [ln.split() for ln in open(os.path.join(GOLDEN, "expected_length.txt")) if ln[0] not in "#\n"]
    rng = _rng(31)
    V = 2
    for alpha_s, gamma_s, el_s in rows:
        alpha, G, EL = float(alpha_s), int(gamma_s), float(el_s)
        # two-token vocabulary, q~ = (1, 0) on token 0, p = (alpha, 1 - alpha): the accept
        # probability of the (always drafted) token 0 is exactly alpha at every position
        N = 200000 if alpha > 0 else 1000
        if alpha > 0:
            lt = np.log(np.array([alpha, 1 - alpha])).astype(np.float32)
        else:
            lt = np.array([-np.inf, 0.0], np.float32)
        lt = np.tile(lt, (N, G + 1, 1))
        tok = np.zeros((N, G), np.int32)
        qi = np.zeros((N, G, 1), np.int32)
        qp = np.ones((N, G, 1), np.float32)
        qc = np.ones((N, G), np.int32)
        u = rng.uniform(0, 1, size=(N, G)).astype(np.float32)
        r = oracle.verify(lt, np.ones(N, np.float32), tok, qi, qp, qc, u, nthreads=4)
        gen_len = np.minimum(r["accept_len"] + 1, G)       # Eq. (5) caps the cycle at gamma
        assert abs(gen_len.mean() - EL) < 0.01, (alpha, gen_len.mean(), EL)
        # with the bonus row the per-call yield is (1 - alpha^(gamma+1)) / (1 - alpha)
        full = (1 - alpha ** (G + 1)) / (1 - alpha)
        assert abs((r["accept_len"] + 1).mean() - full) < 0.012


# ---------------------------------------------------------------------------------------
# printed figures and degenerate inputs
# ---------------------------------------------------------------------------------------

def test_sparse_layout_matches_printed_payload_sizes():
    vals = {}
    for ln in open(os.path.join(GOLDEN, "payload_sizes.txt")):
        ln = ln.split("#")[0].split()
        if ln:
            vals[ln[0]] = ln[1:]
    V = int(vals["vocab_llama31"][0])
    K = int(vals["topk_example_k"][0])
    l = np.zeros((1, 1, V), np.float32)
    qi, qp, qc, _ = oracle.compress(l, np.ones(1, np.float32), top_k=K, top_p=1.0, k_max=K)
    entry = qi.dtype.itemsize + qp.dtype.itemsize
    assert entry == 8
    assert qi[0, 0].nbytes + qp[0, 0].nbytes == int(vals["topk_row_bytes"][0]) < int(vals["topk_row_bytes"][2])
    full = V * qp.dtype.itemsize
    assert full == int(vals["full_row_bytes"][0])
    assert abs(full - int(vals["full_row_bytes"][2])) / full < 0.03
    g = int(vals["uplink_gamma"][0])
    assert g * entry == int(vals["uplink_bytes"][0]) < int(vals["uplink_bytes"][2])


def test_minus_inf_logits_have_zero_weight():
    V = 10
    l = np.full((1, 2, V), -np.inf, np.float32)
    l[0, :, [2, 7]] = 0.0
    T = np.ones(1, np.float32)
    qi, qp, qc, _ = oracle.compress(l[:, :1], T, top_k=4, top_p=1.0, k_max=4)
    assert list(qi[0, 0, :2]) == [2, 7]
    np.testing.assert_allclose(qp[0, 0], [0.5, 0.5, 0, 0])
    for u2 in (0.1, 0.6, 0.99):
        t, _ = oracle.residual_sample(l, T, np.array([1], np.int32), qi, qp, qc,
                                      np.array([[0.5, u2]], np.float32))
        assert t[0] in (2, 7)


def test_invalid_inputs_are_flagged_not_sampled():
    rng = _rng(37)
    B, G, V = 4, 2, 16
    ld = rng.normal(size=(B, G, V)).astype(np.float32)
    lt = rng.normal(size=(B, G + 1, V)).astype(np.float32)
    T = np.ones(B, np.float32)
    ld[1, 0, 3] = np.nan
    qi, qp, qc, tok = oracle.compress(ld, T, top_k=4, top_p=1.0, k_max=4,
                                      u_draft=np.full((B, G), 0.5, np.float32))
    assert qc[1, 0] == -1 and tok[1, 0] == -1 and np.all(qi[1, 0] == -1)
    assert qc[0, 0] == 4 and qc[1, 1] == 4
    lt[2, 1, 5] = np.inf
    T2 = T.copy()
    T2[3] = 0.0
    u = np.full((B, G), 0.5, np.float32)
    r = oracle.verify(lt, T2, np.where(tok < 0, 0, tok), qi, qp, qc, u,
                      u_resample=np.full((B, 2), 0.5, np.float32))
    assert r["accept_len"][0] >= 0 and r["token"][0] >= 0
    for b in (1, 2, 3):           # bad count / +inf logit / zero temperature
        assert r["accept_len"][b] == -1 and r["token"][b] == -1
        assert np.all(r["p_draft"][b] == -1) and np.all(r["resid_mass"][b] == -1)


# ---------------------------------------------------------------------------------------------
# The paper's own direction (Sec. 3.3): Top-K of the target row on the verifier (Eq. 4),
# resampling against the drafter's dense row on the edge
# ---------------------------------------------------------------------------------------------

def test_target_topk_is_library_softmax_at_the_k_largest_logits():
    # Eq. (4): the K components with the highest probabilities and their indices, unnormalised
    rng = _rng(101)
    B, R, V, K = 5, 3, 97, 7
    l = rng.normal(size=(B, R, V)).astype(np.float32) * 2
    l[2, 1, 10] = l[2, 1, 3] = l[2, 1, 50] = 40.0         # ties: lower index first
    T = rng.uniform(0.5, 1.5, size=B).astype(np.float32)
    pos = np.array([0, 2, 1, 1, 0], np.int32)
    pi, pp, pc = oracle.target_topk(l, T, pos, K)
    for b in range(B):
        row = l[b, pos[b]].astype(np.float64)
        p = sp_softmax(row / np.float64(T[b]))
        order = np.lexsort((np.arange(V), -row))[:K]
        assert list(pi[b]) == list(order) and pc[b] == K
        np.testing.assert_allclose(pp[b], p[order], rtol=2e-7)
        assert pp[b].astype(np.float64).sum() <= 1.0 + 1e-6
    assert list(pi[2, :3]) == [3, 10, 50]
    # K >= V: the whole distribution, summing to one
    pi, pp, pc = oracle.target_topk(l, T, pos, V + 5)
    assert np.all(pc == V) and np.all(pi[:, V:] == -1) and np.all(pp[:, V:] == 0)
    np.testing.assert_allclose(pp.astype(np.float64).sum(1), 1.0, atol=1e-6)
    # a position outside the sequence's rows and a bad temperature are flagged
    T2 = T.copy()
    T2[1] = -1.0
    pi, pp, pc = oracle.target_topk(l, T2, np.array([0, 2, 3, 1, -1], np.int32), K)
    assert list(pc) == [K, -1, -1, K, -1] and np.all(pi[1] == -1)


def _edge_reference(draft_row, T, idx, prob, u):
    """norm(max(0, P~ - Q)) over the transmitted components, flat inverse CDF, by library calls."""
    q = sp_softmax(draft_row.astype(np.float64) / np.float64(T))
    r = np.maximum(0.0, prob.astype(np.float64) - q[idx])
    if not r.sum() > 0:
        r = prob.astype(np.float64)
    cum = np.cumsum(r)
    t = int(np.searchsorted(cum, np.float64(u) * cum[-1], side="right"))      # first cum > u * R
    if t >= len(r):
        t = int(np.nonzero(r > 0)[0][-1])
    return int(idx[t]), float(cum[-1])


def test_edge_resample_is_the_formula_of_sec_3_3_over_the_transmitted_components():
    rng = _rng(103)
    B, R, V, K = 6, 2, 64, 9
    lt = rng.normal(size=(B, R, V)).astype(np.float32) * 2
    ld = (0.6 * lt + rng.normal(size=(B, R, V))).astype(np.float32)
    T = rng.uniform(0.6, 1.3, size=B).astype(np.float32)
    pos = rng.integers(0, R, size=B).astype(np.int32)
    pi, pp, pc = oracle.target_topk(lt, T, pos, K)
    for u in np.linspace(0.0, 0.999, 41, dtype=np.float32):
        tok, mass = oracle.edge_resample(ld, T, pos, pi, pp, pc, np.full(B, u, np.float32))
        for b in range(B):
            t_ref, m_ref = _edge_reference(ld[b, pos[b]], T[b], pi[b], pp[b], u)
            assert tok[b] == t_ref
            assert abs(mass[b] - m_ref) <= 1e-12 * max(1.0, m_ref)
            assert tok[b] in pi[b]                      # only transmitted components can be drawn


def test_edge_resample_law_and_zero_weight_entries():
    # the measure of u that maps to a component equals r_t / R; components with P~ <= Q are never drawn
    rng = _rng(107)
    V, K = 12, 12
    lt = rng.normal(size=(1, 1, V)).astype(np.float32) * 1.5
    ld = rng.normal(size=(1, 1, V)).astype(np.float32) * 1.5
    T = np.ones(1, np.float32)
    pos = np.zeros(1, np.int32)
    pi, pp, pc = oracle.target_topk(lt, T, pos, K)
    q = sp_softmax(ld[0, 0].astype(np.float64))
    r = np.maximum(0.0, pp[0].astype(np.float64) - q[pi[0]])
    N = 20000
    counts = np.zeros(V)
    us = ((np.arange(N) + 0.5) / N).astype(np.float32)
    for u in us:
        tok, _ = oracle.edge_resample(ld, T, pos, pi, pp, pc, np.array([u], np.float32))
        counts[tok[0]] += 1
    law = np.zeros(V)
    law[pi[0]] = r / r.sum()
    np.testing.assert_allclose(counts / N, law, atol=2.0 / N + 1e-6)
    assert np.all(counts[pi[0][r == 0]] == 0)


def test_edge_resample_falls_back_to_the_transmitted_components_when_q_covers_them():
    V, K = 8, 3
    ld = np.zeros((1, 1, V), np.float32)
    ld[0, 0, :3] = 5.0                                   # Q puts ~1/3 on each of ids 0, 1, 2
    T = np.ones(1, np.float32)
    pos = np.zeros(1, np.int32)
    pi = np.array([[0, 1, 2]], np.int32)
    pp = np.array([[0.2, 0.1, 0.05]], np.float32)        # all below Q: residual identically zero
    pc = np.array([3], np.int32)
    seen = set()
    for u in np.linspace(0.0, 0.999, 50, dtype=np.float32):
        tok, mass = oracle.edge_resample(ld, T, pos, pi, pp, pc, np.array([u], np.float32))
        seen.add(int(tok[0]))
        assert abs(mass[0] - 0.35) < 1e-6
    assert seen == {0, 1, 2}
    tok, _ = oracle.edge_resample(ld, T, pos, pi, pp, pc, np.array([0.5], np.float32))
    assert tok[0] == 0                                   # cum 0.2 > 0.5 * 0.35
    tok, _ = oracle.edge_resample(ld, T, pos, pi, pp, pc, np.array([0.6], np.float32))
    assert tok[0] == 1


def test_scalar_uplink_plus_edge_resample_with_full_downlink_reproduces_the_target_law():
    # Sec. 3.3 with K = V (nothing truncated): the drafter samples x ~ Q and sends q(x) only; the
    # verifier accepts with min(1, p(x)/q(x)); on rejection the edge resamples from
    # norm(max(0, P - Q)).  The output law must be P (Sec. 2.1).  Exact enumeration over x, the
    # accept probability integrated analytically, the edge law measured on a uniform grid.
    rng = _rng(109)
    V = 10
    lt = rng.normal(size=(1, 2, V)).astype(np.float32) * 1.5
    ld = (0.5 * lt[:, :1] + rng.normal(size=(1, 1, V))).astype(np.float32)
    T = np.array([0.9], np.float32)
    p = sp_softmax(lt[0, 0].astype(np.float64) / np.float64(T[0]))
    q = sp_softmax(ld[0, 0].astype(np.float64) / np.float64(T[0]))
    # the verifier's accept test with the scalar q(x): K = 1 sparse rows holding (x, q(x))
    acc_prob = np.zeros(V)
    for x in range(V):
        qi = np.array([[[x]]], np.int32)
        qp = np.array([[[q[x]]]], np.float32)
        qc = np.array([[1]], np.int32)
        tok = np.array([[x]], np.int32)
        us = np.linspace(0.0, 0.9999, 2001, dtype=np.float32)
        acc = [oracle.verify(lt, T, tok, qi, qp, qc, np.array([[u]], np.float32))["accept_len"][0] for u in us]
        acc_prob[x] = np.mean(acc)
        assert abs(acc_prob[x] - min(1.0, p[x] / q[x])) < 2e-3
    # the edge's law with everything transmitted
    pos = np.zeros(1, np.int32)
    pi, pp, pc = oracle.target_topk(lt, T, pos, V)
    N = 20000
    edge = np.zeros(V)
    for u in ((np.arange(N) + 0.5) / N).astype(np.float32):
        tok, _ = oracle.edge_resample(ld, T, pos, pi, pp, pc, np.array([u], np.float32))
        edge[tok[0]] += 1.0 / N
    out = q * np.minimum(1.0, p / q) + (1.0 - np.sum(np.minimum(p, q))) * edge
    np.testing.assert_allclose(out, p, atol=5e-4)


def test_edge_resample_flags_unusable_input():
    rng = _rng(113)
    B, R, V, K = 5, 2, 20, 4
    lt = rng.normal(size=(B, R, V)).astype(np.float32)
    ld = rng.normal(size=(B, R, V)).astype(np.float32)
    T = np.ones(B, np.float32)
    pos = np.zeros(B, np.int32)
    pi, pp, pc = oracle.target_topk(lt, T, pos, K)
    ld[1, 0, 7] = np.nan
    pi[2, 1] = V
    pc[3] = K + 1
    pos2 = pos.copy()
    pos2[4] = R
    tok, mass = oracle.edge_resample(ld, T, pos2, pi, pp, pc, np.full(B, 0.5, np.float32))
    assert tok[0] >= 0 and mass[0] > 0
    assert list(tok[1:]) == [-1, -1, -1, -1] and np.all(mass[1:] == -1)


# ---------------------------------------------------------------------------------------------
# Prefix / incremental verification (Sec. 3.2 Fast Verification; Sec. 3.3 truncated segments)
# ---------------------------------------------------------------------------------------------

def _range_case(seed, B=12, G=6, V=40, K=6):
    rng = _rng(seed)
    ld = rng.normal(size=(B, G, V)).astype(np.float32) * 2
    lt = (0.8 * np.concatenate([ld, ld[:, :1]], axis=1) + rng.normal(size=(B, G + 1, V))).astype(np.float32)
    T = rng.uniform(0.6, 1.2, size=B).astype(np.float32)
    qi, qp, qc, tok = oracle.compress(ld, T, top_k=K, top_p=1.0, k_max=K, u_draft=rng.random((B, G)).astype(np.float32))
    ua = rng.random((B, G)).astype(np.float32)
    ur = rng.random((B, 2)).astype(np.float32)
    return lt, T, tok, qi, qp, qc, ua, ur


@pytest.mark.parametrize("cuts", [[0, 7], [0, 1, 2, 3, 4, 5, 6, 7], [0, 3, 7], [0, 2, 5, 6, 7], [0, 6, 7]])
def test_verifying_in_row_ranges_equals_verifying_at_once(cuts):
    # rows arrive in pieces; carrying the state through the calls must give what pso_verify gives
    lt, T, tok, qi, qp, qc, ua, ur = _range_case(201)
    B, G = tok.shape
    full = oracle.verify(lt, T, tok, qi, qp, qc, ua, ur)
    out, state, border = None, None, 0
    decided_at = np.full(B, -1)
    for r0, r1 in zip(cuts[:-1], cuts[1:]):
        # rows at and beyond r1 have not arrived: poison them to show they are not read
        seen = lt.copy()
        seen[:, r1:] = np.nan
        out = oracle.verify_range(seen, T, None, r0, r1, state, tok, qi, qp, qc, ua, ur, out=out)
        state = out["state"]
        border += out["borderline_count"]
        undecided = state == 1
        assert np.all(out["accept_len"][undecided] == -2) and np.all(out["token"][undecided] == -2)
        decided_at[(decided_at < 0) & ~undecided] = r1
    assert np.all(state == 0)
    assert np.array_equal(out["accept_len"], full["accept_len"])
    assert np.array_equal(out["token"], full["token"])
    assert border == full["borderline_count"]
    for b in range(B):
        a = int(full["accept_len"][b])
        assert decided_at[b] == min(r for r in cuts[1:] if r > a)   # decided by the first call that sees row a
        n = min(int(decided_at[b]), G)                       # positions of the calls up to the decision
        np.testing.assert_array_equal(out["p_draft"][b, :n], full["p_draft"][b, :n])
        np.testing.assert_array_equal(out["resid_mass"][b, :n], full["resid_mass"][b, :n])
        assert np.all(np.isnan(out["p_draft"][b, n:]))       # positions of later calls were never tested


def test_truncated_segments_equal_verifying_the_shorter_sequence():
    # gamma[b] < G: the sequence's rows are 0 .. gamma[b], row gamma[b] is its bonus row
    lt, T, tok, qi, qp, qc, ua, ur = _range_case(203)
    B, G = tok.shape
    rng = _rng(5)
    gamma = rng.integers(0, G + 1, size=B).astype(np.int32)
    gamma[0], gamma[1] = 0, G
    out = oracle.verify_range(lt, T, gamma, 0, G + 1, None, tok, qi, qp, qc, ua, ur)
    assert np.all(out["state"] == 0)
    for b in range(B):
        g = int(gamma[b])
        ref = oracle.verify(lt[b:b + 1, :g + 1], T[b:b + 1], tok[b:b + 1, :g], qi[b:b + 1, :g], qp[b:b + 1, :g],
                            qc[b:b + 1, :g], ua[b:b + 1, :g], ur[b:b + 1])
        assert out["accept_len"][b] == ref["accept_len"][0] and out["token"][b] == ref["token"][0]


def test_range_call_skips_decided_sequences_and_flags_bad_input():
    lt, T, tok, qi, qp, qc, ua, ur = _range_case(207)
    B, G = tok.shape
    state = np.ones(B, np.int32)
    state[3] = 0
    prev = {"accept_len": np.full(B, 77, np.int32), "token": np.full(B, 88, np.int32),
            "p_draft": np.full((B, G), 0.5), "resid_mass": np.full((B, G), 0.25)}
    lt2 = lt.copy()
    lt2[4, 1, 7] = np.inf               # inside the range
    lt2[5, 5, 7] = np.nan               # outside the range: not read
    gamma = np.full(B, G, np.int32)
    gamma[6] = G + 1                    # out of range
    out = oracle.verify_range(lt2, T, gamma, 0, 3, state, tok, qi, qp, qc, ua, ur, out=prev)
    assert out["accept_len"][3] == 77 and out["token"][3] == 88 and out["state"][3] == 0
    assert np.all(out["p_draft"][3] == 0.5)
    for b in (4, 6):
        assert out["accept_len"][b] == -1 and out["token"][b] == -1 and out["state"][b] == 0
    assert out["accept_len"][5] in (-2, 0, 1, 2)
    # an undecided sequence whose bonus row lies before the range is a caller error
    out = oracle.verify_range(lt, T, np.full(B, 1, np.int32), 3, 5, None, tok, qi, qp, qc, ua, ur)
    assert np.all(out["accept_len"] == -1)


# ---------------------------------------------------------------------------------------------
# Wire format of the sparse rows (Sec. 3.3) and the throughput model (Sec. 3.4, Eqs. 5-10)
# ---------------------------------------------------------------------------------------------

def _wire_case(seed, R=7, K=10):
    rng = _rng(seed)
    l = rng.normal(size=(R, 1, 500)).astype(np.float32) * 3
    qi, qp, qc, _ = oracle.compress(l, np.ones(R, np.float32), top_k=0, top_p=0.8, k_max=K)
    return qi.reshape(R, K), qp.reshape(R, K), qc.reshape(R)


def test_wire_message_sizes_match_the_printed_payload_figures():
    from oracle import wire
    vals = {}
    for ln in open(os.path.join(GOLDEN, "payload_sizes.txt")):
        ln = ln.split("#")[0].split()
        if ln:
            vals[ln[0]] = ln[1:]
    K = int(vals["topk_example_k"][0])
    qi = np.arange(K, dtype=np.int32).reshape(1, K)
    qp = np.full((1, K), 0.1, np.float32)
    qc = np.array([K], np.int32)
    pairs = int(vals["topk_row_bytes"][0])
    m32 = wire.pack(qi, qp, qc, wire.F32)
    # the (id, prob) pairs are the printed 80 bytes; the whole message adds a 16-byte header and the count
    assert m32.size == 16 + 4 + pairs
    m16 = wire.pack(qi, qp, qc, wire.F16)
    assert m16.size == 16 + 4 + 4 * K + 2 * K < int(vals["topk_row_bytes"][2])      # under 100 bytes on the wire
    V = int(vals["vocab_llama31"][0])
    assert V * 4 / m16.size > 1000                                                   # "over three orders of magnitude"


@pytest.mark.parametrize("ptype", [0, 1])
def test_wire_round_trip_and_layout(ptype):
    from oracle import wire
    qi, qp, qc = _wire_case(41)
    qc[3] = -1                                   # an invalid row travels as such
    qi[3], qp[3] = -1, 0
    m = wire.pack(qi, qp, qc, ptype)
    R, K = qi.shape
    N = int(np.maximum(qc, 0).sum())
    # layout, read back with plain struct arithmetic
    import struct
    magic, rows, k, pt, n = struct.unpack_from("<IIHHI", m.tobytes(), 0)
    assert (magic, rows, k, pt, n) == (0x31505350, R, K, ptype, N)
    counts = np.frombuffer(m.tobytes(), "<i2", R, 16)
    assert np.array_equal(counts, qc)
    ids = np.frombuffer(m.tobytes(), "<i4", N, 16 + (2 * R + 3) // 4 * 4)
    assert np.array_equal(ids, np.concatenate([qi[r, :max(qc[r], 0)] for r in range(R)]))
    ui, up, uc = wire.unpack(m, R, K)
    assert np.array_equal(ui, qi) and np.array_equal(uc, qc)
    if ptype == 0:
        assert np.array_equal(up, qp)
    else:
        assert np.array_equal(up, qp.astype(np.float16).astype(np.float32))
        np.testing.assert_allclose(up, qp, rtol=2 ** -11)
    # a message for another shape, a wrong magic and a truncated message are refused as a whole
    for bad in (wire.unpack(m, R + 1, K), wire.unpack(m, R, K + 1), wire.unpack(m[:-4], R, K),
                wire.unpack(np.concatenate([np.zeros(4, np.uint8), m[4:]]), R, K)):
        assert np.all(bad[2] == -1) and np.all(bad[0] == -1) and np.all(bad[1] == 0)


def test_throughput_model_closed_forms_and_limits():
    from oracle import wire
    # Eq. (5) closed form, its limits, and the golden values
    for a in (0.0, 0.3, 0.75, 0.9, 0.999):
        for g in (1, 4, 8):
            closed = (1 - a ** g) / (1 - a)
            assert abs(wire.expected_length(a, g) - closed) < 1e-12 * g
    assert abs(wire.expected_length(1.0 - 1e-12, 6) - 6) < 1e-9 and wire.expected_length(0.0, 6) == 1.0
    rows = [ln.split() for ln in open(os.path.join(GOLDEN, "expected_length.txt")) if ln[0] not in "#\n"]
    for alpha_s, gamma_s, el_s in rows:
        assert abs(wire.expected_length(float(alpha_s), int(gamma_s)) - float(el_s)) < 5e-4
    td, tr, tv = 40.0, 25.0, 10.0
    # Eq. (7) written out; Eq. (9) at alpha = 1 and alpha = 0
    assert abs(wire.throughput_sync(0.8, 5, td, tr, tv) - (1 - 0.8 ** 5) / (0.2 * (td + tr + tv))) < 1e-12
    assert wire.expected_time_async(1.0, 5, td, tr, tv) == max(td, tr + tv)
    assert wire.expected_time_async(0.0, 5, td, tr, tv) == td + tr + tv
    # Eq. (10): compute-bound, alpha -> 1; and the lower bound S -> 1 as alpha -> 0
    assert abs(wire.speedup(1.0 - 1e-9, 5, td, tr, tv) - (1 + (tr + tv) / td)) < 1e-6
    assert abs(wire.speedup(0.0, 5, td, tr, tv) - 1.0) < 1e-12
    # S is never below 1 and grows with alpha
    s = [wire.speedup(a, 5, td, tr, tv) for a in np.linspace(0, 0.999, 50)]
    assert min(s) >= 1.0 and all(b >= a - 1e-12 for a, b in zip(s, s[1:]))


# ---------------------------------------------------------------------------------------
# vocabulary-parallel verification (Sec. 4.1: the verifier model spans several GPUs, so the target
# logits arrive sharded along the vocabulary): slicing, exchanging chunk records and gathered
# entries, and deciding from them gives what the plain oracle gives on the whole vocabulary
# ---------------------------------------------------------------------------------------

@pytest.mark.parametrize("cuts", [[0, 5120], [0, 2048, 5120], [0, 1024, 3072, 4096, 5120 + 77]])
def test_sharded_verification_equals_the_plain_oracle(cuts):
    from oracle import vocab_parallel as vp
    rng = _rng(41)
    B, G, K = 6, 3, 24
    V = cuts[-1]
    base = rng.normal(0, 2.5, size=(B, G + 1, V)).astype(np.float32)
    dl = base[:, :G] + rng.normal(0, 0.7, size=(B, G, V)).astype(np.float32)
    tl = base.copy()
    tl[1, 1, 100:200] = -np.inf                       # a stretch of zero-weight entries
    T = rng.uniform(0.6, 1.3, size=B).astype(np.float32)
    ud, ua = rng.random((B, G), dtype=np.float32), rng.random((B, G), dtype=np.float32)
    ur = rng.random((B, 2), dtype=np.float32)
    qi, qp, qc, tok = oracle.compress(dl, T, top_k=0, top_p=0.9, k_max=K, u_draft=ud)
    tok[2, 0] = (int(qi[2, 0, 0]) + 7) % V            # a drafted token outside the stored support
    ref = oracle.verify(tl, T, tok, qi, qp, qc, ua, ur)
    slices = [np.ascontiguousarray(tl[:, :, a:b]) for a, b in zip(cuts[:-1], cuts[1:])]
    got = vp.verify_sharded(slices, cuts[:-1], T, tok, qi, qp, qc, ua, ur)
    assert np.array_equal(got["accept_len"], ref["accept_len"])
    assert np.array_equal(got["token"], ref["token"])
    assert got["borderline_count"] == ref["borderline_count"]
    np.testing.assert_allclose(got["p_draft"], ref["p_draft"], rtol=1e-12, atol=0)
    np.testing.assert_allclose(got["resid_mass"], ref["resid_mass"], rtol=1e-9, atol=1e-14)
    # the exchange really is needed: a rank that decided from its own slice alone would differ
    if len(slices) > 1:
        alone = vp.verify_sharded(slices[:1], cuts[:1], T, np.minimum(tok, cuts[1] - 1), np.minimum(qi, cuts[1] - 1),
                                  qp, qc, ua, ur)
        assert not np.array_equal(alone["token"], ref["token"])

