"""Pins for the oracle's rejection sampler (Sec. 2.2 Eq. 1; Eq. 5; Eq. 6).

None of these re-types the oracle's formulas: they check exact counting statements,
closed forms, the distributional guarantee and degenerate cases.
"""
import math

import numpy as np
import pytest
from scipy import stats

import torch

from oracle import sampler

V = 16


def _dist(rng, v=V, conc=1.0):
    return rng.dirichlet(np.full(v, conc)).astype(np.float32)


def _u24(rng, shape):
    return rng.integers(0, 1 << 24, size=shape, dtype=np.int64).astype(np.uint32)


# ---- integer inverse CDF ---------------------------------------------------------------

def test_icdf_exhaustive_over_all_uniforms():
    """For V=16 every one of the 2^24 uniforms is drawn; the number that land on token v must be
    ceil(C_v 2^24 / W) - ceil(C_{v-1} 2^24 / W) with C the exact integer prefix sums (counting
    statement), hence within 2^-24 of w_v / W."""
    rng = np.random.default_rng(0)
    r = _dist(rng)
    r[3] = 0.0                      # a zero-mass token must never be drawn
    r[7] = -0.25                    # negative residual entries carry no mass
    toks = sampler.icdf_draw_many(r, np.arange(1 << 24, dtype=np.uint32))
    counts = np.bincount(toks, minlength=V)
    w = [int(math.floor(float(x) * 2.0 ** 44)) if x > 0 else 0 for x in r]   # exact in Python floats
    W = sum(w)
    c = 0
    for v in range(V):
        lo = -(-(c << 24) // W)
        c += w[v]
        hi = -(-(c << 24) // W)
        assert counts[v] == hi - lo
        assert abs(counts[v] / 2.0 ** 24 - w[v] / W) <= 2.0 ** -24
    assert counts[3] == 0 and counts[7] == 0
    assert np.all(np.diff(toks) >= 0)           # monotone in the uniform


def test_icdf_scalar_and_vector_forms_agree():
    """Big-integer product (scalar form) == split 64-bit product (vector form)."""
    rng = np.random.default_rng(1)
    for trial in range(20):
        r = _dist(rng, v=300, conc=0.3) * np.float32(rng.uniform(0.1, 1.0))
        us = _u24(rng, 200)
        us[:3] = [0, (1 << 24) - 1, 1]
        many = sampler.icdf_draw_many(r, us)
        for u, t in zip(us, many):
            assert sampler.icdf_draw(r, int(u))[0] == t


def test_icdf_extremes():
    r = np.array([0, 0, 0.5, 0, 0.25, 0], np.float32)
    assert sampler.icdf_draw(r, 0)[0] == 2                  # lowest index with mass
    assert sampler.icdf_draw(r, (1 << 24) - 1)[0] == 4      # u -> 1 lands on the last mass
    assert sampler.icdf_draw(np.zeros(5, np.float32), 5) == (-1, 0)
    one_hot = np.zeros(9, np.float32)
    one_hot[6] = 1.0
    assert all(sampler.icdf_draw(one_hot, u)[0] == 6 for u in (0, 1, 12345, (1 << 24) - 1))


def test_icdf_order_free_total():
    """W is an integer sum: any summation order gives the same total."""
    rng = np.random.default_rng(2)
    r = _dist(rng, v=5000, conc=0.2)
    w = sampler.integer_weights(r)
    perm = rng.permutation(len(w))
    assert int(w.sum(dtype=np.uint64)) == int(w[perm].sum(dtype=np.uint64)) == sum(int(x) for x in w)


# ---- accept rule -----------------------------------------------------------------------

def test_accept_rate_matches_eq5():
    """P(accept) over 10^6 seeded draws == sum_d min(p, q) = 1 - TV (Eq. 5), within 4 sigma."""
    rng = np.random.default_rng(3)
    N = 1_000_000
    p, q = _dist(rng), _dist(rng)
    d = sampler.icdf_draw_many(q, _u24(rng, N))[:, None]
    a, _ = sampler.decide_many(np.stack([p, p]), q[None], d, _u24(rng, (N, 2)))
    alpha = sampler.acceptance_probability(p, q)
    tv = 0.5 * np.abs(p.astype(np.float64) - q.astype(np.float64)).sum()
    assert abs(alpha - (1 - tv)) < 1e-6
    sigma = math.sqrt(alpha * (1 - alpha) / N)
    assert abs(a.mean() - alpha) < 4 * sigma


def test_identical_draft_and_target_always_accept():
    rng = np.random.default_rng(4)
    K, N = 3, 20000
    p = np.stack([_dist(rng) for _ in range(K + 1)])
    d = np.stack([sampler.icdf_draw_many(p[k], _u24(rng, N)) for k in range(K)], axis=1)
    us = _u24(rng, (N, K + 1))
    us[:100, :K] = (1 << 24) - 1                 # the least favourable uniforms too
    a, _ = sampler.decide_many(p, p[:K], d, us)
    assert np.all(a == K)
    for i in range(50):
        assert sampler.decide(p, p[:K], d[i], us[i])[0] == K


def test_draft_outside_target_support_is_always_rejected():
    """q one-hot on a token with p = 0: never accepted (even with u = 0), and the replacement is
    distributed as p (max(0, p - q) = p)."""
    rng = np.random.default_rng(5)
    N = 400_000
    p = _dist(rng)
    p[5] = 0.0
    p = (p / p.sum()).astype(np.float32)
    q = np.zeros(V, np.float32)
    q[5] = 1.0
    us = _u24(rng, (N, 2))
    us[:10, 0] = 0
    a, tok = sampler.decide_many(np.stack([p, p]), q[None], np.full((N, 1), 5), us)
    assert np.all(a == 0) and not np.any(tok == 5)
    keep = p > 0
    chi, pv = stats.chisquare(np.bincount(tok, minlength=V)[keep], N * p[keep] / p[keep].sum())
    assert pv > 1e-4


def test_scalar_and_vector_decisions_agree():
    rng = np.random.default_rng(6)
    K = 3
    p = np.stack([_dist(rng) for _ in range(K + 1)])
    q = np.stack([_dist(rng) for _ in range(K)])
    N = 3000
    d = np.stack([sampler.icdf_draw_many(q[k], _u24(rng, N)) for k in range(K)], axis=1)
    us = _u24(rng, (N, K + 1))
    a, tok = sampler.decide_many(p, q, d, us)
    for i in range(N):
        ai, ti, warn = sampler.decide(p, q, d[i], us[i])
        assert (ai, ti, warn) == (a[i], tok[i], 0)


# ---- exactness of the committed distribution ---------------------------------------------

def test_first_committed_token_follows_target_chi_square():
    """10^6 cycles, vocabulary 16: the first committed token (d_1 if accepted, else the
    replacement) is distributed as p_1 (Sec. 2.2: the committed sequence is distributed exactly
    as the target's)."""
    rng = np.random.default_rng(7)
    N, K = 1_000_000, 3
    p = np.stack([_dist(rng, conc=0.7) for _ in range(K + 1)])
    q = np.stack([_dist(rng, conc=0.7) for _ in range(K)])
    d = np.stack([sampler.icdf_draw_many(q[k], _u24(rng, N)) for k in range(K)], axis=1)
    a, tok = sampler.decide_many(p, q, d, _u24(rng, (N, K + 1)))
    first = np.where(a >= 1, d[:, 0], tok)
    chi, pv = stats.chisquare(np.bincount(first, minlength=V), N * p[0].astype(np.float64) / p[0].sum())
    assert pv > 1e-4, (chi, pv)
    # a broken rule is detected: committing the raw draft instead fails the same test
    chi_bad, pv_bad = stats.chisquare(np.bincount(d[:, 0], minlength=V), N * p[0].astype(np.float64) / p[0].sum())
    assert pv_bad < 1e-12
    # the token after a full acceptance is the bonus draw from p_{K+1}
    full = a == K
    chi2, pv2 = stats.chisquare(np.bincount(tok[full], minlength=V),
                                full.sum() * p[K].astype(np.float64) / p[K].sum())
    assert pv2 > 1e-4


def test_two_token_joint_follows_markov_target():
    """Order-1 Markov target p(.|prev) and draft q(.|prev), K = 2, cycles repeated until two tokens
    are committed: the joint of the first two committed tokens is p(x1|s) p(x2|x1) (64 cells)."""
    rng = np.random.default_rng(8)
    v = 8
    P = np.stack([_dist(rng, v) for _ in range(v)])
    Q = np.stack([_dist(rng, v) for _ in range(v)])
    start, N, K = 0, 120_000, 2
    counts = np.zeros((v, v), np.int64)

    def cycle(prev):
        d, q, p = [], [], []
        ctx = prev
        for k in range(K):
            q.append(Q[ctx])
            p.append(P[ctx])
            d.append(sampler.draw_token(Q[ctx], int(rng.integers(1 << 24)))[0])
            ctx = d[-1]
        p.append(P[ctx])
        a, t, _ = sampler.decide(np.array(p), np.array(q), d, rng.integers(0, 1 << 24, K + 1))
        return d[:a] + [t]

    for _ in range(N):
        out = cycle(start)
        if len(out) < 2:
            out += cycle(out[-1])
        counts[out[0], out[1]] += 1
    expect = N * (P[start][:, None].astype(np.float64) * P.astype(np.float64))
    chi, pv = stats.chisquare(counts.ravel(), expect.ravel() * (N / expect.sum()))
    assert pv > 1e-4, (chi, pv)


def test_expected_accepted_length_eq6():
    """Context-free p, q: mean accepted drafts over 10^6 cycles == sum_l prod_{i<=l} alpha_i."""
    rng = np.random.default_rng(9)
    N, K = 1_000_000, 3
    p = np.stack([_dist(rng) for _ in range(K + 1)])
    q = np.stack([(0.6 * p[k] + 0.4 * _dist(rng)).astype(np.float32) for k in range(K)])
    d = np.stack([sampler.icdf_draw_many(q[k], _u24(rng, N)) for k in range(K)], axis=1)
    a, _ = sampler.decide_many(p, q, d, _u24(rng, (N, K + 1)))
    alphas = [sampler.acceptance_probability(p[k], q[k]) for k in range(K)]
    expect = sampler.expected_accepted_length(alphas)
    # brute-force the expectation independently of the closed form
    brute = sum(l * (np.prod(alphas[:l]) * ((1 - alphas[l]) if l < K else 1.0)) for l in range(K + 1))
    assert abs(expect - brute) < 1e-12
    assert abs(a.mean() - expect) < 4 * a.std() / math.sqrt(N)
    assert a.min() >= 0 and a.max() <= K


def test_depth_zero_is_plain_sampling():
    rng = np.random.default_rng(10)
    p = _dist(rng)
    for u in _u24(rng, 200):
        a, t, warn = sampler.decide(p[None], np.zeros((0, V), np.float32), [], [u])
        assert a == 0 and t == sampler.draw_token(p, u)[0]


def test_zero_residual_falls_back_to_target():
    """p == q at the rejected position cannot happen (p >= q accepts), but an underflowing
    residual can: then the draw comes from p and a warning bit is set."""
    p = np.array([[0.5, 0.5, 0, 0], [0.25, 0.25, 0.25, 0.25]], np.float32)
    q = np.array([[0.5 + 2 ** -24, 0.5 - 2 ** -24, 0, 0]], np.float32)
    # token 0: p < q, u close to 1 rejects; residual p - q = +2^-24 on token 1 only (> 2^-44): normal
    a, t, warn = sampler.decide(p, q, [0], [(1 << 24) - 1, 0])
    assert (a, t, warn) == (0, 1, 0)
    tiny = np.float32(2.0 ** -60)
    p2 = np.array([[1 - 0.0, tiny, 0, 0], [1, 0, 0, 0]], np.float32)
    q2 = np.array([[0, 1.0, 0, 0]], np.float32)         # draft token 1 has p = 2^-60 < q
    a, t, warn = sampler.decide(p2, q2, [1], [(1 << 24) - 1, 77])
    assert a == 0 and t == 0 and warn == 0               # residual on token 0 is 1.0: fine
    p3 = np.array([[tiny, tiny, 0, 0], [1, 0, 0, 0]], np.float32)
    a, t, warn = sampler.decide(p3, np.array([[0, 0, 1.0, 0]], np.float32), [2], [5, 5])
    assert a == 0 and warn == (sampler.WARN_ZERO_RESIDUAL | sampler.WARN_ZERO_MASS) and t == 0


# ---- softmax and the synthetic acceptance recipe --------------------------------------------

def test_softmax_against_scipy_and_temperature():
    from scipy.special import softmax as sp_softmax
    rng = np.random.default_rng(11)
    x = rng.normal(0, 3, (5, 1000))
    for T in (1.0, 0.7, 2.0):
        np.testing.assert_allclose(sampler.softmax_probs(x, T), sp_softmax(x / T, axis=-1),
                                   rtol=1e-6, atol=1e-12)
    assert sampler.softmax_probs(x).dtype == np.float32
    np.testing.assert_allclose(sampler.softmax_probs(x + 1000.0), sampler.softmax_probs(x), rtol=1e-5)


def test_noisy_logit_acceptance_closed_form():
    """Draft logits = target + N(0, sigma) over a large flat vocabulary: alpha -> 2 Phi(-sigma/2)
    = erfc(sigma / (2 sqrt 2)).  sigma = 0.908 gives 0.65 (the sampler-only workload)."""
    rng = np.random.default_rng(12)
    Vbig = 151936
    for sigma in (0.6, 0.908, math.sqrt(2)):
        t = rng.standard_normal((4, Vbig))
        dr = t + sigma * rng.standard_normal((4, Vbig))
        al = np.mean([sampler.acceptance_probability(sampler.softmax_probs(t[i]),
                                                     sampler.softmax_probs(dr[i])) for i in range(4)])
        assert abs(al - math.erfc(sigma / (2 * math.sqrt(2)))) < 0.01
    assert abs(math.erfc(0.908 / (2 * math.sqrt(2))) - 0.65) < 2e-3


# ---- nucleus (top-p) truncation -----------------------------------------------------------------------

def _textbook_top_p(p, top_p):
    """Sort descending, keep a token while the mass before it is below top_p (exact rationals)."""
    from fractions import Fraction
    order = sorted(range(len(p)), key=lambda i: -p[i])
    total = sum(Fraction(float(x)) for x in p)
    keep, before = np.zeros(len(p), bool), Fraction(0)
    for i in order:
        if before < Fraction(float(np.float32(top_p))) * total:
            keep[i] = True
        before += Fraction(float(p[i]))
    return keep


def test_nucleus_equals_textbook_rule_without_ties():
    rng = np.random.default_rng(31)
    for trial in range(40):
        v = int(rng.integers(2, 60))
        p = _dist(rng, v, conc=float(rng.choice([0.2, 1.0, 5.0])))
        assert len(np.unique(p)) == v
        top_p = float(rng.uniform(0.05, 0.99))
        # 2^-44 quantisation can move a cut only if the mass before a token is within V * 2^-44 of it
        ref = _textbook_top_p(p, top_p)
        srt = np.sort(p.astype(np.float64))[::-1]
        margin = np.abs(np.concatenate([[0.0], np.cumsum(srt)[:-1]]) - np.float32(top_p) * srt.sum()).min()
        if margin > 1e-9:
            np.testing.assert_array_equal(sampler.nucleus_keep(p, top_p), ref)


def test_nucleus_against_library_sort_and_cumsum():
    rng = np.random.default_rng(32)
    p = _dist(rng, 500, conc=0.3)
    for top_p in (0.1, 0.5, 0.7, 0.9):
        t = torch.from_numpy(p.astype(np.float64))
        srt, idx = torch.sort(t, descending=True)
        before = torch.cumsum(srt, 0) - srt
        keep = torch.zeros(500, dtype=torch.bool)
        keep[idx[before < top_p * float(t.sum())]] = True
        np.testing.assert_array_equal(sampler.nucleus_keep(p, top_p), keep.numpy())


def test_nucleus_properties():
    rng = np.random.default_rng(33)
    p = _dist(rng, 200, conc=0.5)
    for top_p in (0.3, 0.7, 0.95):
        keep = sampler.nucleus_keep(p, top_p)
        kept = np.sort(p[keep].astype(np.float64))
        assert kept.sum() >= top_p * p.sum(dtype=np.float64) - 1e-9          # covers top_p of the mass
        assert kept.sum() - kept[0] < top_p * p.sum(dtype=np.float64)        # and is minimal
        assert p[keep].min() > p[~keep].max()                               # a prefix of the sorted order
        assert keep[np.argmax(p)]
        f = sampler.nucleus_filter(p, top_p)
        np.testing.assert_allclose(f.sum(dtype=np.float64), 1.0, atol=1e-6)
        np.testing.assert_allclose(f[keep], p[keep] / kept.sum(), rtol=1e-6)
        assert (f[~keep] == 0).all()
    assert sampler.nucleus_keep(p, 1e-6).sum() == 1                        # only the mode
    assert sampler.nucleus_keep(p, 1.0).all()                              # everything with mass
    np.testing.assert_array_equal(sampler.nucleus_filter(p, 1.0), p)
    # scale of the weights does not matter (unnormalised weights give the same set)
    np.testing.assert_array_equal(sampler.nucleus_keep(p * np.float32(0.25), 0.7), sampler.nucleus_keep(p, 0.7))
    with pytest.raises(ValueError):
        sampler.nucleus_keep(p, 0.0)


def test_nucleus_keeps_every_member_of_a_tie_at_the_cut():
    p = np.array([0.4, 0.2, 0.2, 0.1, 0.1], np.float32)
    np.testing.assert_array_equal(sampler.nucleus_keep(p, 0.5), [True, True, True, False, False])
    np.testing.assert_array_equal(sampler.nucleus_keep(p, 0.4), [True, False, False, False, False])
    np.testing.assert_array_equal(sampler.nucleus_keep(p, 0.41), [True, True, True, False, False])
    np.testing.assert_array_equal(sampler.nucleus_keep(p, 0.85), [True, True, True, True, True])
    z = np.array([0.5, 0.0, 0.5, 0.0], np.float32)                          # zero-mass tokens are never kept
    np.testing.assert_array_equal(sampler.nucleus_keep(z, 1.0), [True, False, True, False])


def test_cycle_with_truncated_target_follows_the_truncated_law():
    """Losslessness with top-p: the first committed token of a cycle is distributed as the truncated
    target, although the head's distribution is not truncated (chi-square, 200k cycles)."""
    from scipy import stats
    rng = np.random.default_rng(34)
    v = 24
    p = np.stack([_dist(rng, v, 0.6), _dist(rng, v, 0.6)])
    q = _dist(rng, v, 0.6)[None]
    pf = sampler.nucleus_filter(p, 0.7)
    assert 1 < (pf[0] > 0).sum() < v
    n = 200_000
    d = sampler.icdf_draw_many(q[0], _u24(rng, n))[:, None]
    a, tok = sampler.decide_many(pf, q, d, _u24(rng, (n, 2)))
    first = np.where(a >= 1, d[:, 0], tok)
    support = pf[0] > 0
    assert not np.isin(first, np.nonzero(~support)[0]).any()
    obs = np.bincount(first, minlength=v)[support]
    chi = stats.chisquare(obs, pf[0][support].astype(np.float64) / pf[0][support].sum(dtype=np.float64) * n)
    assert chi.pvalue > 1e-4, chi


def test_overlap_is_one_lipschitz_in_the_target_and_the_chain_bound_follows():
    """App. F: when the target moves from p to p' the overlap with a fixed head moves by at most TV(p, p'), and the
    expected accepted length of a depth-K chain by at most K(K+1)/2 times the largest such move."""
    rng = np.random.default_rng(21)
    for trial in range(200):
        K = int(rng.integers(1, 8))
        q = [_dist(rng) for _ in range(K)]
        p0 = [_dist(rng) for _ in range(K)]
        mix = rng.uniform(0, 0.3)
        p1 = [((1 - mix) * p0[k] + mix * _dist(rng)).astype(np.float32) for k in range(K)]
        a0 = np.array([sampler.acceptance_probability(p0[k], q[k]) for k in range(K)])
        a1 = np.array([sampler.acceptance_probability(p1[k], q[k]) for k in range(K)])
        tv = np.array([0.5 * np.abs(p0[k].astype(np.float64) - p1[k].astype(np.float64)).sum() for k in range(K)])
        assert (np.abs(a1 - a0) <= tv + 1e-6).all()
        gap = abs(sampler.expected_accepted_length(a1) - sampler.expected_accepted_length(a0))
        assert gap <= K * (K + 1) / 2 * tv.max() + 1e-6
