"""Pins of the verification checker against what the paper and the mathematics fix.

Each test would fail for a plausible mistake somewhere in oracle/verify.py: a dropped
positive part, p/q inverted, an open instead of closed inequality on the wrong side,
an off-by-one row for the residual or bonus token, a missing temperature, a wrong
inverse-CDF edge.
"""
import math

import numpy as np
import pytest

from conftest import golden_lines
from oracle import verify as ov


def _golden():
    g = {}
    for f in golden_lines("verify_worked_example.txt"):
        g[f[0]] = np.array([float(x) for x in f[1:]])
    return g


def _chi2_pvalue(obs, expected_prob, n):
    from scipy.stats import chi2
    exp = expected_prob * n
    keep = exp > 0
    assert obs[~keep].sum() == 0, "mass observed where the law has none"
    stat = ((obs[keep] - exp[keep]) ** 2 / exp[keep]).sum()
    return float(chi2.sf(stat, keep.sum() - 1))


def test_worked_three_token_example_exact():
    g = _golden()
    p, q = g["p"], g["q"]
    lp, lq = np.log(p), np.log(q)
    assert np.allclose(ov.softmax_row(lp, 1.0), p, atol=1e-15)
    assert abs(ov.acceptance_probability(p, q) - g["alpha"][0]) < 1e-15
    # residual distribution
    res = ov.positive_part(p - q)
    assert np.allclose(res / res.sum(), g["residual"], atol=1e-15)
    # thresholds: token x is accepted iff u <= ratio[x]
    for x in range(3):
        thr = g["ratio"][x]
        for u, want in [(thr - 1e-9, True), (thr + 1e-9, False)]:
            if u >= 1.0:
                continue
            r = ov.verify_sequence(np.stack([lp, lp]), np.stack([lq]), [x], 1, [u], 0.5, 1.0)
            assert (r.tau == 1) == want
    # exact law of the first emitted token by quadrature over (x~q, u_accept, u_resample):
    # thresholds 0.6 and 2/3 and every CDF edge of the residual fall on grid edges for N = 3000
    N = 3000
    us = (np.arange(N) + 0.5) / N
    law = np.zeros(3)
    for x in range(3):
        acc = np.array([ov.verify_sequence(np.stack([lp, lp]), np.stack([lq]), [x], 1, [u], 0.5, 1.0).tau
                        for u in us[::10]])
        # accepted fraction for this drafted token
        frac = acc.mean()
        assert abs(frac - min(1.0, p[x] / q[x])) < 1e-12
        law[x] += q[x] * frac
        # rejected: emitted token from the residual (does not depend on u_accept beyond rejection)
        if frac < 1.0:
            emitted = [ov.verify_sequence(np.stack([lp, lp]), np.stack([lq]), [x], 1, [0.999], ur, 1.0).token
                       for ur in us[::10]]
            hist = np.bincount(emitted, minlength=3) / len(emitted)
            law += q[x] * (1 - frac) * hist
    assert np.allclose(law, g["emitted"], atol=1e-12)


@pytest.mark.parametrize("V,gamma,seed", [(3, 1, 0), (5, 2, 1), (8, 3, 2)])
def test_emitted_tokens_follow_the_target_chi_square(V, gamma, seed):
    """Proposition 1: the output is distributed as canonical decoding from the target.
    Rows here do not depend on earlier tokens, so the exact joint law of one round is
      P(y = k+1, x_1..x_k = a_1..a_k, x_{k+1} = b)
        = prod_{j<=k} min(p_j(a_j), q_j(a_j)) * [p_k+1(b) - min(p,q)_k+1(b)]   for k < gamma
        = prod_{j<=gamma} min(p_j, q_j)(a_j) * p_bonus(b)                      for k = gamma.
    Checked: law of the first token (= p_0) and the law of (y, last token)."""
    rng = np.random.default_rng(seed)
    T = 0.8
    tl = rng.normal(0, 1.5, size=(gamma + 1, V))
    dl = tl[:gamma] + rng.normal(0, 0.8, size=(gamma, V))
    P = np.stack([ov.softmax_row(r, T) for r in tl])
    Q = np.stack([ov.softmax_row(r, T) for r in dl])
    n = 60000
    first = np.zeros(V)
    ylast = np.zeros((gamma + 1, V))
    for _ in range(n):
        toks = [rng.choice(V, p=Q[j]) for j in range(gamma)]        # drafting, independent sampler
        r = ov.verify_sequence(tl, dl, toks, gamma, rng.random(gamma), rng.random(), T)
        first[r.out_tokens[0]] += 1
        ylast[r.y - 1, r.out_tokens[-1]] += 1
    assert _chi2_pvalue(first, P[0], n) > 1e-4
    alpha = np.minimum(P[:gamma], Q).sum(axis=1)
    law = np.zeros((gamma + 1, V))
    for k in range(gamma):
        law[k] = np.prod(alpha[:k]) * (P[k] - np.minimum(P[k], Q[k]))
    law[gamma] = np.prod(alpha) * P[gamma]
    assert abs(law.sum() - 1.0) < 1e-12
    assert _chi2_pvalue(ylast.ravel(), law.ravel(), n) > 1e-4


def test_acceptance_rate_matches_closed_form():
    rng = np.random.default_rng(5)
    V, T = 16, 1.3
    tl = rng.normal(0, 2, size=(2, V))
    dl = tl[:1] + rng.normal(0, 1, size=(1, V))
    P, Q = ov.softmax_row(tl[0], T), ov.softmax_row(dl[0], T)
    alpha = ov.acceptance_probability(P, Q)
    n = 40000
    acc = 0
    for _ in range(n):
        x = rng.choice(V, p=Q)
        acc += ov.verify_sequence(tl, dl, [x], 1, [rng.random()], rng.random(), T).tau
    assert abs(acc / n - alpha) < 4 * math.sqrt(alpha * (1 - alpha) / n)


def test_accepted_length_is_truncated_geometric():
    g = _golden()
    alpha, L = float(g["tgd_alpha"][0]), int(g["tgd_L"][0])
    pmf = ov.truncated_geometric_pmf(alpha, L)
    assert np.allclose(pmf, g["tgd_pmf"], atol=1e-12) and abs(pmf.sum() - 1) < 1e-12
    mean = (np.arange(1, L + 2) * pmf).sum()
    assert abs(mean - g["tgd_mean"][0]) < 1e-12
    assert abs(mean - (1 - alpha ** (L + 1)) / (1 - alpha)) < 1e-12     # Appendix, proof of tightness
    # a (P, Q) pair with sum min(p, q) = 0.6, the same at every position
    p = np.array([0.7, 0.2, 0.1]); q = np.array([0.3, 0.6, 0.1])
    assert abs(ov.acceptance_probability(p, q) - alpha) < 1e-15
    tl = np.tile(np.log(p), (L + 1, 1)); dl = np.tile(np.log(q), (L, 1))
    rng = np.random.default_rng(11)
    n = 50000
    hist = np.zeros(L + 1)
    for _ in range(n):
        toks = rng.choice(3, p=q, size=L)
        hist[ov.verify_sequence(tl, dl, toks, L, rng.random(L), rng.random(), 1.0).y - 1] += 1
    assert _chi2_pvalue(hist, pmf, n) > 1e-4


def test_identical_models_accept_everything():
    rng = np.random.default_rng(3)
    tl = rng.normal(0, 3, size=(6, 50))
    for trial in range(50):
        toks = rng.integers(0, 50, size=5)
        r = ov.verify_sequence(tl, tl[:5].copy(), toks, 5, rng.random(5), rng.random(), 0.7)
        assert r.tau == 5 and r.y == 6 and r.out_tokens[:5] == list(toks)
        assert np.allclose(r.p_tok, r.q_tok)


def test_length_bounds_and_output_layout():
    rng = np.random.default_rng(4)
    for trial in range(200):
        gamma = int(rng.integers(0, 7))
        tl = rng.normal(0, 2, size=(gamma + 1, 12)); dl = rng.normal(0, 2, size=(gamma, 12))
        toks = rng.integers(0, 12, size=gamma)
        r = ov.verify_sequence(tl, dl, toks, gamma, rng.random(gamma), rng.random(), 1.0)
        assert 1 <= r.y <= gamma + 1 and r.y == r.tau + 1 == len(r.out_tokens)
        assert r.out_tokens[:r.tau] == list(toks[:r.tau])
        assert 0.0 <= r.cdf_lo < r.cdf_hi <= 1.0 + 1e-12


def test_temperature_is_applied_as_logits_over_T():
    row = np.array([1.0, 2.0, 4.0])
    want = np.exp(row / 0.5) / np.exp(row / 0.5).sum()
    assert np.allclose(ov.softmax_row(row, 0.5), want, atol=1e-15)
    # shifting a row does not change anything; scaling does
    assert np.allclose(ov.softmax_row(row + 100.0, 0.5), want, atol=1e-13)
    assert not np.allclose(ov.softmax_row(row, 1.0), want)


def test_inverse_cdf_against_brute_force_and_zero_mass():
    rng = np.random.default_rng(9)
    for trial in range(300):
        V = int(rng.integers(1, 40))
        mass = rng.random(V) * (rng.random(V) < 0.6)
        if mass.sum() == 0:
            mass[rng.integers(0, V)] = 1.0
        u = rng.random()
        v, lo, hi = ov.inverse_cdf(mass, u)
        run, want = 0.0, None
        for k in range(V):                         # smallest v with running sum > u * total
            run += mass[k]
            if run > u * mass.sum():
                want = k
                break
        assert v == want and mass[v] > 0 and lo <= u < hi
    # edges: u just below / at an interior edge (closed on the left: u == edge goes right)
    mass = np.array([0.25, 0.0, 0.25, 0.5])
    assert ov.inverse_cdf(mass, 0.25 - 1e-12)[0] == 0
    assert ov.inverse_cdf(mass, 0.25)[0] == 2
    assert ov.inverse_cdf(mass, 0.5)[0] == 3


def test_bonus_and_residual_use_the_right_rows():
    # row 0: p concentrated on token 0, q on token 1 -> drafting token 1 is rejected,
    # the residual is the point mass on token 0.  Row 1 (bonus) is a point mass on token 2.
    big = 40.0
    tl = np.array([[big, 0, 0, 0], [0, 0, big, 0]])
    dl = np.array([[0, big, 0, 0]])
    r = ov.verify_sequence(tl, dl, [1], 1, [0.5], 0.7, 1.0)
    assert r.tau == 0 and r.token == 0
    # drafting token 0 (q tiny, p ~ 1) is accepted, then the bonus comes from row 1
    r = ov.verify_sequence(tl, dl, [0], 1, [0.999], 0.7, 1.0)
    assert r.tau == 1 and r.token == 2 and r.out_tokens == [0, 2]
    # gamma = 0 is canonical decoding: one token from target row 0
    r = ov.verify_sequence(tl, None, [], 0, [], 0.3, 1.0)
    assert r.tau == 0 and r.y == 1 and r.token == 0


def test_residual_without_mass_falls_back_to_the_target_row():
    """Norm([P - Q]_+) needs a positive total (notation paragraph before Algorithm 6).  With identical
    models the accept test cannot reject, so the stop is forced: the residual at the stop row is then
    exactly zero, the step samples from that row's target distribution instead and says so."""
    rng = np.random.default_rng(31)
    for trial in range(100):
        V = int(rng.integers(2, 30))
        gamma = int(rng.integers(1, 5))
        tl = rng.normal(0, 2, size=(gamma + 1, V))
        toks = rng.integers(0, V, size=gamma)
        stop = int(rng.integers(0, gamma))
        u = rng.random()
        T = float(rng.choice([0.5, 1.0, 2.0]))
        r = ov.verify_sequence(tl, tl[:gamma].copy(), toks, gamma, rng.random(gamma), u, T, forced_tau=stop)
        assert r.used_fallback and r.tau == stop and r.y == stop + 1
        # the token of the stop row's own distribution for this uniform, by a written-out loop
        P = np.exp(tl[stop] / T - (tl[stop] / T).max())
        P /= P.sum()
        run, want = 0.0, None
        for v in range(V):
            run += P[v]
            if run > u * P.sum():
                want = v
                break
        assert r.token == want and r.out_tokens == list(toks[:stop]) + [want]
        # not the bonus row's token law: the rows differ, so the intervals do
        assert r.cdf_lo <= u < r.cdf_hi and abs((r.cdf_hi - r.cdf_lo) - P[want]) < 1e-12
    # a residual with mass anywhere never takes that branch
    r = ov.verify_sequence(np.array([[1.0, 0.0], [0.0, 0.0]]), np.array([[0.0, 1.0]]), [1], 1, [0.99], 0.5, 1.0)
    assert not r.used_fallback and r.tau == 0 and r.token == 0


def test_greedy_against_brute_force_with_ties():
    rng = np.random.default_rng(21)
    for trial in range(300):
        V, gamma = int(rng.integers(2, 9)), int(rng.integers(0, 5))
        tl = rng.integers(-2, 3, size=(gamma + 1, V)).astype(np.float64)   # many exact ties
        toks = rng.integers(0, V, size=gamma)
        r = ov.verify_sequence(tl, None, toks, gamma, np.zeros(gamma), 0.5, 0.0)
        tau = 0
        for j in range(gamma):
            best = max(range(V), key=lambda v: (tl[j, v], -v))             # highest logit, lowest index
            if toks[j] != best:
                break
            tau += 1
        best = max(range(V), key=lambda v: (tl[tau, v], -v))
        assert r.tau == tau and r.token == best and r.out_tokens == list(toks[:tau]) + [best]


def test_greedy_is_the_small_temperature_limit():
    rng = np.random.default_rng(22)
    agree = 0
    for trial in range(100):
        V, gamma = 10, 3
        tl = rng.normal(0, 3, size=(gamma + 1, V)); dl = tl[:gamma] + rng.normal(0, 1.0, size=(gamma, V))
        toks = dl.argmax(axis=1)                                           # greedy drafting
        g = ov.verify_sequence(tl, None, toks, gamma, np.zeros(gamma), 0.5, 0.0)
        s = ov.verify_sequence(tl, dl, toks, gamma, rng.random(gamma), rng.random(), 1e-3)
        agree += (g.out_tokens == s.out_tokens)
    assert agree >= 97


def test_draft_token_partitions_the_unit_interval_like_q():
    """x~ ~ Q by inverse CDF: the set of uniforms that map to token v is an interval of length Q(v),
    so on an equally spaced grid of N uniforms every token's count is within 1 of N * Q(v); tokens
    of zero mass never appear; temperature 0 gives the lowest arg-max."""
    rng = np.random.default_rng(5)
    row = rng.normal(0, 2, size=13)
    row[4] = -np.inf                                   # a token of zero mass
    for T in (1.0, 0.5):
        q = np.exp(row / T - np.max(row / T)); q /= q.sum()
        N = 200000
        us = (np.arange(N) + 0.5) / N
        toks = np.array([ov.draft_token(row, u, T)[0] for u in us[::40]])        # spot check of the call itself
        c = np.cumsum(q)
        assert (toks == np.searchsorted(c, us[::40], side="right")).all()
        counts = np.bincount(np.searchsorted(c, us, side="right"), minlength=13)
        assert np.abs(counts - N * q).max() <= 1.0 + 1e-9 and counts[4] == 0
        v, lo, hi = ov.draft_token(row, 0.37, T)
        assert lo <= 0.37 < hi and abs((hi - lo) - q[v]) < 1e-12
    tie = np.array([1.0, 3.0, 3.0, -2.0])
    assert ov.draft_token(tie, 0.9, 0.0)[0] == 1
