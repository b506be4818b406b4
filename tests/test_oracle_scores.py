"""Pins for the oracle's scoring functions against what the paper and the
mathematics fix: library routines, closed forms, brute force on tiny
vocabularies, invariants and limits."""
import math

import mpmath
import numpy as np
import pytest
from scipy.special import log_ndtr, logsumexp, ndtr, softmax
from scipy.stats import chi2 as chi2_dist

import oracle
import workloads as wl
from oracle import posterior

EPS = 1e-12


def _bits(x):
    return wl.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def _f64(bits):
    return wl.bf16_bits_to_f32(bits).astype(np.float64)


def _small(T, d, V, seed, w_scale=1.0):
    g = np.random.default_rng(seed)
    h = _bits(g.standard_normal((T, d)))
    W = _bits(g.standard_normal((V, d)) * w_scale / math.sqrt(d))
    return h, W


def _meta(T, seed=0x5EED5EED5EED5EED, start=1):
    return np.full(T, seed, dtype=np.uint64), np.arange(start, start + T, dtype=np.uint32)


# ---------------------------------------------------------------- logits
def test_logits_match_a_library_matmul():
    h, W = _small(7, 24, 13, 1)
    got = oracle.logits(h, W)
    want = _f64(h) @ _f64(W).T  # rows of W are vocabulary ids: a transposed operand would not even fit
    assert got.shape == (7, 13)
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-13)


def test_bf16_conversion_is_exact_and_rounds_to_nearest_even():
    x = np.array([1.0, -2.5, 0.1, 3.0e-5, 1.00390625, 1.01171875, 65280.0], dtype=np.float32)
    b = wl.f32_to_bf16_bits(x)
    back = wl.bf16_bits_to_f32(b)
    assert back[0] == 1.0 and back[1] == -2.5
    assert back[4] == 1.0  # 1 + 2^-8 is a tie between 1 and 1 + 2^-7: even mantissa wins
    assert back[5] == 1.015625  # 1 + 3*2^-8 ties to 1 + 2^-6 (even)
    assert np.all(np.abs(back - x) <= np.abs(x) * 2.0**-8)


# ------------------------------------------------ Gumbel-max sampler == softmax
@pytest.mark.parametrize("temperature", [1.0, 0.7])
def test_gumbel_max_sampler_draws_from_the_temperature_softmax(temperature):
    """The defining property of the Gumbel-max trick (Sec. "Gumbel-Max Trick"):
    over seeds, argmax_v l_v + Temp G_v is distributed as softmax(l/Temp).  A
    wrong sign in the Gumbel transform, noise not scaled by the temperature, or a
    noise stream that ignores the position all fail this."""
    V, d, N = 12, 16, 40_000
    h1, W = _small(1, d, V, 2, w_scale=2.0)
    h = np.repeat(h1, N, axis=0)
    seeds = np.array([wl.splitmix64(i // 50) for i in range(N)], dtype=np.uint64)
    positions = (np.arange(N) % 50 + 1).astype(np.uint32)
    sampled, _ = oracle.sample_gm(h, W, seeds, positions, temperature)
    p = softmax((_f64(h1) @ _f64(W).T)[0] / temperature)
    counts = np.bincount(sampled, minlength=V)
    stat = float(((counts - N * p) ** 2 / (N * p)).sum())
    assert stat < chi2_dist.ppf(1 - 1e-5, V - 1)
    # sanity: the test has power -- the wrong temperature is rejected
    q = softmax((_f64(h1) @ _f64(W).T)[0] / (temperature * 1.5))
    assert float(((counts - N * q) ** 2 / (N * q)).sum()) > chi2_dist.ppf(1 - 1e-5, V - 1)


def test_honest_gumbel_max_tokens_have_nonnegative_margin_at_every_sigma():
    """A token drawn by the sampler with the shared seed is the verifier's argmax:
    exact match, every A_i >= 0, hence pi >= 1/2 whatever sigma is."""
    T, d, V = 64, 32, 300
    h, W = _small(T, d, V, 3)
    seeds, positions = _meta(T)
    honest, runner = oracle.sample_gm(h, W, seeds, positions, 0.7)
    for sigma in (1.0, 0.05, 0.001):
        r = oracle.score_gm(h, W, honest, seeds, positions, 0.7, sigma, EPS)
        assert np.all(r.match == 1) and np.array_equal(r.argmax, honest)
        assert np.all(r.margin >= 0) and not np.any(np.signbit(r.margin))
        np.testing.assert_allclose(r.margin, r.top2_margin, rtol=0, atol=0)
        assert np.all(r.score >= math.log(0.5))
    # sigma -> 0 reduces to exact matching: honest -> ln(1 + eps), anything else -> ln(eps)
    r0 = oracle.score_gm(h, W, honest, seeds, positions, 0.7, 1e-9, EPS)
    np.testing.assert_allclose(r0.score, math.log1p(EPS), atol=1e-15)
    r1 = oracle.score_gm(h, W, runner, seeds, positions, 0.7, 1e-9, EPS)
    np.testing.assert_allclose(r1.score, math.log(EPS), atol=1e-12)
    assert np.all(r1.match == 0) and np.all(r1.margin <= 0)
    np.testing.assert_allclose(r1.margin, -r1.top2_margin, rtol=0, atol=0)


def test_margin_and_argmax_against_a_numpy_replay():
    T, d, V = 16, 32, 257
    h, W = _small(T, d, V, 4)
    seeds, positions = _meta(T, seed=0xFEEDFACECAFEBEEF, start=5)
    g = np.random.default_rng(5)
    tokens = g.integers(0, V, size=T).astype(np.int32)
    temperature = 0.9
    # every other row claims the verifier's own sample, so that both kinds of competitor occur:
    # the sample for a wrong claim, the runner-up for a right one
    honest, _ = oracle.sample_gm(h, W, seeds, positions, temperature)
    tokens[::2] = honest[::2]
    r = oracle.score_gm(h, W, tokens, seeds, positions, temperature, 0.3, EPS)
    logits = _f64(h) @ _f64(W).T
    assert np.all(r.margin[::2] > 0) and np.array_equal(r.margin[::2], r.top2_margin[::2])
    assert np.sum(r.margin[1::2] < 0) >= T // 2 - 2
    for i in range(T):
        G = oracle.gumbel_noise_row(int(seeds[i]), int(positions[i]), V)
        y = logits[i] + temperature * G
        order = np.argsort(-y, kind="stable")
        assert r.argmax[i] == order[0] and r.runner_up[i] == order[1]
        assert r.top2_margin[i] == pytest.approx(y[order[0]] - y[order[1]], abs=1e-12)
        assert r.top23_margin[i] == pytest.approx(y[order[1]] - y[order[2]], abs=1e-12)
        others = np.delete(y, tokens[i])
        assert r.margin[i] == pytest.approx(y[tokens[i]] - others.max(), abs=1e-12)
        assert r.y_claimed[i] == pytest.approx(y[tokens[i]], abs=1e-12)
        assert r.rank[i] == list(np.argsort(-logits[i], kind="stable")).index(tokens[i])  # no ties in this data
        assert r.score[i] == pytest.approx(
            math.log(ndtr(r.margin[i] / (0.3 * math.sqrt(2))) + EPS), abs=1e-12)
        assert r.lse[i] == pytest.approx(logsumexp(logits[i] / temperature), rel=1e-14)


# ------------------------------------------- closed form vs the algorithm itself
def test_closed_form_equals_the_sampling_loop_of_the_algorithm():
    """With one competitor and Gaussian noise the expectation in Alg. Token-DiFR
    is Phi(A / (sigma sqrt 2)); the literal M-sample loop must agree within its
    standard error, and so must Gauss-Hermite quadrature."""
    V, d = 40, 16
    h, W = _small(1, d, V, 6, w_scale=3.0)
    seeds, positions = _meta(1, seed=11, start=9)
    logits = (_f64(h) @ _f64(W).T)[0]
    G = oracle.gumbel_noise_row(11, 9, V)
    rng = np.random.default_rng(8)
    temperature = 1.0
    order = np.argsort(-(logits + temperature * G))
    for claimed in (int(order[0]), int(order[1]), int(order[3])):
        for sigma in (1.0, 0.25):
            r = oracle.score_gm(h, W, np.array([claimed], dtype=np.int32), seeds, positions, temperature, sigma, EPS)
            pi = math.exp(r.score[0]) - EPS
            M = 200_000
            mc = posterior.token_difr_monte_carlo(logits, G, temperature, claimed, 1, sigma,
                                                  sigma * rng.standard_normal(M))
            assert abs(mc - pi) < 4.5 * math.sqrt(max(pi * (1 - pi), 1e-6) / M) + 1e-9
            quad = posterior.token_difr_quadrature(logits, G, temperature, claimed, 1, sigma)
            assert quad == pytest.approx(pi, abs=1e-9)


def test_two_token_vocabulary_closed_form_is_the_exact_fixed_seed_posterior():
    """With |V| = 2 there is exactly one competitor, so the one-competitor score is
    the fixed-seed posterior itself: the probability, over independent N(0,sigma^2)
    perturbations of both logits, that the sampler with the noise held fixed returns
    the claimed token."""
    d = 8
    h, W = _small(1, d, 2, 9, w_scale=1.0)
    logits = (_f64(h) @ _f64(W).T)[0]
    rng = np.random.default_rng(10)
    for pos in (1, 2, 3):
        seeds, positions = _meta(1, seed=77, start=pos)
        G = oracle.gumbel_noise_row(77, pos, 2)
        for claimed in (0, 1):
            sigma = 0.8
            r = oracle.score_gm(h, W, np.array([claimed], dtype=np.int32), seeds, positions, 1.0, sigma, EPS)
            pi = math.exp(r.score[0]) - EPS
            n = 400_000
            brute = posterior.fixed_seed_posterior_mc(logits, G, 1.0, claimed, sigma, n, rng)
            assert abs(brute - pi) < 4.5 * math.sqrt(max(pi * (1 - pi), 1e-6) / n)
    # the two claims partition the outcomes
    a = oracle.score_gm(h, W, np.array([0], dtype=np.int32), seeds, positions, 1.0, 0.8, 0.0)
    b = oracle.score_gm(h, W, np.array([1], dtype=np.int32), seeds, positions, 1.0, 0.8, 0.0)
    assert math.exp(a.score[0]) + math.exp(b.score[0]) == pytest.approx(1.0, abs=1e-14)


def test_full_subset_quadrature_is_the_posterior_and_one_competitor_bounds_it():
    V, d = 6, 8
    h, W = _small(1, d, V, 12, w_scale=2.0)
    logits = (_f64(h) @ _f64(W).T)[0]
    G = oracle.gumbel_noise_row(5, 4, V)
    rng = np.random.default_rng(13)
    seeds, positions = _meta(1, seed=5, start=4)
    sigma = 0.7
    for claimed in range(V):
        full = posterior.token_difr_quadrature(logits, G, 1.0, claimed, V - 1, sigma)
        n = 300_000
        brute = posterior.fixed_seed_posterior_mc(logits, G, 1.0, claimed, sigma, n, rng)
        assert abs(brute - full) < 4.5 * math.sqrt(max(full * (1 - full), 1e-6) / n)
        r = oracle.score_gm(h, W, np.array([claimed], dtype=np.int32), seeds, positions, 1.0, sigma, 0.0)
        assert math.exp(r.score[0]) >= full - 1e-12  # dropping factors <= 1 can only raise the estimate


def test_score_tail_matches_log_ndtr():
    for A in (-3.0, -0.4, 0.0, 0.2, 5.0):
        for sigma in (1.0, 0.05):
            z = A / (sigma * math.sqrt(2))
            assert oracle.gm_pi(A, sigma) == pytest.approx(ndtr(z), rel=1e-13, abs=1e-300)
            if log_ndtr(z) > -25:
                assert oracle.gm_score(A, sigma, 0.0) == pytest.approx(log_ndtr(z), rel=1e-12, abs=1e-14)
    assert oracle.gm_score(-50.0, 0.05, EPS) == pytest.approx(math.log(EPS), abs=1e-12)  # the floor


# ----------------------------------------------------------------- invariance
def test_vocabulary_permutation_with_its_noise_leaves_the_score_unchanged():
    T, d, V = 12, 16, 97
    h, W = _small(T, d, V, 14)
    seeds, positions = _meta(T, seed=0x1122334455667788)
    g = np.random.default_rng(15)
    tokens = g.integers(0, V, size=T).astype(np.int32)
    base = oracle.score_gm(h, W, tokens, seeds, positions, 0.8, 0.2, EPS)
    perm = g.permutation(V)  # new id j holds old id perm[j]
    inv = np.argsort(perm)
    Wp = np.ascontiguousarray(W[perm])
    moved = oracle.score_gm(h, Wp, inv[tokens].astype(np.int32), seeds, positions, 0.8, 0.2, EPS,
                            noise_id=perm.astype(np.int32))
    np.testing.assert_allclose(moved.score, base.score, rtol=0, atol=1e-13)
    np.testing.assert_allclose(np.abs(moved.margin), np.abs(base.margin), rtol=0, atol=1e-13)
    np.testing.assert_allclose(moved.lse, base.lse, rtol=1e-14)
    assert np.array_equal(perm[moved.argmax], base.argmax)
    assert np.array_equal(moved.rank, base.rank)
    # without carrying the noise along, the replay changes
    plain = oracle.score_gm(h, Wp, inv[tokens].astype(np.int32), seeds, positions, 0.8, 0.2, EPS)
    assert not np.array_equal(perm[plain.argmax], base.argmax)


def test_rows_are_independent_and_keyed_by_seed_and_position():
    T, d, V = 10, 16, 64
    h, W = _small(T, d, V, 16)
    seeds, positions = _meta(T)
    tokens = np.arange(T, dtype=np.int32)
    full = oracle.score_gm(h, W, tokens, seeds, positions, 1.0, 0.5, EPS)
    order = np.random.default_rng(1).permutation(T)
    shuf = oracle.score_gm(np.ascontiguousarray(h[order]), W, tokens[order], seeds[order], positions[order],
                           1.0, 0.5, EPS)
    assert np.array_equal(shuf.score, full.score[order])
    assert np.array_equal(shuf.argmax, full.argmax[order])


# ------------------------------------------------------------ edge cases
def test_out_of_range_claim_is_maximally_suspicious():
    T, d, V = 4, 8, 32
    h, W = _small(T, d, V, 17)
    seeds, positions = _meta(T)
    tokens = np.array([-1, V, 3, 2**31 - 1], dtype=np.int32)
    r = oracle.score_gm(h, W, tokens, seeds, positions, 1.0, 0.5, EPS)
    for i in (0, 1, 3):
        assert r.score[i] == pytest.approx(math.log(EPS)) and r.margin[i] == -np.inf
        assert r.row_status[i] & 1 and r.match[i] == 0
    assert r.row_status[2] == 0
    ri = oracle.score_ipt(h, W, tokens, seeds, positions, 1.0, 0.5, EPS)
    for i in (0, 1, 3):
        assert ri.score[i] == pytest.approx(math.log(EPS)) and ri.row_status[i] & 1


def test_zero_temperature_is_greedy_decoding():
    T, d, V = 8, 16, 50
    h, W = _small(T, d, V, 18)
    seeds, positions = _meta(T)
    logits = _f64(h) @ _f64(W).T
    r = oracle.score_gm(h, W, logits.argmax(axis=1).astype(np.int32), seeds, positions, 0.0, 0.5, EPS)
    assert np.all(r.match == 1)
    srt = np.sort(logits, axis=1)
    np.testing.assert_allclose(r.margin, srt[:, -1] - srt[:, -2], atol=1e-13)


# ------------------------------------------------------------------- IPT
def test_ipt_score_against_a_brute_force_cdf_and_numerical_integration():
    """Alg. Token-IPT-DiFR on a tiny vocabulary, recomputed with 40-digit
    arithmetic: softmax, cumulative sums, and the Gaussian density integrated
    numerically over the claimed token's interval."""
    mpmath.mp.dps = 40
    T, d, V = 6, 8, 9
    h, W = _small(T, d, V, 19, w_scale=2.0)
    seeds, positions = _meta(T, seed=0x0F0E0D0C0B0A0908, start=3)
    tokens = np.array([0, 1, 4, 8, 7, 2], dtype=np.int32)
    temperature = 0.7
    logits = _f64(h) @ _f64(W).T
    for sigma in (1.0, 0.05):
        r = oracle.score_ipt(h, W, tokens, seeds, positions, temperature, sigma, EPS)
        for i in range(T):
            z = [mpmath.mpf(float(x)) / mpmath.mpf(temperature) for x in logits[i]]
            Z = sum(mpmath.exp(x) for x in z)
            p = [mpmath.exp(x) / Z for x in z]
            a = sum(p[: tokens[i]])
            b = a + p[tokens[i]]
            word = oracle.ro_word(int(seeds[i]), int(positions[i]), 1, 0)
            mu = mpmath.mpf(2 * word + 1) / 2**33
            dens = lambda x: mpmath.exp(-((x - mu) ** 2) / (2 * sigma**2)) / (sigma * mpmath.sqrt(2 * mpmath.pi))
            mass = mpmath.quad(dens, [a, b])
            assert r.u[i] == float(mu)
            assert r.cdf_lo[i] == pytest.approx(float(a), abs=1e-14)
            assert r.p_claimed[i] == pytest.approx(float(p[tokens[i]]), rel=1e-12)
            assert r.lse[i] == pytest.approx(float(mpmath.log(Z)), rel=1e-14)
            assert r.score[i] == pytest.approx(float(mpmath.log(mass + EPS)), abs=1e-9)


def test_ipt_masses_telescope_over_the_vocabulary():
    """Summed over every possible claim the interval masses give
    Phi((1-mu)/sigma) - Phi(-mu/sigma)."""
    d, V = 8, 11
    h1, W = _small(1, d, V, 20, w_scale=2.0)
    h = np.repeat(h1, V, axis=0)
    seeds = np.full(V, 99, dtype=np.uint64)
    positions = np.full(V, 6, dtype=np.uint32)
    for sigma in (0.3, 0.02):
        r = oracle.score_ipt(h, W, np.arange(V, dtype=np.int32), seeds, positions, 1.0, sigma, 0.0)
        mu = r.u[0]
        assert r.mass.sum() == pytest.approx(ndtr((1 - mu) / sigma) - ndtr(-mu / sigma), abs=1e-12)
        np.testing.assert_allclose(np.diff(r.cdf_lo), r.p_claimed[:-1], atol=1e-14)


def test_honest_ipt_tokens_contain_the_uniform_and_follow_the_softmax():
    """A token from the IPT sampler with the same uniform has a <= mu < b, so its
    mass is at least Phi(p/sigma) - 1/2 and tends to 1 as sigma -> 0; over seeds
    the sampler draws from the softmax (which fixes the direction of the CDF)."""
    V, d, N = 10, 16, 30_000
    h1, W = _small(1, d, V, 21, w_scale=2.0)
    h = np.repeat(h1, N, axis=0)
    seeds = np.array([wl.splitmix64(1000 + i // 40) for i in range(N)], dtype=np.uint64)
    positions = (np.arange(N) % 40 + 1).astype(np.uint32)
    temperature = 1.3
    tok = oracle.sample_ipt(h, W, seeds, positions, temperature)
    p = softmax((_f64(h1) @ _f64(W).T)[0] / temperature)
    counts = np.bincount(tok, minlength=V)
    assert float(((counts - N * p) ** 2 / (N * p)).sum()) < chi2_dist.ppf(1 - 1e-5, V - 1)
    sub = slice(0, 2000)
    r = oracle.score_ipt(h[sub], W, tok[sub], seeds[sub], positions[sub], temperature, 0.05, 0.0)
    assert np.all(r.cdf_lo <= r.u) and np.all(r.u < r.cdf_lo + r.p_claimed)
    assert np.all(r.mass >= ndtr(r.p_claimed / 0.05) - 0.5 - 1e-12)
    r0 = oracle.score_ipt(h[sub], W, tok[sub], seeds[sub], positions[sub], temperature, 1e-7, 0.0)
    inside = (r0.u - r0.cdf_lo > 1e-5) & (r0.cdf_lo + r0.p_claimed - r0.u > 1e-5)
    np.testing.assert_allclose(r0.mass[inside], 1.0, atol=1e-12)
    # the IPT uniform is itself uniform
    hist, _ = np.histogram(oracle.score_ipt(h, W, tok, seeds, positions, temperature, 1.0).u, bins=16, range=(0, 1))
    assert float(((hist - N / 16) ** 2 / (N / 16)).sum()) < chi2_dist.ppf(1 - 1e-5, 15)


def test_interval_mass_has_no_cancellation_in_either_tail():
    mpmath.mp.dps = 40
    for za, zb in ((6.0, 6.5), (-7.5, -7.0), (-0.3, 0.4), (0.0, 1e-9), (-9.0, 9.0)):
        want = mpmath.ncdf(zb) - mpmath.ncdf(za)
        assert oracle.normal_interval_mass(za, zb) == pytest.approx(float(want), rel=1e-9)


# ------------------------------------------------------------- detection
def test_detection_and_pooling_against_numpy():
    g = np.random.default_rng(22)
    T = 1000
    scores = g.normal(-2.0, 3.0, size=T)
    scores[17] = np.nan
    margins = g.normal(0.5, 1.0, size=T)
    margins[5] = 0.0
    margins[6] = -0.0
    offs = np.array([0, 100, 100, 613, 1000], dtype=np.int32)
    tau = -4.0
    flags, stats = oracle.detect(scores, tau, margins, offs)
    want_flags = (scores < tau) | np.isnan(scores)
    assert np.array_equal(flags.astype(bool), want_flags)
    for s in range(4):
        lo, hi = offs[s], offs[s + 1]
        assert stats["n_flagged"][s] == want_flags[lo:hi].sum()
        assert stats["n_match"][s] == np.sum(~np.signbit(margins[lo:hi]))
        if hi > lo:
            if np.isnan(scores[lo:hi]).any():
                assert math.isnan(stats["sum"][s])
            else:
                assert stats["sum"][s] == pytest.approx(scores[lo:hi].sum(), rel=1e-12)
            assert stats["min"][s] == np.nanmin(scores[lo:hi])
        else:
            assert stats["sum"][s] == 0.0 and stats["min"][s] == np.inf
    # equality with the threshold is safe
    f2, _ = oracle.detect(np.array([tau, np.nextafter(tau, -np.inf)]), tau)
    assert list(f2) == [0, 1]
    f3, st3 = oracle.detect(scores, tau, margins, None)
    assert st3["n_flagged"][0] == want_flags.sum()


def test_exact_ties_go_to_the_lowest_id():
    """Two identical rows of W give two identical logits; under greedy decoding (no noise) the lower id is the
    sample, the higher id the runner-up, and claiming the higher id is a mismatch by the tie-break alone:
    margin -0.0, not +0.0."""
    T, d, V = 6, 16, 40
    h, W = _small(T, d, V, 23)
    seeds, positions = _meta(T)
    logits = _f64(h) @ _f64(W).T
    top = logits.argmax(axis=1)
    W = W.copy()
    lo_id, hi_id, third = 7, 31, 19
    # row by row: ids 7 and 31 both get the W row of that row's largest logit
    for r in range(T):
        Wr = W.copy()
        Wr[lo_id] = W[top[r]]
        Wr[hi_id] = W[top[r]]
        if top[r] not in (lo_id, hi_id):
            Wr[top[r]] = 0  # the original holder steps back
        for claim, want_match, want_sign in ((lo_id, 1, False), (hi_id, 0, True)):
            res = oracle.score_gm(h[r : r + 1], Wr, np.array([claim], dtype=np.int32), seeds[r : r + 1],
                                  positions[r : r + 1], 0.0, 0.5, EPS)
            assert res.argmax[0] == lo_id and res.runner_up[0] == hi_id
            assert res.margin[0] == 0.0 and bool(np.signbit(res.margin[0])) == want_sign
            assert res.match[0] == want_match and res.top2_margin[0] == 0.0
        # a third identical row in between: it becomes the runner-up, and claiming it still loses to id 7
        Wr[third] = Wr[lo_id]
        res = oracle.score_gm(h[r : r + 1], Wr, np.array([third], dtype=np.int32), seeds[r : r + 1],
                              positions[r : r + 1], 0.0, 0.5, EPS)
        assert res.argmax[0] == lo_id and res.runner_up[0] == third and res.top23_margin[0] == 0.0
        assert res.margin[0] == 0.0 and np.signbit(res.margin[0]) and res.match[0] == 0
