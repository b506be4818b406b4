"""Pins for the oracle's full Alg. Token-DiFR (top-k/top-p cutoff, B_i terms, s competitors)."""
import math

import numpy as np
import pytest
from scipy.special import ndtr

import oracle
import workloads as wl
from oracle import filtered, posterior


def _row(V, seed, scale=2.0):
    g = np.random.default_rng(seed)
    logits = scale * g.standard_normal(V)
    G = oracle.gumbel_noise_row(0xABCDEF12345 + seed, 3 + seed, V)
    return logits, G


def test_cutoff_on_hand_worked_examples():
    l = np.array([0.0, 3.0, 1.0, 2.0])  # softmax at Temp 1: 0.032, 0.644, 0.087, 0.237
    inf = math.inf
    assert filtered.filter_cutoff(l, 1.0, 0, 1.0) == -inf
    assert filtered.filter_cutoff(l, 1.0, 4, 1.0) == -inf          # top-k of the whole vocabulary filters nothing
    assert filtered.filter_cutoff(l, 1.0, 2, 1.0) == 2.0
    assert filtered.filter_cutoff(l, 1.0, 1, 1.0) == 3.0
    assert filtered.filter_cutoff(l, 1.0, 0, 0.6) == 3.0           # 0.644 >= 0.6 already
    assert filtered.filter_cutoff(l, 1.0, 0, 0.65) == 2.0          # 0.644 < 0.65 <= 0.881
    assert filtered.filter_cutoff(l, 1.0, 0, 0.9) == 1.0           # 0.881 < 0.9 <= 0.968
    assert filtered.filter_cutoff(l, 1.0, 0, 0.97) == 0.0
    assert filtered.filter_cutoff(l, 1.0, 3, 0.95) == 1.0          # renormalised over the top 3: 0.665, 0.910, 1
    assert filtered.filter_cutoff(l, 1.0, 3, 0.90) == 2.0
    # a lower temperature sharpens the distribution: the same top_p keeps fewer ids
    assert filtered.filter_cutoff(l, 0.5, 0, 0.65) == 3.0          # softmax(2 l): 0.867 first
    assert filtered.filter_cutoff(l, 0.0, 0, 0.5) == 3.0


@pytest.mark.parametrize("seed", [1, 2, 3])
def test_one_competitor_without_filter_is_the_closed_form(seed):
    logits, G = _row(50, seed)
    y = logits + 0.7 * G
    for claimed in (int(np.argmax(y)), int(np.argsort(-y)[1]), 7):
        for sigma in (0.05, 0.5, 2.0):
            c = posterior.active_subset(y, claimed, 1)[0]
            want = oracle.gm_pi(y[claimed] - y[c], sigma)
            got = filtered.token_difr_filtered(logits, G, 0.7, claimed, 1, sigma)
            assert got == pytest.approx(want, rel=1e-8, abs=1e-15)


def test_many_competitors_without_filter_match_gauss_hermite():
    logits, G = _row(40, 5)
    y = logits + G
    for claimed in (int(np.argmax(y)), int(np.argsort(-y)[2])):
        for s in (2, 4, 8, 39):
            want = posterior.token_difr_quadrature(logits, G, 1.0, claimed, s, 0.8)
            got = filtered.token_difr_filtered(logits, G, 1.0, claimed, s, 0.8)
            assert got == pytest.approx(want, rel=1e-7)


def test_filtered_expectation_equals_the_simulated_event():
    """With every other id in the active subset the expectation is exactly the probability that the claimed token
    survives the (fixed) cutoff and wins under the fixed noise."""
    V, sigma, temperature = 6, 0.7, 1.0
    logits = np.array([1.2, 0.9, 0.3, -0.2, 1.0, -1.5])
    G = oracle.gumbel_noise_row(99, 4, V)
    rng = np.random.default_rng(7)
    n = 1_000_000
    for top_k, top_p in ((3, 1.0), (0, 0.8), (4, 0.9)):
        cutoff = filtered.filter_cutoff(logits, temperature, top_k, top_p)
        assert np.isfinite(cutoff)
        for claimed in (0, 4, 2):
            want = filtered.model_posterior_mc(logits, G, temperature, claimed, sigma, cutoff, n, rng)
            got = filtered.token_difr_filtered(logits, G, temperature, claimed, V - 1, sigma, cutoff)
            se = math.sqrt(max(got * (1 - got), 1e-9) / n)
            assert abs(got - want) < 4.5 * se + 1e-6, (top_k, top_p, claimed, got, want)


def test_filtered_expectation_equals_the_algorithms_own_monte_carlo_loop():
    logits, G = _row(30, 9)
    cutoff = filtered.filter_cutoff(logits, 1.0, 5, 0.9)
    rng = np.random.default_rng(11)
    M = 400_000
    y = logits + G
    for claimed in (int(np.argmax(y)), int(np.argsort(-logits)[3])):
        for s in (1, 3):
            x = 0.6 * rng.standard_normal(M)
            mc = posterior.token_difr_monte_carlo(logits, G, 1.0, claimed, s, 0.6, x, cutoff)
            got = filtered.token_difr_filtered(logits, G, 1.0, claimed, s, 0.6, cutoff)
            assert abs(got - mc) < 4.5 * math.sqrt(0.25 / M)


def test_limits_of_the_filter_terms():
    logits, G = _row(30, 13)
    y = logits + G
    claimed = int(np.argmax(y))
    base = filtered.token_difr_filtered(logits, G, 1.0, claimed, 4, 0.5)
    # a cutoff far below every logit changes nothing; one far above the claimed logit leaves no mass
    assert filtered.token_difr_filtered(logits, G, 1.0, claimed, 4, 0.5, logits.min() - 50.0) == pytest.approx(base, rel=1e-9)
    assert filtered.token_difr_filtered(logits, G, 1.0, claimed, 4, 0.5, logits[claimed] + 20.0) < 1e-12
    # a competitor far below the cutoff is filtered out almost surely: it stops competing
    S = posterior.active_subset(y, claimed, 1)
    c = int(S[0])
    cut = logits[c] + 12.0
    if logits[claimed] > cut + 6.0:
        assert filtered.token_difr_filtered(logits, G, 1.0, claimed, 1, 0.5, cut) == pytest.approx(1.0, abs=1e-6)
    # more competitors can only lower the estimate; a filter that removes competitors can only raise it
    vals = [filtered.token_difr_filtered(logits, G, 1.0, claimed, s, 0.5) for s in (1, 2, 4, 8, 29)]
    assert all(a >= b - 1e-12 for a, b in zip(vals, vals[1:]))
    runner = int(np.argsort(-y)[1])
    lo_cut = filtered.filter_cutoff(logits, 1.0, 3, 1.0)
    if logits[runner] > lo_cut + 3.0:
        f = filtered.token_difr_filtered(logits, G, 1.0, runner, 4, 0.5, lo_cut)
        u = filtered.token_difr_filtered(logits, G, 1.0, runner, 4, 0.5)
        assert f >= u - 1e-9


def test_score_rows_wrap_the_pieces():
    g = np.random.default_rng(3)
    T, d, V = 4, 16, 30
    h = wl.f32_to_bf16_bits(g.standard_normal((T, d)).astype(np.float32))
    W = wl.f32_to_bf16_bits((g.standard_normal((V, d)) / 4).astype(np.float32))
    seeds = np.full(T, 77, dtype=np.uint64)
    positions = np.arange(1, T + 1, dtype=np.uint32)
    tokens = np.array([3, 5, V + 2, 0], dtype=np.int32)
    score, pi, cut = filtered.score_gm_filtered(h, W, tokens, seeds, positions, 1.0, 0.3, 1e-12, 0, 1.0, 1)
    ref = oracle.score_gm(h, W, tokens, seeds, positions, 1.0, 0.3, 1e-12)
    np.testing.assert_allclose(score, ref.score, rtol=0, atol=1e-7)  # s = 1, no filter: the shipped estimator
    assert score[2] == math.log(1e-12) and np.all(cut == -math.inf)
    score_f, _, cut_f = filtered.score_gm_filtered(h, W, tokens, seeds, positions, 1.0, 0.3, 1e-12, 5, 0.9, 3)
    L = oracle.logits(h, W)
    assert np.all(cut_f >= np.sort(L, axis=1)[:, -5]) and np.all(np.isfinite(score_f))


# ------------------------------------------------------------- Token-IPT-DiFR under the filter
def test_filtered_distribution_on_a_hand_worked_example():
    l = np.array([0.0, 3.0, 1.0, 2.0])
    p = filtered.filtered_probs(l, 1.0, 3, 0.90)      # top 3 = ids 1, 3, 2; nucleus 0.9 keeps ids 1 and 3
    e3, e2 = math.exp(3.0), math.exp(2.0)
    np.testing.assert_allclose(p, [0.0, e3 / (e3 + e2), 0.0, e2 / (e3 + e2)], rtol=1e-14)
    assert filtered.filter_kept(l, 1.0, 0, 1.0).tolist() == [1, 3, 2, 0]
    full = filtered.filtered_probs(l, 1.0, 0, 1.0)
    np.testing.assert_allclose(full, np.exp(l) / np.exp(l).sum(), rtol=1e-14)
    # the cutoff is the smallest kept logit
    for k, pp in ((3, 0.9), (2, 1.0), (0, 0.65)):
        kept = filtered.filter_kept(l, 1.0, k, pp)
        assert filtered.filter_cutoff(l, 1.0, k, pp) == l[kept].min()


def test_ipt_score_without_filter_is_the_plain_one_and_with_filter_obeys_the_identities():
    g = np.random.default_rng(21)
    T, d, V = 40, 16, 60
    h = wl.f32_to_bf16_bits(g.standard_normal((T, d)).astype(np.float32))
    W = wl.f32_to_bf16_bits((2.0 * g.standard_normal((V, d)) / 4).astype(np.float32))
    seeds = g.integers(1, 2**62, size=T).astype(np.uint64)
    positions = np.arange(1, T + 1, dtype=np.uint32)
    tokens = g.integers(0, V, size=T).astype(np.int32)
    plain = oracle.score_ipt(h, W, tokens, seeds, positions, 0.8, 0.1, 1e-12)
    s0, pt0, a0, mu0, cut0 = filtered.score_ipt_filtered(h, W, tokens, seeds, positions, 0.8, 0.1, 1e-12, 0, 1.0)
    np.testing.assert_allclose(s0, plain.score, rtol=0, atol=1e-9)
    np.testing.assert_allclose(a0, plain.cdf_lo, rtol=0, atol=1e-12)
    np.testing.assert_allclose(mu0, plain.u, rtol=0, atol=0)
    assert np.all(np.isneginf(cut0))

    L = oracle.logits(h, W)
    sigma = 0.07
    for top_k, top_p in ((8, 1.0), (12, 0.9)):
        # honest claims of the filtered sampler contain mu in their CDF interval
        honest = np.array([filtered.ipt_sample_filtered(L[r], 0.8, top_k, top_p, mu0[r]) for r in range(T)], dtype=np.int32)
        s, pt, a, mu, cut = filtered.score_ipt_filtered(h, W, honest, seeds, positions, 0.8, sigma, 1e-12, top_k, top_p)
        assert np.all(a <= mu) and np.all(mu < a + pt)
        assert np.all(L[np.arange(T), honest] >= cut)                      # a sampled id survived the filter
        assert np.all(s >= np.log(ndtr(pt / sigma) - 0.5 + 1e-12) - 1e-9)   # mu inside [a, b): at worst at an end
        # an id the filter removed has probability zero: floor score
        removed = np.array([int(np.argmin(L[r])) for r in range(T)], dtype=np.int32)
        sr, ptr, _, _, _ = filtered.score_ipt_filtered(h, W, removed, seeds, positions, 0.8, sigma, 1e-12, top_k, top_p)
        assert np.all(ptr == 0.0) and np.allclose(sr, math.log(1e-12))
        # telescoping: the masses of all claims add up to the Gaussian mass of [0, 1]
        r = 3
        total = 0.0
        for t in range(V):
            st, _, _, _, _ = filtered.score_ipt_filtered(h[r:r + 1], W, np.array([t], dtype=np.int32), seeds[r:r + 1],
                                                         positions[r:r + 1], 0.8, sigma, 1e-300, top_k, top_p)
            total += math.exp(st[0])
        want = oracle.normal_interval_mass((0.0 - mu0[r]) / sigma, (1.0 - mu0[r]) / sigma)
        assert total == pytest.approx(want, rel=1e-9)


def test_min_p_on_hand_worked_examples():
    """min-p keeps the ids whose probability is at least min_p times the largest (Sec. "Sampling From Large
    Language Models"): worked through on probabilities 1/2, 1/4, 1/8, 1/16, 1/16."""
    probs = np.array([0.5, 0.25, 0.125, 0.0625, 0.0625])
    l = np.log(probs) + 3.0  # any common shift
    # min_p 0.2 at Temp 1: the bar is 0.1 -> ids 0, 1, 2 survive; a logit survives iff it reaches ln(0.1) + 3
    assert filtered.filter_cutoff(l, 1.0, 0, 1.0, 0.2) == pytest.approx(math.log(0.1) + 3.0, rel=1e-15)
    assert sorted(filtered.filter_kept(l, 1.0, 0, 1.0, 0.2).tolist()) == [0, 1, 2]
    np.testing.assert_allclose(filtered.filtered_probs(l, 1.0, 0, 1.0, 0.2), [4 / 7, 2 / 7, 1 / 7, 0, 0], rtol=1e-14)
    # exactly on the bar (min_p 0.25: the bar is 1/8) the id survives
    assert sorted(filtered.filter_kept(l, 1.0, 0, 1.0, 0.25).tolist()) == [0, 1, 2]
    # Temp 2 flattens the distribution (p ~ sqrt): sqrt(1/16) / sqrt(1/2) = 0.354 >= 0.2, everything survives
    assert sorted(filtered.filter_kept(l, 2.0, 0, 1.0, 0.2).tolist()) == [0, 1, 2, 3, 4]
    assert filtered.filter_cutoff(l, 2.0, 0, 1.0, 0.2) == pytest.approx(math.log(0.5) + 3.0 + 2.0 * math.log(0.2))
    # no min-p: nothing changes; min_p 1 keeps the largest only; greedy decoding likewise
    assert filtered.filter_cutoff(l, 1.0, 0, 1.0, 0.0) == -math.inf
    assert filtered.filter_kept(l, 1.0, 0, 1.0, 1.0).tolist() == [0]
    assert filtered.filter_kept(l, 0.0, 0, 1.0, 0.3).tolist() == [0]
    # with a top-k in front the stricter of the two decides
    assert filtered.filter_cutoff(l, 1.0, 2, 1.0, 0.2) == l[1]                       # top-2 is stricter
    assert filtered.filter_cutoff(l, 1.0, 4, 1.0, 0.2) == pytest.approx(math.log(0.1) + 3.0)  # min-p is stricter
    assert sorted(filtered.filter_kept(l, 1.0, 4, 1.0, 0.2).tolist()) == [0, 1, 2]
    # the IPT sampler on the min-p distribution: cumulative 4/7, 6/7, 1
    assert filtered.ipt_sample_filtered(l, 1.0, 0, 1.0, 0.5, 0.2) == 0
    assert filtered.ipt_sample_filtered(l, 1.0, 0, 1.0, 0.6, 0.2) == 1
    assert filtered.ipt_sample_filtered(l, 1.0, 0, 1.0, 0.9, 0.2) == 2


def test_min_p_cutoff_is_the_survival_threshold_of_the_simulated_event():
    """With the min-p bound as the cutoff the expectation still equals the literal simulation of the event
    (every id a competitor; an id takes part iff its perturbed logit reaches the fixed bound)."""
    logits, G = _row(12, 9, scale=1.5)
    cutoff = filtered.filter_cutoff(logits, 1.0, 0, 1.0, 0.3)
    assert np.sum(logits >= cutoff) < 12  # the filter bites
    claimed = int(np.argmax(logits + G))
    want = filtered.model_posterior_mc(logits, G, 1.0, claimed, 0.6, cutoff, 400_000, np.random.default_rng(5))
    got = filtered.token_difr_filtered(logits, G, 1.0, claimed, 11, 0.6, cutoff)
    assert got == pytest.approx(want, abs=4 * math.sqrt(want * (1 - want) / 400_000) + 1e-4)
