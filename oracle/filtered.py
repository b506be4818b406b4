"""Alg. Token-DiFR in full: top-k / top-p cutoff, the B_i terms and an active
subset of s competitors -- TEST INFRASTRUCTURE, plain numpy / scipy.

    pi = E_{x ~ N(0, sigma^2)} [ 1{l_t* + x > cutoff} * prod_{i in S} Phi(max(x + A_i, B_i) / sigma) ]

with S the top-s ids by y = l + Temp*G (the claimed token left out),
A_i = y_t* - y_i, B_i = cutoff - l_i, and `cutoff` the smallest logit that
survives the sampling filter (the reading of the algorithm's garbled definition
of its cutoff): keep the top_k largest logits, then, among those, the shortest prefix in
descending order whose renormalised temperature-softmax mass reaches top_p.  A min-p
filter (Sec. "Sampling From Large Language Models" names it beside top-k and top-p;
the algorithm does not) keeps the ids whose probability is at least min_p times the
largest one, i.e. l >= l_max + Temp ln(min_p): that bound is itself the value a logit
has to reach to survive, so it enters the cutoff as max(cutoff of top-k/top-p, bound).
The expectation is evaluated by adaptive quadrature (a library routine) split at
the kinks of the integrand; the algorithm's own Monte-Carlo loop is in
`posterior.token_difr_monte_carlo`.
"""
from __future__ import annotations

import math

import numpy as np
from scipy.integrate import quad
from scipy.special import log_ndtr

from . import posterior


def min_p_bound(logits: np.ndarray, temperature: float, min_p: float) -> float:
    """The logit an id must reach to survive min-p: p_v >= min_p * p_max  <=>  l_v >= l_max + Temp ln(min_p).
    -inf when min_p is 0 (no filter); under greedy decoding (Temp = 0) only the largest logit survives."""
    if not min_p > 0.0:
        return -math.inf
    top = float(np.max(np.asarray(logits, dtype=np.float64)))
    return top + temperature * math.log(min_p) if temperature > 0.0 else top


def filter_cutoff(logits: np.ndarray, temperature: float, top_k: int, top_p: float, min_p: float = 0.0) -> float:
    """The value a logit must reach to survive top-k, then top-p, then min-p: the smallest logit the first two
    keep, or the min-p bound where that is higher (-inf when nothing is set)."""
    logits = np.asarray(logits, dtype=np.float64)
    V = logits.shape[0]
    k_on = 0 < top_k < V
    p_on = top_p < 1.0
    bound = min_p_bound(logits, temperature, min_p)
    if not k_on and not p_on:
        return bound
    order = np.argsort(-logits, kind="stable")  # descending, ties: lowest id first
    kept = order[:top_k] if k_on else order
    if p_on:
        if temperature > 0.0:
            z = logits[kept] / temperature
            p = np.exp(z - z.max())
            c = np.cumsum(p) / p.sum()
            n = int(np.searchsorted(c, top_p, side="left")) + 1  # first prefix whose mass is >= top_p
        else:
            n = 1  # a greedy sampler's nucleus is the largest logit
        kept = kept[: min(n, len(kept))]
    return max(float(logits[kept[-1]]), bound)


def token_difr_filtered(logits, gumbel, temperature, claimed, s, sigma, cutoff=-math.inf) -> float:
    """The expectation above, by adaptive quadrature."""
    logits = np.asarray(logits, dtype=np.float64)
    gumbel = np.asarray(gumbel, dtype=np.float64)
    y = logits + temperature * gumbel
    S = posterior.active_subset(y, claimed, s)
    A = posterior.margins(logits, gumbel, temperature, claimed, S)
    B = cutoff - logits[S]

    def integrand(x):
        t = np.maximum(x + A, B) / sigma
        return math.exp(-0.5 * (x / sigma) ** 2 + float(np.sum(log_ndtr(t)))) / (sigma * math.sqrt(2.0 * math.pi))

    # The expectation runs over the whole real line; below cutoff - l_claimed the claimed token is filtered out
    # and the integrand is zero.  Outside +-38 sigma (and 38 sigma past the largest -A) the weight of
    # x ~ N(0, sigma^2) is below 1e-313, the smallest magnitudes fp64 still represents.
    lo = max(cutoff - logits[claimed], -38.0 * sigma)
    hi = max(38.0 * sigma, float(np.max(-A, initial=0.0)) + 38.0 * sigma)
    if lo >= hi:
        return 0.0
    kinks = [float(b - a) for a, b in zip(A, B) if np.isfinite(b) and lo < b - a < hi]
    # break the range where the integrand peaks as well: the peak is narrow (about sigma) in a wide range
    grid = np.linspace(lo, hi, 6001)
    peak = float(grid[int(np.argmax([integrand(x) for x in grid]))])
    pts = sorted(set(kinks + [p for p in (peak - sigma, peak, peak + sigma) if lo < p < hi]))
    val, _ = quad(integrand, lo, hi, points=pts or None, epsabs=1e-18, epsrel=1e-11, limit=400)
    return float(min(max(val, 0.0), 1.0))


def model_posterior_mc(logits, gumbel, temperature, claimed, sigma, cutoff, n_draws, rng) -> float:
    """The event the expectation measures, simulated literally with every id a competitor: each logit gets an
    independent N(0, sigma^2) perturbation; an id takes part iff its perturbed logit exceeds the (fixed) cutoff;
    the claimed token comes out iff it takes part and beats every other participant under the fixed noise."""
    logits = np.asarray(logits, dtype=np.float64)
    gumbel = np.asarray(gumbel, dtype=np.float64)
    V = logits.shape[0]
    hits = done = 0
    while done < n_draws:
        n = min(200_000, n_draws - done)
        pert = logits[None, :] + sigma * rng.standard_normal((n, V))
        alive = pert > cutoff
        yy = np.where(alive, pert + temperature * gumbel[None, :], -np.inf)
        others = np.delete(yy, claimed, axis=1).max(axis=1)
        hits += int(np.sum(alive[:, claimed] & (yy[:, claimed] > others)))
        done += n
    return hits / n_draws


def score_gm_filtered(h_bits, W_bits, tokens, seeds, positions, temperature, sigma, eps=1e-12, top_k=0, top_p=1.0,
                      s=1, min_p=0.0):
    """Per row: (score = ln(pi + eps), pi, cutoff).  Out-of-range claims score ln(eps)."""
    from . import gumbel_noise_row, logits as all_logits

    L = all_logits(h_bits, W_bits)
    T, V = L.shape
    score = np.empty(T)
    pi = np.zeros(T)
    cut = np.empty(T)
    for r in range(T):
        cut[r] = filter_cutoff(L[r], temperature, top_k, top_p, min_p)
        t = int(tokens[r])
        if 0 <= t < V:
            G = gumbel_noise_row(int(seeds[r]), int(positions[r]), V)
            pi[r] = token_difr_filtered(L[r], G, temperature, t, s, sigma, cut[r])
        score[r] = math.log(pi[r] + eps)
    return score, pi, cut


# ---------------------------------------------------------------- Token-IPT-DiFR under the sampling filter
def filter_kept(logits: np.ndarray, temperature: float, top_k: int, top_p: float, min_p: float = 0.0) -> np.ndarray:
    """Ids that survive top-k, then top-p, then min-p (all ids when none is set), in descending logit order."""
    logits = np.asarray(logits, dtype=np.float64)
    V = logits.shape[0]
    order = np.argsort(-logits, kind="stable")
    kept = order[:top_k] if 0 < top_k < V else order
    if top_p < 1.0:
        if temperature > 0.0:
            z = logits[kept] / temperature
            p = np.exp(z - z.max())
            c = np.cumsum(p) / p.sum()
            n = int(np.searchsorted(c, top_p, side="left")) + 1
        else:
            n = 1
        kept = kept[: min(n, len(kept))]
    return kept[logits[kept] >= min_p_bound(logits, temperature, min_p)]


def filtered_probs(logits: np.ndarray, temperature: float, top_k: int, top_p: float, min_p: float = 0.0) -> np.ndarray:
    """The distribution the filtered sampler draws from: softmax(l / Temp) restricted to the surviving ids and
    renormalised (Alg. Token-IPT-DiFR: the same temperature / top-k / nucleus policy as generation)."""
    logits = np.asarray(logits, dtype=np.float64)
    kept = filter_kept(logits, temperature, top_k, top_p, min_p)
    p = np.zeros_like(logits)
    z = logits[kept] / temperature
    e = np.exp(z - z.max())
    p[kept] = e / e.sum()
    return p


def ipt_sample_filtered(logits, temperature, top_k, top_p, mu: float, min_p: float = 0.0) -> int:
    """Alg. IPT Sampler on the filtered distribution: min{v : C_v > mu}."""
    p = filtered_probs(logits, temperature, top_k, top_p, min_p)
    hit = np.nonzero(np.cumsum(p) > mu)[0]
    return int(hit[0]) if len(hit) else int(np.nonzero(p)[0][-1])


def score_ipt_filtered(h_bits, W_bits, tokens, seeds, positions, temperature, sigma, eps=1e-12, top_k=0, top_p=1.0,
                       min_p=0.0):
    """Per row: (score, p_claimed, cdf_lo, mu, cutoff) of Token-IPT-DiFR with the filtered distribution."""
    from . import ipt_uniform, logits as all_logits, normal_interval_mass

    L = all_logits(h_bits, W_bits)
    T, V = L.shape
    score = np.empty(T)
    pt = np.full(T, np.nan)
    a = np.full(T, np.nan)
    mu = np.empty(T)
    cut = np.empty(T)
    for r in range(T):
        mu[r] = ipt_uniform(int(seeds[r]), int(positions[r]))
        cut[r] = filter_cutoff(L[r], temperature, top_k, top_p, min_p)
        t = int(tokens[r])
        mass = 0.0
        if 0 <= t < V:
            p = filtered_probs(L[r], temperature, top_k, top_p, min_p)
            a[r] = float(np.sum(p[:t]))
            pt[r] = float(p[t])
            mass = normal_interval_mass((a[r] - mu[r]) / sigma, (a[r] + pt[r] - mu[r]) / sigma)
        score[r] = math.log(mass + eps)
    return score, pt, a, mu, cut
