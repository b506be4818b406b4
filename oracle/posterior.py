"""Token-DiFR beyond one competitor, in plain numpy -- TEST INFRASTRUCTURE.

The scoring path uses Alg. Token-DiFR with an active subset of one competitor
and no top-k/top-p filter, where the expectation has a closed form.  This module
states the algorithm in its general form so that the closed form can be checked:

* `token_difr_monte_carlo`  the sample mean the algorithm returns, over given noise draws;
* `token_difr_quadrature`   the same expectation by Gauss-Hermite quadrature;
* `fixed_seed_posterior_mc` the definition it estimates (Sec. "Fixed-Seed
  Posterior Distribution"): perturb every logit, re-run the Gumbel-max sampler
  with the noise held fixed, count how often the claimed token comes out.
"""
from __future__ import annotations

import numpy as np
from scipy.special import ndtr


def active_subset(y: np.ndarray, claimed: int, s: int) -> np.ndarray:
    """Top-s ids ranked by y = l + Temp*G, the claimed token itself left out."""
    order = np.argsort(-y, kind="stable")
    order = order[order != claimed]
    return order[:s]


def margins(logits: np.ndarray, gumbel: np.ndarray, temperature: float, claimed: int, subset: np.ndarray):
    """A_i = l_t* - l_i + Temp (G_t* - G_i) for i in the active subset."""
    return logits[claimed] - logits[subset] + temperature * (gumbel[claimed] - gumbel[subset])


def token_difr_monte_carlo(logits, gumbel, temperature, claimed, s, sigma, noise_samples, cutoff=-np.inf):
    """The sample mean that Alg. Token-DiFR returns, written as the estimator it is:

        pi_hat = mean_j  1{l_t* + x_j > cutoff} * prod_{i in S} Phi(max(x_j + A_i, B_i) / sigma)

    over the draws x_j = `noise_samples` of the claimed token's noise, with Gaussian noise of std sigma on every
    competitor, B_i = cutoff - l_i, and `cutoff` the smallest logit that survives the top-k/top-p filter
    (-inf: no filter).  One array expression over (draws x competitors)."""
    logits = np.asarray(logits, dtype=np.float64)
    gumbel = np.asarray(gumbel, dtype=np.float64)
    x = np.asarray(noise_samples, dtype=np.float64)
    S = active_subset(logits + temperature * gumbel, claimed, s)
    A = margins(logits, gumbel, temperature, claimed, S)
    B = cutoff - logits[S]
    survives = (logits[claimed] + x > cutoff).astype(np.float64)
    factors = ndtr(np.maximum(x[:, None] + A[None, :], B[None, :]) / sigma)
    return float(np.mean(survives * np.prod(factors, axis=1)))


def token_difr_quadrature(logits, gumbel, temperature, claimed, s, sigma, order=200):
    """E_{x ~ N(0, sigma^2)} prod_{i in S} Phi((x + A_i)/sigma), no filter."""
    logits = np.asarray(logits, dtype=np.float64)
    gumbel = np.asarray(gumbel, dtype=np.float64)
    y = logits + temperature * gumbel
    S = active_subset(y, claimed, s)
    A = margins(logits, gumbel, temperature, claimed, S)
    nodes, weights = np.polynomial.hermite.hermgauss(order)
    x = np.sqrt(2.0) * sigma * nodes
    vals = np.prod(ndtr((x[:, None] + A[None, :]) / sigma), axis=1)
    return float(np.sum(weights * vals) / np.sqrt(np.pi))


def fixed_seed_posterior_mc(logits, gumbel, temperature, claimed, sigma, n_draws, rng):
    """Pr over independent N(0, sigma^2) perturbations of every logit that the
    Gumbel-max sampler, noise fixed, returns `claimed`."""
    logits = np.asarray(logits, dtype=np.float64)
    gumbel = np.asarray(gumbel, dtype=np.float64)
    hits = 0
    done = 0
    while done < n_draws:
        n = min(200_000, n_draws - done)
        pert = logits[None, :] + sigma * rng.standard_normal((n, logits.shape[0]))
        hits += int(np.sum(np.argmax(pert + temperature * gumbel[None, :], axis=1) == claimed))
        done += n
    return hits / n_draws
