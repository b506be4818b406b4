"""Token-DiFR beyond one competitor, in plain numpy -- TEST INFRASTRUCTURE.

The scoring path uses Alg. Token-DiFR with an active subset of one competitor
and no top-k/top-p filter, where the expectation has a closed form.  This module
states the algorithm in its general form so that the closed form can be checked:

* `token_difr_monte_carlo`  the algorithm's sampling loop, step by step;
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
    """Alg. Token-DiFR: `noise_samples` are the M draws x_j of the claimed token's
    noise; every competitor's noise CDF is Gaussian with std sigma; `cutoff` is the
    smallest logit that survives the top-k/top-p filter (-inf: no filter)."""
    logits = np.asarray(logits, dtype=np.float64)
    gumbel = np.asarray(gumbel, dtype=np.float64)
    y = logits + temperature * gumbel
    S = active_subset(y, claimed, s)
    A = margins(logits, gumbel, temperature, claimed, S)
    B = cutoff - logits[S]
    total = 0.0
    for x in np.asarray(noise_samples, dtype=np.float64):
        if logits[claimed] + x > cutoff:
            total += float(np.prod(ndtr(np.maximum(x + A, B) / sigma)))
    return total / len(noise_samples)


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
