"""Pins for the oracle's risk classes, admissible sets and information bound
(Sec. "Empirical Results"; Alg. "Per-Token Risk Classification via GLS and Rank")."""
import math
import os

import numpy as np
import pytest

import oracle
import workloads as wl

EPS = 1e-12


def _bits(x):
    return wl.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def _small(T, d, V, seed):
    g = np.random.default_rng(seed)
    h = _bits(g.standard_normal((T, d)))
    W = _bits(g.standard_normal((V, d)) * 2.0 / math.sqrt(d))
    seeds = np.full(T, 0xC0FFEE1234567, dtype=np.uint64)
    positions = np.arange(1, T + 1, dtype=np.uint32)
    return h, W, seeds, positions


def test_three_classes_follow_the_algorithm_case_by_case():
    # (score, rank) pairs around tau = -2, R = 3 (ranks count from 0: the suspicious ids are ranks 0, 1, 2),
    # one of each branch plus the boundaries
    scores = np.array([-1.0, -2.0, -2.0000001, -5.0, -5.0, -5.0, np.nan, np.nan])
    ranks = np.array([100, 100, 0, 2, 3, 0, 0, 9], dtype=np.int32)
    got = oracle.classify(scores, -2.0, ranks, 3)
    #   safe   safe (equal)  susp.  susp. (last of the top R)  danger  susp.  NaN is not >= tau: susp. / danger
    assert got.tolist() == [0, 0, 1, 1, 2, 1, 1, 2]
    # without ranks only the threshold acts, exactly like the detection flags
    flags, _ = oracle.detect(scores, -2.0)
    assert np.array_equal(oracle.classify(scores, -2.0), flags)


def test_rank_cutoff_counts_ids_the_way_the_ablations_describe():
    """Appendix "Logit-Rank Ablations": with cutoff 1 only the top-ranked token may be suspicious; with cutoff 4
    the top four, which is why such a token carries log2(4) = 2 bits.  Worked through on a row of known
    logits: the flagged claim is moved down the ranking and the suspicious ids are counted."""
    d, V = 8, 12
    # h = e_0 and W[v, 0] = -v: logits 0, -1, -2, ... so id v has exactly v larger logits (rank v)
    h = _bits(np.eye(1, d))
    W = np.zeros((V, d), dtype=np.float32)
    W[:, 0] = -np.arange(V)
    W = _bits(W)
    seeds, positions = np.array([7], dtype=np.uint64), np.array([1], dtype=np.uint32)
    ranks = np.array([oracle.score_gm(h, W, np.array([v], dtype=np.int32), seeds, positions, 1.0, 1.0, EPS).rank[0]
                      for v in range(V)], dtype=np.int32)
    assert ranks.tolist() == list(range(V))
    flagged = np.full(V, -30.0)  # every claim fails the threshold
    for R in (1, 4, 8):
        classes = oracle.classify(flagged, -2.0, ranks, R)
        assert (classes == 1).sum() == R  # a suspicious token is one of exactly R ids => log2 R bits
        assert classes.tolist() == [1] * R + [2] * (V - R)
    # cutoff 1: the claim holding the second-largest logit is already dangerous
    assert oracle.classify(flagged[:2], -2.0, ranks[:2], 1).tolist() == [1, 2]


@pytest.mark.parametrize("sigma,temperature", [(1.0, 1.0), (0.3, 0.7), (0.05, 1.0)])
def test_admissible_set_equals_rescoring_every_id_as_the_claim(sigma, temperature):
    """A_t(tau) = {i : FSSL_t(i) >= tau}: count it by calling the (separately pinned) scoring routine once per
    candidate claim."""
    T, d, V = 5, 16, 40
    h, W, seeds, positions = _small(T, d, V, 11)
    all_scores = np.empty((T, V))
    for i in range(V):
        all_scores[:, i] = oracle.score_gm(h, W, np.full(T, i, dtype=np.int32), seeds, positions, temperature,
                                           sigma, EPS).score
    for tau in (-0.5, math.log(0.5), -3.0, -12.0, math.log(EPS) + 1e-9, -40.0):
        want = (all_scores >= tau).sum(axis=1)
        got = oracle.admissible_count(h, W, seeds, positions, temperature, sigma, tau, EPS)
        assert np.array_equal(got, want), (tau, got, want)


def test_admissible_set_limits():
    T, d, V = 6, 16, 64
    h, W, seeds, positions = _small(T, d, V, 12)
    # tau at or below the floor ln(eps): every id is admissible
    assert np.all(oracle.admissible_count(h, W, seeds, positions, 1.0, 0.5, math.log(EPS), EPS) == V)
    # tau above ln(1 + eps): nothing is
    assert np.all(oracle.admissible_count(h, W, seeds, positions, 1.0, 0.5, 1e-6, EPS) == 0)
    # sigma -> 0 turns the score into exact matching: only the verifier's own sample is admissible
    r = oracle.score_gm(h, W, np.zeros(T, dtype=np.int32), seeds, positions, 1.0, 1e-6, EPS)
    assert np.all(r.top2_margin > 1e-3)
    assert np.all(oracle.admissible_count(h, W, seeds, positions, 1.0, 1e-6, -1.0, EPS) == 1)
    # the set grows as tau falls and as sigma grows
    c = [oracle.admissible_count(h, W, seeds, positions, 1.0, 1.0, tau, EPS) for tau in (-0.1, -1.0, -5.0, -20.0)]
    assert all(np.all(a <= b) for a, b in zip(c, c[1:]))
    s = [oracle.admissible_count(h, W, seeds, positions, 1.0, sg, -3.0, EPS) for sg in (0.1, 0.5, 2.0)]
    assert all(np.all(a <= b) for a, b in zip(s, s[1:]))
    # the verifier's own sample is admissible whenever tau <= ln(1/2): its margin is >= 0
    assert np.all(oracle.admissible_count(h, W, seeds, positions, 1.0, 0.2, math.log(0.5), EPS) >= 1)


def test_exfiltratable_information_worked_cases():
    V, R = 1024, 8
    classes = np.array([0, 0, 0, 1, 2, 0], dtype=np.uint8)
    counts = np.array([1, 2, 16, 500, 500, 0], dtype=np.int32)
    bits, seq = oracle.exfiltratable_bits(classes, counts, R, V, np.array([0, 3, 6], dtype=np.int32))
    assert bits.tolist() == [0.0, 1.0, 4.0, 3.0, 10.0, 0.0]
    assert seq.tolist() == [5.0, 13.0]
    _, one = oracle.exfiltratable_bits(classes, counts, R, V)
    assert one.tolist() == [18.0]
    # a suspicious token never carries more than a dangerous one, nor a safe one more than log2 |V|
    assert math.log2(R) <= math.log2(V)


def test_exfiltratable_information_caps_the_paper_states():
    """Suspicious tokens carry log2(rank cutoff) bits (2 at cutoff 4, 3 at cutoff 8), dangerous ones
    log2 |V|: the figures the paper prints, read from the fixture."""
    path = os.path.join(os.path.dirname(__file__), "golden", "risk_class_bits.txt")
    rows = [ln.split() for ln in open(path) if ln.strip() and not ln.startswith("#")]
    assert len(rows) == 4
    for cls, R, V, want in rows:
        bits, _ = oracle.exfiltratable_bits(np.array([int(cls)], dtype=np.uint8), np.array([7], dtype=np.int32),
                                            int(R), int(V))
        assert bits.tolist() == [float(want)]
