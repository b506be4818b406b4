"""Seeded random shapes and parameters: GPU scores against the oracle, element by element, far from the round
numbers the other tests use (tile and strip boundaries at odd places, tiny and lopsided problems)."""
import math

import numpy as np
import pytest

import oracle
import workloads as wl
from gpu_util import Device, f32

pytestmark = pytest.mark.gpu

EPS = 1e-12
SCORE_TOL = 2e-3


def _case(i):
    g = np.random.default_rng(1000 + i)
    T = int(g.choice([1, 2, 31, 127, 128, 129, 255, 257, 300, 513, 700]))
    d = 8 * int(g.integers(1, 66))
    V = int(g.choice([2, 3, 15, 16, 17, 255, 256, 257, 511, 1000, 4095, 4097, 8191, 8200, 9999]))
    temperature = float(g.choice([0.0, 0.25, 0.7, 1.0, 1.9]))
    sigma = float(g.choice([0.02, 0.05, 0.3, 1.0, 4.0]))
    scale = float(g.choice([0.3, 1.0, 4.0]))
    return T, d, V, temperature, sigma, scale, g


@pytest.mark.parametrize("i", range(24))
def test_random_problem(i):
    T, d, V, temperature, sigma, scale, g = _case(i)
    h = wl.f32_to_bf16_bits(g.standard_normal((T, d)).astype(np.float32))
    W = wl.f32_to_bf16_bits((scale * g.standard_normal((V, d)) / math.sqrt(d)).astype(np.float32))
    seeds = g.integers(0, 2**63, size=T, dtype=np.int64).astype(np.uint64) * np.uint64(2) + np.uint64(1)
    positions = g.integers(0, 2**31, size=T, dtype=np.int64).astype(np.uint32)
    honest, runner = oracle.sample_gm(h, W, seeds, positions, f32(temperature))
    tokens = honest.copy()
    pick = g.random(T)
    tokens[pick < 0.2] = runner[pick < 0.2]
    rnd = g.integers(-2, V + 2, size=T)
    tokens[pick > 0.8] = rnd[pick > 0.8]
    tokens = tokens.astype(np.int32)
    dev = Device(h, W, seeds, positions)

    ref = oracle.score_gm(h, W, tokens, seeds, positions, f32(temperature), f32(sigma), f32(EPS))
    got = dev.score("gm", tokens, temperature, sigma, EPS)
    np.testing.assert_allclose(got["score"], ref.score, rtol=0, atol=SCORE_TOL)
    fin = np.isfinite(ref.margin)
    np.testing.assert_allclose(got["margin"][fin], ref.margin[fin], rtol=0, atol=1e-4 * max(1.0, scale))
    assert np.array_equal(got["margin"][~fin], ref.margin[~fin])
    clear = ref.top2_margin >= 1e-3 * max(1.0, scale)
    assert np.array_equal(got["argmax"][clear], ref.argmax[clear])
    assert np.array_equal(got["row_status"], ref.row_status)
    if temperature > 0:
        np.testing.assert_allclose(got["lse"], ref.lse, rtol=1e-3, atol=1e-3)
        sigma_ipt = float(g.choice([0.05, 0.2, 1.0]))
        itok = oracle.sample_ipt(h, W, seeds, positions, f32(temperature)).astype(np.int32)
        itok[pick > 0.7] = tokens[pick > 0.7]
        iref = oracle.score_ipt(h, W, itok, seeds, positions, f32(temperature), f32(sigma_ipt), f32(EPS))
        igot = dev.score("ipt", itok, temperature, sigma_ipt, EPS)
        np.testing.assert_allclose(igot["score"], iref.score, rtol=0, atol=SCORE_TOL)
        ok = iref.row_status == 0
        np.testing.assert_allclose(igot["cdf_lo"][ok], iref.cdf_lo[ok], rtol=2e-5, atol=2e-6)
        assert np.array_equal(igot["row_status"], iref.row_status)
    else:
        assert np.all(np.isnan(got["lse"]))
