"""The widened calls (raw-logit rank, both estimators in one pass, admissible sets) at
full size, in the launch configuration the benchmark times: the oracle re-scores a
seeded sample of rows one by one, and properties that hold at any size are checked
on all rows.  (The two estimators themselves are compared row by row with stored
oracle values in test_gpu_golden_full.py.)"""
import numpy as np
import pytest
import torch

import oracle
import workloads as wl
from gpu_util import SEQ_STATS_DTYPE, Device, f32, to_dev

import paper_2511_02620_b200 as difr

pytestmark = pytest.mark.gpu

SCORE_TOL = 2e-3
LSE_RTOL = 1e-3
ARGMAX_MARGIN = 1e-3
EPS = 1e-12
N_SAMPLE = 48

_cache = {}


def _inputs(name, T):
    key = (name, T)
    if key not in _cache:
        _cache.clear()  # one workload resident at a time
        w = wl.WORKLOADS[name]
        if T:
            w = wl.with_T(w, T)
        inp = wl.make_inputs(w)
        _cache[key] = (w, inp, Device(inp.h, inp.W, inp.seeds, inp.positions))
    return _cache[key]


def _sampled_claims(w, inp, rows, temperature, kind):
    """Claims for the sampled rows from the oracle's own samplers; a third of them tampered."""
    hs = np.ascontiguousarray(inp.h_server[rows])
    if kind == "gm":
        honest, runner = oracle.sample_gm(hs, inp.W, inp.seeds[rows], inp.positions[rows], temperature)
    else:
        honest = oracle.sample_ipt(hs, inp.W, inp.seeds[rows], inp.positions[rows], temperature)
        runner = (honest + 1) % w.V
    g = np.random.default_rng(wl.stream_seed(w, 3))
    claims = honest.copy()
    k = np.arange(len(rows))
    claims[k % 6 == 1] = runner[k % 6 == 1]
    rnd = g.integers(0, w.V, size=len(rows))
    claims[k % 6 == 4] = rnd[k % 6 == 4]
    return claims.astype(np.int32)


@pytest.mark.parametrize("name,T,temperature,sigma", [("llama3b", 0, 1.0, 1.0), ("moe30b", 0, 0.7, 0.3)])
def test_full_size_rank_both_and_admissible_sets(name, T, temperature, sigma):
    """The widened calls at full size: ranks, both scores and admissible-set sizes on sampled rows against the
    oracle (the integers identical), and size-independent properties on all rows."""
    w, inp, dev = _inputs(name, T)
    rows = wl.sample_rows(w, 24, salt=2)
    g = np.random.default_rng(wl.stream_seed(w, 9))
    tokens = g.integers(0, w.V, size=w.T).astype(np.int32)
    tokens[rows] = _sampled_claims(w, inp, rows, f32(temperature), "gm")
    out = difr.DifrOut.allocate(w.T, w.d, w.V, sigma, EPS)
    f = lambda: torch.full((w.T,), float("nan"), dtype=torch.float32, device="cuda")
    out.y_max, out.y_second, out.score_ipt, out.sigma_ipt = f(), f(), f(), 0.05
    out.rank = torch.full((w.T,), -7, dtype=torch.int32, device="cuda")
    difr.difr_score_both(dev.h, dev.W, to_dev(tokens), dev.seeds, dev.positions, f32(temperature), out)
    taus = [f32(-0.9), f32(-3.0)]
    counts = torch.full((2, w.T), -1, dtype=torch.int32, device="cuda")
    difr.difr_admissible(dev.h, dev.W, dev.seeds, dev.positions, f32(temperature), out, taus, counts)
    torch.cuda.synchronize()
    assert int(out.device_status.item()) == 0

    hs, Ws = np.ascontiguousarray(inp.h[rows]), inp.W
    ref = oracle.score_gm(hs, Ws, tokens[rows], inp.seeds[rows], inp.positions[rows], f32(temperature), f32(sigma),
                          f32(EPS))
    ref_ipt = oracle.score_ipt(hs, Ws, tokens[rows], inp.seeds[rows], inp.positions[rows], f32(temperature),
                               f32(0.05), f32(EPS))
    np.testing.assert_allclose(out.score.cpu().numpy()[rows], ref.score, rtol=0, atol=SCORE_TOL)
    np.testing.assert_allclose(out.score_ipt.cpu().numpy()[rows], ref_ipt.score, rtol=0, atol=SCORE_TOL)
    # ranks: the oracle's integers
    rank = out.rank.cpu().numpy()
    assert np.array_equal(rank[rows], ref.rank)
    assert np.all((rank >= 0) & (rank < w.V))
    assert np.all(out.row_status.cpu().numpy() & 32 == 0)
    # admissible sets: the oracle's integers
    got = counts.cpu().numpy()
    for j, tau in enumerate(taus):
        want = oracle.admissible_count(hs, Ws, inp.seeds[rows], inp.positions[rows], f32(temperature), f32(sigma),
                                       tau, f32(EPS))
        assert np.array_equal(got[j][rows], want), (j, got[j][rows], want)
    assert np.all(got[0] <= got[1]) and np.all(got[1] >= 1) and np.all(got[1] <= w.V)
