"""Parity at the full sizes of the five workloads, in the launch configuration
the benchmark times: the GPU scores every row, the oracle re-scores a seeded
sample of rows one by one (its honest claims come from its own sampler on the
server-side hidden states), and properties that hold at any size are checked on
all rows."""
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

CASES = [
    ("llama3b", 0, 0.7, 0.05),
    ("llama3b", 0, 1.0, 1.0),
    ("llama8b", 0, 1.0, 0.05),
    ("moe30b", 0, 0.7, 0.05),
    ("longstream", 4096, 1.0, 0.05),
    ("longstream", 131072, 1.0, 1.0),
]

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


def _threshold_in_a_gap(scores, quantile=0.3, min_gap=2e-2):
    s = np.sort(scores)
    gaps = np.diff(s)
    ok = np.nonzero(gaps >= min_gap)[0]
    assert len(ok), "no gap wide enough for an unambiguous threshold"
    i = ok[np.argmin(np.abs(ok - quantile * len(s)))]
    return float(np.float32(0.5 * (s[i] + s[i + 1])))


@pytest.mark.parametrize("name,T,temperature,sigma", CASES)
def test_full_size_gm(name, T, temperature, sigma):
    w, inp, dev = _inputs(name, T)
    rows = wl.sample_rows(w, N_SAMPLE)
    g = np.random.default_rng(wl.stream_seed(w, 7))
    tokens = g.integers(0, w.V, size=w.T).astype(np.int32)
    tokens[rows] = _sampled_claims(w, inp, rows, f32(temperature), "gm")
    got = dev.score("gm", tokens, temperature, sigma, EPS)
    ref = oracle.score_gm(np.ascontiguousarray(inp.h[rows]), inp.W, tokens[rows], inp.seeds[rows],
                          inp.positions[rows], f32(temperature), f32(sigma), f32(EPS))
    np.testing.assert_allclose(got["score"][rows], ref.score, rtol=0, atol=SCORE_TOL)
    np.testing.assert_allclose(got["margin"][rows], ref.margin, rtol=0, atol=1e-4)
    clear = ref.top2_margin >= ARGMAX_MARGIN
    assert np.array_equal(got["argmax"][rows][clear], ref.argmax[clear])
    clear2 = clear & (ref.top23_margin >= ARGMAX_MARGIN)
    assert np.array_equal(got["runner_up"][rows][clear2], ref.runner_up[clear2])
    np.testing.assert_allclose(got["lse"][rows], ref.lse, rtol=LSE_RTOL)
    # every row: well-formed outputs and the exact-match bookkeeping
    assert np.all(got["row_status"] == 0)
    assert np.all(np.isfinite(got["score"])) and np.all(got["score"] <= 1e-6)
    assert np.all((got["argmax"] >= 0) & (got["argmax"] < w.V) & (got["runner_up"] >= 0) & (got["runner_up"] < w.V))
    assert np.all(got["argmax"] != got["runner_up"])
    assert np.array_equal(got["argmax"] == tokens, ~np.signbit(got["margin"]))
    # most honest claims of the sample match even though the server saw perturbed hidden states
    honest_rows = np.arange(len(rows)) % 6 != 1
    honest_rows &= np.arange(len(rows)) % 6 != 4
    assert ref.match[honest_rows].mean() > 0.8
    # detection decisions on the sample, threshold placed in a gap of the oracle's scores
    tau = _threshold_in_a_gap(ref.score)
    ref_flags, _ = oracle.detect(ref.score, tau, ref.margin, None)
    flags = torch.empty(w.T, dtype=torch.uint8, device="cuda")
    stats = torch.zeros((len(inp.seq_offsets) - 1, 4), dtype=torch.int32, device="cuda")
    difr.difr_detect(to_dev(got["score"]), tau, to_dev(got["margin"]), None, 0, to_dev(inp.seq_offsets), flags, stats)
    torch.cuda.synchronize()
    f = flags.cpu().numpy()
    assert np.array_equal(f[rows], ref_flags)
    st = stats.cpu().numpy().view(SEQ_STATS_DTYPE).reshape(-1)
    assert st["n_flagged"].sum() == f.sum()
    assert st["n_match"].sum() == (got["argmax"] == tokens).sum()
    per_seq = got["score"].reshape(-1, w.seq_len)
    np.testing.assert_allclose(st["sum"], per_seq.astype(np.float64).sum(axis=1), rtol=1e-4)
    assert np.array_equal(st["min"], per_seq.min(axis=1))


@pytest.mark.parametrize("name,T,temperature,sigma", [("llama3b", 0, 1.0, 1.0), ("moe30b", 0, 0.7, 0.05)])
def test_full_size_ipt(name, T, temperature, sigma):
    w, inp, dev = _inputs(name, T)
    rows = wl.sample_rows(w, N_SAMPLE, salt=1)
    g = np.random.default_rng(wl.stream_seed(w, 8))
    tokens = g.integers(0, w.V, size=w.T).astype(np.int32)
    tokens[rows] = _sampled_claims(w, inp, rows, f32(temperature), "ipt")
    got = dev.score("ipt", tokens, temperature, sigma, EPS)
    ref = oracle.score_ipt(np.ascontiguousarray(inp.h[rows]), inp.W, tokens[rows], inp.seeds[rows],
                           inp.positions[rows], f32(temperature), f32(sigma), f32(EPS))
    np.testing.assert_allclose(got["score"][rows], ref.score, rtol=0, atol=SCORE_TOL)
    np.testing.assert_allclose(got["lse"][rows], ref.lse, rtol=LSE_RTOL)
    np.testing.assert_allclose(got["cdf_lo"][rows], ref.cdf_lo, rtol=0, atol=2e-6)
    np.testing.assert_allclose(got["p_claimed"][rows], ref.p_claimed, rtol=1e-3, atol=1e-12)
    assert np.all(got["row_status"] == 0)
    assert np.all((got["cdf_lo"] >= -1e-6) & (got["cdf_lo"] <= 1 + 1e-6))
    assert np.all((got["u"] > 0) & (got["u"] < 1))


@pytest.mark.parametrize("name,T,temperature,sigma", [("llama3b", 0, 1.0, 1.0), ("moe30b", 0, 0.7, 0.3)])
def test_full_size_rank_both_and_admissible_sets(name, T, temperature, sigma):
    """The widened calls at full size: ranks, both scores and admissible-set sizes on sampled rows against the
    oracle (integers within the reach of the kernel's fp32 rounding, equal on almost every row), and
    size-independent properties on all rows."""
    from scipy.special import ndtr

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
    # ranks
    logits = oracle.logits(hs, Ws)
    lt = logits[np.arange(len(rows)), tokens[rows]][:, None]
    others = np.ones_like(logits, dtype=bool)
    others[np.arange(len(rows)), tokens[rows]] = False
    lo = ((logits > lt + 2e-5) & others).sum(axis=1)
    hi = ((logits > lt - 2e-5) & others).sum(axis=1)
    rank = out.rank.cpu().numpy()
    assert np.all(rank[rows] >= lo) and np.all(rank[rows] <= hi)
    assert (rank[rows] == ref.rank).mean() >= 0.9
    assert np.all((rank >= 0) & (rank < w.V))
    # admissible sets
    y = logits.copy()
    for i, r in enumerate(rows):
        y[i] += f32(temperature) * oracle.gumbel_noise_row(int(inp.seeds[r]), int(inp.positions[r]), w.V)
    order = np.sort(y, axis=1)
    ymax, ysec = order[:, -1:], order[:, -2:-1]
    A = np.where(y == ymax, ymax - ysec, y - ymax)
    got = counts.cpu().numpy()
    for j, tau in enumerate(taus):
        size = lambda shift: (np.log(ndtr((A + shift) / (f32(sigma) * np.sqrt(2.0))) + f32(EPS)) >= tau).sum(axis=1)
        want = oracle.admissible_count(hs, Ws, inp.seeds[rows], inp.positions[rows], f32(temperature), f32(sigma),
                                       tau, f32(EPS))
        assert np.array_equal(size(0.0), want)
        assert np.all(got[j][rows] >= size(-1e-3)) and np.all(got[j][rows] <= size(1e-3))
    assert np.all(got[0] <= got[1]) and np.all(got[1] >= 1) and np.all(got[1] <= w.V)
