"""Parity at the full sizes of the five workloads against stored oracle values.

`tests/golden/make_full_golden.py` (oracle and workload generators only) wrote, for every case, the claims the
oracle's samplers produce on the server-side hidden states, the workload's tampering, and the oracle's scores
of those claims: all rows of the tiny / llama3b / llama8b / moe30b workloads and of the long stream at
T = 4096, and a seeded 4096-row subset with every tampered row at T = 32768, 131072 and 262144.  Here the
library scores the whole workload in the launch configuration the benchmark times and every stored row is
compared element by element, for both estimators and over the paper's range of noise widths; the detection
decisions at the calibrated thresholds must be identical on every compared row."""
import hashlib
import os

import numpy as np
import pytest
import torch

import oracle
import workloads as wl
from gpu_util import SEQ_STATS_DTYPE, Device, to_dev

import paper_2511_02620_b200 as difr

pytestmark = pytest.mark.gpu

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
SCORE_TOL = 2e-3       # |score - oracle|
LSE_RTOL = 1e-3
ARGMAX_MARGIN = 1e-3   # ids must agree unless the oracle's own margin is below this ...
EXACT_MARGIN = 1e-6    # ... and, since the finalize kernel ranks its candidates in fp64, they do down to here

# one workload resident at a time: cases of the same (workload, T) stand together
CASES = ("tiny", "llama3b_t07", "llama3b_t10", "llama8b", "moe30b", "longstream_4096", "longstream_32768",
         "longstream_131072", "longstream_262144")

_cache = {}


def _digest(a):
    return hashlib.sha256(np.ascontiguousarray(a).tobytes()).hexdigest()


def _load(case):
    path = os.path.join(GOLDEN, f"full_{case}.npz")
    if not os.path.exists(path):
        pytest.skip(f"{os.path.basename(path)} has not been generated (tests/golden/make_full_golden.py {case})")
    g = np.load(path)
    key = (str(g["workload"]), int(g["T"]))
    if key not in _cache:
        _cache.clear()
        w = wl.WORKLOADS[key[0]]
        if key[1] != w.T:
            w = wl.with_T(w, key[1])
        inp = wl.make_inputs(w)
        # the stored values belong to these very inputs
        assert _digest(inp.W) == str(g["digest_W"]), "the seeded generator no longer reproduces W"
        _cache[key] = (w, inp, Device(inp.h, inp.W, inp.seeds, inp.positions))
    w, inp, dev = _cache[key]
    rows = g["rows"].astype(np.int64)
    assert _digest(inp.h[rows]) == str(g["digest_h"]), "the seeded generator no longer reproduces h"
    assert _digest(inp.seeds[rows]) == str(g["digest_seeds"])
    assert _digest(inp.positions[rows]) == str(g["digest_positions"])
    return g, w, inp, dev, rows


def _detect_on_rows(scores, margins, tau, n_rows):
    """difr_detect over the compared rows, gathered into one array and cut into sequences of 512 rows."""
    offs = np.arange(0, n_rows + 1, 512, dtype=np.int32)
    if offs[-1] != n_rows:
        offs = np.append(offs, np.int32(n_rows))
    flags = torch.full((n_rows,), 9, dtype=torch.uint8, device="cuda")
    stats = torch.zeros((len(offs) - 1, 4), dtype=torch.int32, device="cuda")
    difr.difr_detect(scores, float(tau), margins, None, 0, to_dev(offs), flags, stats)
    torch.cuda.synchronize()
    return flags.cpu().numpy(), stats.cpu().numpy().view(SEQ_STATS_DTYPE).reshape(-1), offs


def _check_token_difr(case):
    g, w, inp, dev, rows = _load(case)
    n = len(rows)
    temperature, eps = float(g["temperature"]), float(g["eps"])
    tokens = np.zeros(w.T, dtype=np.int32)
    tokens[rows] = g["tokens_gm"]
    rows_dev = torch.from_numpy(rows).cuda()
    clear = g["top2_margin"] >= EXACT_MARGIN
    clear2 = clear & (g["top23_margin"] >= EXACT_MARGIN)
    assert (g["top2_margin"] >= ARGMAX_MARGIN).sum() <= clear.sum()
    for j, sigma in enumerate(g["sigmas_gm"]):
        got = dev.score("gm", tokens, temperature, float(sigma), eps)
        worst = np.max(np.abs(got["score"][rows] - g["score_gm"][j]))
        assert worst <= SCORE_TOL, f"sigma {sigma}: max |score - oracle| = {worst} over {n} rows"
        if j == 0:
            np.testing.assert_allclose(got["margin"][rows], g["margin"], rtol=2e-6, atol=1e-6)
            assert np.array_equal(np.signbit(got["margin"][rows]), np.signbit(g["margin"]))
            assert np.array_equal(got["argmax"][rows][clear], g["argmax"][clear])
            assert np.array_equal(got["runner_up"][rows][clear2], g["runner_up"][clear2])
            np.testing.assert_allclose(got["lse"][rows], g["lse"], rtol=LSE_RTOL)
            assert np.array_equal(got["row_status"][rows], g["row_status"])
            # every row of the workload: well-formed outputs and the exact-match bookkeeping
            assert np.all(got["row_status"] == 0)
            assert np.all(np.isfinite(got["score"])) and np.all(got["score"] <= 1e-6)
            assert np.all((got["argmax"] >= 0) & (got["argmax"] < w.V))
            assert np.all((got["runner_up"] >= 0) & (got["runner_up"] < w.V))
            assert np.all(got["argmax"] != got["runner_up"])
            assert np.array_equal(got["argmax"] == tokens, ~np.signbit(got["margin"]))
        # detection at the calibrated threshold: no stored score lies within the guard band of tau
        tau, guard = float(g["tau_gm"][j]), float(g["guard_gm"][j])
        assert guard > 2 * SCORE_TOL
        ref_scores = g["score_gm"][j].astype(np.float64)
        score_dev = to_dev(got["score"])[rows_dev].contiguous()
        margin_dev = to_dev(got["margin"])[rows_dev].contiguous()
        flags, stats, offs = _detect_on_rows(score_dev, margin_dev, tau, n)
        ref_flags, ref_stats = oracle.detect(ref_scores, tau, g["margin"], offs)
        assert np.array_equal(flags, ref_flags), f"sigma {sigma}: {np.sum(flags != ref_flags)} decisions differ"
        assert np.array_equal(stats["n_flagged"], ref_stats["n_flagged"])
        assert np.array_equal(stats["n_match"], ref_stats["n_match"])
        np.testing.assert_allclose(stats["sum"], ref_stats["sum"], rtol=1e-5, atol=0.02)
        np.testing.assert_allclose(stats["min"], ref_stats["min"], rtol=0, atol=SCORE_TOL)
        # tampered rows are what the threshold is for: where honest claims (almost) always replay, the calibrated
        # threshold flags most of them.  (Where more than 1 % of the honest claims fail to replay because the
        # server saw perturbed hidden states, their scores reach the floor and the 1 % threshold sits at it.)
        if sigma <= 0.05 and g["tampered"].sum() >= 8 and float(g["honest_match_rate"]) > 0.995:
            assert flags[g["tampered"]].mean() > 0.5
    # raw-logit rank (an exact integer) and the three risk classes at rank cutoff 8, on every compared row
    out = difr.DifrOut.allocate(w.T, w.d, w.V, float(g["sigmas_gm"][1]), eps)
    out.rank = torch.full((w.T,), -7, dtype=torch.int32, device="cuda")
    difr.difr_score_gm(dev.h, dev.W, to_dev(tokens), dev.seeds, dev.positions, temperature, out)
    torch.cuda.synchronize()
    assert int(out.device_status.item()) == 0
    rank = out.rank.cpu().numpy()
    assert np.array_equal(rank[rows], g["rank"]), f"{np.sum(rank[rows] != g['rank'])} ranks differ"
    assert np.all(out.row_status.cpu().numpy() & 32 == 0)
    tau = float(g["tau_gm"][1])
    classes = torch.full((n,), 9, dtype=torch.uint8, device="cuda")
    difr.difr_detect(out.score[rows_dev].contiguous(), tau, out.margin[rows_dev].contiguous(),
                     out.rank[rows_dev].contiguous(), 8, None, classes, None)
    torch.cuda.synchronize()
    want = oracle.classify(g["score_gm"][1].astype(np.float64), tau, g["rank"], 8)
    assert np.array_equal(classes.cpu().numpy(), want)
    # whole-workload detection (every sequence of the workload, not only the compared rows)
    flags = torch.empty(w.T, dtype=torch.uint8, device="cuda")
    stats = torch.zeros((len(inp.seq_offsets) - 1, 4), dtype=torch.int32, device="cuda")
    tau = float(g["tau_gm"][-1])
    difr.difr_detect(to_dev(got["score"]), tau, to_dev(got["margin"]), None, 0, to_dev(inp.seq_offsets), flags, stats)
    torch.cuda.synchronize()
    f = flags.cpu().numpy()
    st = stats.cpu().numpy().view(SEQ_STATS_DTYPE).reshape(-1)
    assert st["n_flagged"].sum() == f.sum()
    assert st["n_match"].sum() == (got["argmax"] == tokens).sum()
    per_seq = got["score"].reshape(-1, w.seq_len)
    np.testing.assert_allclose(st["sum"], per_seq.astype(np.float64).sum(axis=1), rtol=1e-4, atol=1e-3)
    assert np.array_equal(st["min"], per_seq.min(axis=1))


def _check_token_ipt_difr(case):
    g, w, inp, dev, rows = _load(case)
    n = len(rows)
    temperature, eps = float(g["temperature"]), float(g["eps"])
    tokens = np.zeros(w.T, dtype=np.int32)
    tokens[rows] = g["tokens_ipt"]
    rows_dev = torch.from_numpy(rows).cuda()
    for j, sigma in enumerate(g["sigmas_ipt"]):
        got = dev.score("ipt", tokens, temperature, float(sigma), eps)
        worst = np.max(np.abs(got["score"][rows] - g["score_ipt"][j]))
        assert worst <= SCORE_TOL, f"sigma {sigma}: max |score - oracle| = {worst} over {n} rows"
        if j == 0:
            np.testing.assert_allclose(got["lse"][rows], g["lse"], rtol=LSE_RTOL)
            np.testing.assert_allclose(got["cdf_lo"][rows], g["cdf_lo"], rtol=0, atol=2e-6)
            np.testing.assert_allclose(got["p_claimed"][rows], g["p_claimed"], rtol=1e-3, atol=1e-12)
            np.testing.assert_allclose(got["u"][rows], g["u"], rtol=0, atol=1e-7)
            assert np.all(got["row_status"] == 0)
            assert np.all((got["cdf_lo"] >= -1e-6) & (got["cdf_lo"] <= 1 + 1e-6))
            assert np.all((got["u"] > 0) & (got["u"] < 1))
        tau, guard = float(g["tau_ipt"][j]), float(g["guard_ipt"][j])
        assert guard > 2 * SCORE_TOL
        score_dev = to_dev(got["score"])[rows_dev].contiguous()
        flags, stats, offs = _detect_on_rows(score_dev, None, tau, n)
        ref_flags, ref_stats = oracle.detect(g["score_ipt"][j].astype(np.float64), tau, None, offs)
        assert np.array_equal(flags, ref_flags), f"sigma {sigma}: {np.sum(flags != ref_flags)} decisions differ"
        assert np.array_equal(stats["n_flagged"], ref_stats["n_flagged"])
    # the narrowest width the header states the tolerance for: the oracle's closed form on its own stored (a, p, u)
    sigma = float(np.float32(0.01))
    got = dev.score("ipt", tokens, temperature, sigma, eps)
    want = np.array([oracle.ipt_score(float(a), float(a + p), float(u), sigma, eps)
                     for a, p, u in zip(g["cdf_lo"], g["p_claimed"], g["u"])])
    worst = np.max(np.abs(got["score"][rows] - want))
    assert worst <= SCORE_TOL, f"sigma {sigma}: max |score - oracle| = {worst} over {n} rows"


# case-major order: both estimators of a case run on the same resident inputs
@pytest.mark.parametrize("case,estimator", [(c, e) for c in CASES for e in ("token_difr", "token_ipt_difr")])
def test_scores_match_the_stored_oracle_values(case, estimator):
    (_check_token_difr if estimator == "token_difr" else _check_token_ipt_difr)(case)
