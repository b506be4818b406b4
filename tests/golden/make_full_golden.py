"""Writes the stored oracle values the full-size GPU parity tests compare against.

    python tests/golden/make_full_golden.py [case ...]      (cases: see CASES; default: all missing ones)

Imports only `oracle/` and `workloads/`.  For every case it draws the seeded
inputs, lets the oracle's own samplers (Alg. "Gumbel-Max Sampler", Alg. "IPT
Sampler") produce the honest claims on the server-side hidden states, replaces
the workload's seeded fraction of them, scores the claims with the oracle on the
verifier's hidden states, calibrates the detection threshold on the untampered
rows (1 % false positives, Sec. "Classification via Thresholding") and stores
everything in `tests/golden/full_<case>.npz`.

Rows: all of them for the tiny / llama3b / llama8b / moe30b workloads and for the
long stream at T = 4096; for the long stream at T >= 32768 a seeded subset of
4096 rows that contains every tampered row (the fp64 contraction costs 1.6 GFLOP
per row there).

The oracle is slow: the whole set takes a few hours of an 8-core host.
"""
from __future__ import annotations

import hashlib
import os
import sys
import time

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(os.path.dirname(HERE))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import oracle  # noqa: E402
import workloads as wl  # noqa: E402
from oracle.calibration import threshold_at_fpr, threshold_in_gap  # noqa: E402

EPS = float(np.float32(1e-12))
SIGMAS_GM = tuple(float(np.float32(s)) for s in (1.0, 0.05, 0.01, 0.001))   # the paper sweeps 0.001 .. 1
SIGMAS_IPT = tuple(float(np.float32(s)) for s in (1.0, 0.1, 0.05))
TARGET_FPR = 0.01
MIN_GAP = 2e-2
N_SUBSET = 4096

# name -> (workload, T (0: the workload's own), temperature)
CASES = {
    "tiny": ("tiny", 0, 1.0),
    "llama3b_t07": ("llama3b", 0, 0.7),
    "llama3b_t10": ("llama3b", 0, 1.0),
    "llama8b": ("llama8b", 0, 1.0),
    "moe30b": ("moe30b", 0, 0.7),
    "longstream_4096": ("longstream", 4096, 1.0),
    "longstream_32768": ("longstream", 32768, 1.0),
    "longstream_131072": ("longstream", 131072, 1.0),
    "longstream_262144": ("longstream", 262144, 1.0),
}
# cheapest evidence first: the sizes no other test covers, then by cost
ORDER = ("tiny", "longstream_262144", "longstream_32768", "llama3b_t10", "llama3b_t07", "longstream_131072",
         "longstream_4096", "llama8b", "moe30b")


def path_of(case: str) -> str:
    return os.path.join(HERE, f"full_{case}.npz")


def digest(a: np.ndarray) -> str:
    return hashlib.sha256(np.ascontiguousarray(a).tobytes()).hexdigest()


def select_rows(w: wl.Workload) -> np.ndarray:
    """All rows, or (long streams) every tampered row plus a seeded sample, 4096 in all."""
    if not (w.name == "longstream" and w.T > N_SUBSET):
        return np.arange(w.T, dtype=np.int64)
    _, mask = wl.tamper(w, np.zeros(w.T, dtype=np.int32), np.zeros(w.T, dtype=np.int32))
    bad = np.nonzero(mask)[0]
    pool = wl.sample_rows(w, N_SUBSET + len(bad))  # sorted, seeded
    extra = pool[~np.isin(pool, bad)][: N_SUBSET - len(bad)]
    return np.sort(np.concatenate([bad, extra])).astype(np.int64)


def tampered_claims(w: wl.Workload, rows: np.ndarray, honest: np.ndarray, runner: np.ndarray):
    """The workload's seeded tampering applied to the selected rows (the rows it picks do not depend on the
    claims, and every row it picks is among `rows`)."""
    full_h = np.zeros(w.T, dtype=np.int32)
    full_r = np.zeros(w.T, dtype=np.int32)
    full_h[rows] = honest
    full_r[rows] = runner
    tokens, mask = wl.tamper(w, full_h, full_r)
    assert np.all(np.isin(np.nonzero(mask)[0], rows))
    return tokens[rows].astype(np.int32), mask[rows]


def calibrate(scores: np.ndarray, benign: np.ndarray):
    tau0 = threshold_at_fpr(scores[benign], TARGET_FPR)
    tau, guard = threshold_in_gap(scores, tau0, MIN_GAP)
    tau32 = float(np.float32(tau))  # the C ABI takes a float
    guard -= abs(tau32 - tau)
    return tau32, guard, tau0


def make_case(case: str) -> None:
    name, T, temperature = CASES[case]
    temperature = float(np.float32(temperature))
    w = wl.WORKLOADS[name]
    if T:
        w = wl.with_T(w, T)
    t0 = time.time()
    inp = wl.make_inputs(w)
    rows = select_rows(w)
    n = len(rows)
    h = np.ascontiguousarray(inp.h[rows])
    hs = np.ascontiguousarray(inp.h_server[rows])
    seeds, positions = inp.seeds[rows], inp.positions[rows]
    print(f"[{case}] inputs in {time.time() - t0:.0f} s; {n} rows, {oracle.num_threads()} threads", flush=True)

    # the inference server: both samplers on its own hidden states, one contraction per row
    t0 = time.time()
    zeros = np.zeros(n, dtype=np.int32)
    gm_s, ipt_s = oracle.score_both(hs, inp.W, zeros, zeros, seeds, positions, temperature, 1.0, 1.0, EPS)
    honest_gm, runner_gm, honest_ipt = gm_s.argmax.copy(), gm_s.runner_up.copy(), ipt_s.sampled.copy()
    print(f"[{case}] samplers in {time.time() - t0:.0f} s", flush=True)
    tokens_gm, tampered = tampered_claims(w, rows, honest_gm, runner_gm)
    tokens_ipt, tampered_ipt = tampered_claims(w, rows, honest_ipt, runner_gm)
    assert np.array_equal(tampered, tampered_ipt)

    # the verifier: both estimators on its hidden states
    t0 = time.time()
    gm, ipt = oracle.score_both(h, inp.W, tokens_gm, tokens_ipt, seeds, positions, temperature, SIGMAS_GM[0],
                                SIGMAS_IPT[0], EPS)
    print(f"[{case}] scores in {time.time() - t0:.0f} s", flush=True)

    score_gm = np.empty((len(SIGMAS_GM), n), dtype=np.float64)
    score_gm[0] = gm.score
    for j, s in enumerate(SIGMAS_GM[1:], start=1):
        score_gm[j] = [oracle.gm_score(float(a), s, EPS) for a in gm.margin]
    score_ipt = np.empty((len(SIGMAS_IPT), n), dtype=np.float64)
    score_ipt[0] = ipt.score
    for j, s in enumerate(SIGMAS_IPT[1:], start=1):
        score_ipt[j] = [oracle.ipt_score(float(a), float(a + p), float(u), s, EPS)
                        for a, p, u in zip(ipt.cdf_lo, ipt.p_claimed, ipt.u)]

    benign = ~tampered
    cal_gm = [calibrate(score_gm[j], benign) for j in range(len(SIGMAS_GM))]
    cal_ipt = [calibrate(score_ipt[j], benign) for j in range(len(SIGMAS_IPT))]

    np.savez_compressed(
        path_of(case),
        workload=name, T=w.T, temperature=temperature, eps=EPS, rows=rows.astype(np.int32),
        digest_h=digest(h), digest_W=digest(inp.W), digest_seeds=digest(seeds), digest_positions=digest(positions),
        tampered=tampered, tokens_gm=tokens_gm, tokens_ipt=tokens_ipt,
        honest_match_rate=float(gm.match[benign].mean()),
        sigmas_gm=np.array(SIGMAS_GM), score_gm=score_gm.astype(np.float32), margin=gm.margin,
        argmax=gm.argmax, runner_up=gm.runner_up, top2_margin=gm.top2_margin.astype(np.float32),
        top23_margin=gm.top23_margin.astype(np.float32), lse=gm.lse.astype(np.float32), rank=gm.rank,
        row_status=gm.row_status,
        tau_gm=np.array([c[0] for c in cal_gm]), guard_gm=np.array([c[1] for c in cal_gm]),
        tau_gm_quantile=np.array([c[2] for c in cal_gm]),
        sigmas_ipt=np.array(SIGMAS_IPT), score_ipt=score_ipt.astype(np.float32), p_claimed=ipt.p_claimed,
        cdf_lo=ipt.cdf_lo, u=ipt.u,
        tau_ipt=np.array([c[0] for c in cal_ipt]), guard_ipt=np.array([c[1] for c in cal_ipt]),
        tau_ipt_quantile=np.array([c[2] for c in cal_ipt]),
    )
    print(f"[{case}] wrote {path_of(case)} ({os.path.getsize(path_of(case)) / 1e6:.2f} MB); "
          f"honest match rate {gm.match[benign].mean():.4f}", flush=True)


def main(argv):
    cases = argv or [c for c in ORDER if not os.path.exists(path_of(c))]
    for c in cases:
        if c not in CASES:
            raise SystemExit(f"unknown case {c}; known: {', '.join(CASES)}")
    for c in cases:
        make_case(c)


if __name__ == "__main__":
    main(sys.argv[1:])
