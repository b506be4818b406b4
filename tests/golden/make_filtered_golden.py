"""Writes the stored oracle values of the filtered estimators at full size.

    python tests/golden/make_filtered_golden.py [case ...]      (cases: see CASES; default: all missing ones)

Imports only `oracle/` and `workloads/`.  For a seeded subset of the rows of
`full_<case>.npz` (made by make_full_golden.py: the claims come from there) it
scores Alg. "Token-DiFR" in full and Alg. "Token-IPT-DiFR" under each sampling
policy of POLICIES with `oracle/filtered.py` and stores scores and cutoffs in
`tests/golden/filtered_<case>.npz`.  Where a nucleus ends, the neighbouring
logits and prefix masses are stored too, so that a test can tell a decision
within rounding of a tie from a wrong one without the row's logits.

About twenty minutes of an 8-core host.
"""
from __future__ import annotations

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
from oracle import filtered  # noqa: E402

EPS = float(np.float32(1e-12))
SIGMA_GM = float(np.float32(0.3))
SIGMA_IPT = float(np.float32(0.1))
# (top_k, top_p, min_p, s): the paper's experimental setting; a nucleus over the whole vocabulary; a top-k beyond
# the candidate lists; min-p
POLICIES = ((50, 0.95, 0.0, 4), (0, 0.95, 0.0, 2), (1000, 1.0, 0.0, 3), (0, 1.0, 0.05, 1))
# case -> (the full golden it takes rows and claims from, number of rows)
CASES = {"llama3b_t10": ("llama3b_t10", 192), "longstream_262144": ("longstream_262144", 96)}


def path_of(case: str) -> str:
    return os.path.join(HERE, f"filtered_{case}.npz")


def pick(g, n: int) -> np.ndarray:
    """Indices into the full golden's rows: every tampered row first (at most a third), the rest evenly spaced."""
    bad = np.nonzero(g["tampered"])[0][: n // 3]
    rest = np.setdiff1d(np.linspace(0, len(g["rows"]) - 1, 4 * n).astype(np.int64), bad)[: n - len(bad)]
    return np.sort(np.concatenate([bad, rest]))


def nucleus_neighbours(l_row, temperature, top_k, top_p):
    """(logit one position before the oracle's last kept id, one after it, relative mass of the prefix that is one
    shorter, of the oracle's prefix): what a position-tolerant comparison of the cutoff needs."""
    V = l_row.shape[0]
    z = np.sort(l_row)[::-1]
    k = top_k if 0 < top_k < V else V
    e = np.exp((z[:k] - z[0]) / temperature)
    c = np.cumsum(e) / e.sum()
    n = min(int(np.searchsorted(c, top_p, side="left")) + 1, k)
    prev_l = z[n - 2] if n >= 2 else np.inf
    next_l = z[n] if n < k else -np.inf
    c_prev = c[n - 2] if n >= 2 else 0.0
    return float(prev_l), float(next_l), float(c_prev), float(c[n - 1])


def make_case(case: str) -> None:
    full, n = CASES[case]
    g = np.load(os.path.join(HERE, f"full_{full}.npz"))
    w = wl.WORKLOADS[str(g["workload"])]
    if int(g["T"]) != w.T:
        w = wl.with_T(w, int(g["T"]))
    temperature = float(g["temperature"])
    inp = wl.make_inputs(w)
    idx = pick(g, n)
    rows = g["rows"][idx].astype(np.int64)
    h = np.ascontiguousarray(inp.h[rows])
    seeds, positions = inp.seeds[rows], inp.positions[rows]
    tok_gm, tok_ipt = g["tokens_gm"][idx].astype(np.int32), g["tokens_ipt"][idx].astype(np.int32)
    L = oracle.logits(h, inp.W)
    store = dict(case=full, index=idx.astype(np.int32), rows=rows.astype(np.int32), tokens_gm=tok_gm,
                 tokens_ipt=tok_ipt, temperature=temperature, eps=EPS, sigma_gm=SIGMA_GM, sigma_ipt=SIGMA_IPT,
                 policies=np.array(POLICIES, dtype=np.float64))
    for j, (top_k, top_p, min_p, s) in enumerate(POLICIES):
        t0 = time.time()
        top_p32, min_p32 = float(np.float32(top_p)), float(np.float32(min_p))
        score, _, cut = filtered.score_gm_filtered(h, inp.W, tok_gm, seeds, positions, temperature, SIGMA_GM, EPS,
                                                   top_k, top_p32, s, min_p32)
        score_i, pt, a, mu, cut_i = filtered.score_ipt_filtered(h, inp.W, tok_ipt, seeds, positions, temperature,
                                                                 SIGMA_IPT, EPS, top_k, top_p32, min_p32)
        near = np.array([nucleus_neighbours(L[r], temperature, top_k, top_p32) for r in range(len(rows))])
        bar = L.max(axis=1) + temperature * np.log(min_p32) if min_p > 0 else np.full(len(rows), -np.inf)
        store.update({f"gm_score_{j}": score, f"gm_cutoff_{j}": cut, f"ipt_score_{j}": score_i, f"ipt_p_{j}": pt,
                      f"ipt_a_{j}": a, f"ipt_cutoff_{j}": cut_i, f"near_{j}": near, f"min_p_bar_{j}": bar})
        print(f"[{case}] policy {j} {POLICIES[j]} in {time.time() - t0:.0f} s", flush=True)
    np.savez_compressed(path_of(case), **store)
    print(f"[{case}] wrote {path_of(case)}", flush=True)


def main(argv):
    cases = argv or [c for c in CASES if not os.path.exists(path_of(c))]
    for c in cases:
        if c not in CASES:
            raise SystemExit(f"unknown case {c}; known: {', '.join(CASES)}")
    for c in cases:
        make_case(c)


if __name__ == "__main__":
    main(sys.argv[1:])
