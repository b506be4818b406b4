"""The filtered estimators at full size against stored oracle values.

`tests/golden/make_filtered_golden.py` (oracle and workload generators only) scored a seeded subset of rows of the
llama3b workload and of the long stream at T = 262144 (every kind of claim the full-size goldens hold: honest,
tampered, filtered out) with Alg. "Token-DiFR" in full and Alg. "Token-IPT-DiFR" under four sampling policies: the
paper's experimental setting (top-k 50, top-p 0.95), a nucleus over the whole vocabulary, a top-k of 1000, min-p.
Here the library scores the whole workload in one call per policy (block by block at these sizes) and the stored
rows are compared: scores within the tolerance, cutoffs the oracle's, or the neighbouring position where the
nucleus decision lies within 3e-5 (relative mass) of a tie."""
import os

import numpy as np
import pytest
import torch

import workloads as wl
from gpu_util import Device, to_dev

import paper_2511_02620_b200 as difr

pytestmark = pytest.mark.gpu

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
SCORE_TOL = 2e-3
TIE_MASS = 3e-5


def _cutoff_ok(got, want, near, top_p, bar):
    prev_l, next_l, c_prev, c_at = near
    if (np.isneginf(got) and np.isneginf(want)) or abs(got - want) <= 1e-5:
        return True
    if np.isfinite(bar) and abs(want - bar) <= 1e-9:
        return False  # the min-p bound decides: no neighbouring position to fall back on
    if top_p < 1.0 and abs(got - prev_l) <= 1e-5:   # stopped one earlier: it saw that prefix reach top_p
        return top_p - c_prev <= TIE_MASS
    if top_p < 1.0 and abs(got - next_l) <= 1e-5:   # stopped one later: it saw the oracle's prefix fall short
        return c_at - top_p <= TIE_MASS
    return False


@pytest.mark.parametrize("case", ["llama3b_t10", "longstream_262144"])
def test_filtered_estimators_match_the_stored_oracle_values(case):
    path = os.path.join(GOLDEN, f"filtered_{case}.npz")
    if not os.path.exists(path):
        pytest.skip(f"{os.path.basename(path)} has not been generated (tests/golden/make_filtered_golden.py {case})")
    g = np.load(path)
    full = np.load(os.path.join(GOLDEN, f"full_{str(g['case'])}.npz"))
    w = wl.WORKLOADS[str(full["workload"])]
    if int(full["T"]) != w.T:
        w = wl.with_T(w, int(full["T"]))
    inp = wl.make_inputs(w)
    dev = Device(inp.h, inp.W, inp.seeds, inp.positions)
    rows = g["rows"].astype(np.int64)
    assert np.array_equal(rows, full["rows"][g["index"]])
    temperature, eps = float(g["temperature"]), float(g["eps"])
    tok_gm = np.zeros(w.T, dtype=np.int32)
    tok_gm[rows] = g["tokens_gm"]
    tok_ipt = np.zeros(w.T, dtype=np.int32)
    tok_ipt[rows] = g["tokens_ipt"]
    workspace = torch.empty(difr.difr_filtered_workspace_bytes(w.T, w.d, w.V), dtype=torch.uint8, device="cuda")

    def call(fn, tokens, sigma, top_k, top_p, min_p, s=None):
        out = difr.DifrOut.allocate(w.T, w.d, w.V, sigma, eps)
        out.workspace = workspace
        out.cutoff = torch.full((w.T,), float("nan"), dtype=torch.float32, device="cuda")
        args = (dev.h, dev.W, to_dev(tokens), dev.seeds, dev.positions, temperature, top_k, top_p)
        if s is None:
            fn(*args, out, min_p=min_p)
        else:
            fn(*args, s, out, min_p=min_p)
        torch.cuda.synchronize()
        assert int(out.device_status.item()) == 0
        return out

    for j, (top_k, top_p, min_p, s) in enumerate(g["policies"]):
        top_k, s = int(top_k), int(s)
        top_p, min_p = float(np.float32(top_p)), float(np.float32(min_p))
        near, bar = g[f"near_{j}"], g[f"min_p_bar_{j}"]
        out = call(difr.difr_score_gm_filtered, tok_gm, float(g["sigma_gm"]), top_k, top_p, min_p, s)
        got, cut = out.score.cpu().numpy()[rows], out.cutoff.cpu().numpy().astype(np.float64)[rows]
        status = out.row_status.cpu().numpy()
        assert np.all(status & (4 | 8 | 16) == 0), f"policy {j}"
        ok = [_cutoff_ok(cut[i], g[f"gm_cutoff_{j}"][i], near[i], top_p, bar[i]) for i in range(len(rows))]
        assert all(ok), (j, np.nonzero(~np.array(ok))[0])
        worst = np.max(np.abs(got - g[f"gm_score_{j}"]))
        assert worst <= SCORE_TOL, f"policy {j}: max |score - oracle| = {worst}"
        whole = out.score.cpu().numpy()
        assert np.all(np.isfinite(whole)) and np.all(whole <= 1e-6)

        o2 = call(difr.difr_score_ipt_filtered, tok_ipt, float(g["sigma_ipt"]), top_k, top_p, min_p)
        assert np.all(o2.row_status.cpu().numpy() & (8 | 16) == 0), f"policy {j}"
        cut2 = o2.cutoff.cpu().numpy().astype(np.float64)[rows]
        want_cut = g[f"ipt_cutoff_{j}"]
        same = np.isclose(cut2, want_cut, rtol=0, atol=1e-5) | (np.isneginf(cut2) & np.isneginf(want_cut))
        ok2 = [bool(same[i]) or _cutoff_ok(cut2[i], want_cut[i], near[i], top_p, bar[i]) for i in range(len(rows))]
        if min_p == 0.0:
            assert all(ok2), (j, np.nonzero(~np.array(ok2))[0])
        assert same.mean() > 0.7   # (a flat head's nucleus ends where neighbouring ids are 1e-5 of the mass apart)
        # where the kept set is the oracle's, so are the probabilities and the score
        np.testing.assert_allclose(o2.score.cpu().numpy()[rows][same], g[f"ipt_score_{j}"][same], rtol=0,
                                   atol=SCORE_TOL, err_msg=f"policy {j}")
        np.testing.assert_allclose(o2.p_claimed.cpu().numpy()[rows][same], g[f"ipt_p_{j}"][same], rtol=2e-4, atol=1e-9)
        # (min-p: an id whose logit lies within fp32 rounding of the bound is kept by one side and not by the other;
        # on this flat head one row in ten has such an id, and its mass, at most min_p of the largest, moves `a`)
        np.testing.assert_allclose(o2.cdf_lo.cpu().numpy()[rows][same], g[f"ipt_a_{j}"][same], rtol=0,
                                   atol=2e-5 if min_p == 0.0 else 2e-4, err_msg=f"policy {j}")
