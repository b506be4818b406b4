"""GPU-vs-oracle parity of the full Token-DiFR estimator (top-k / top-p cutoff, B_i terms, s competitors)."""
import math

import numpy as np
import pytest
import torch

import oracle
import workloads as wl
from gpu_util import Device, f32, to_dev
from oracle import filtered

import paper_2511_02620_b200 as difr

pytestmark = pytest.mark.gpu

EPS = 1e-12
SCORE_TOL = 2e-3


def _small(T, d, V, seed, scale=1.0):
    g = np.random.default_rng(seed)
    h = wl.f32_to_bf16_bits(g.standard_normal((T, d)).astype(np.float32))
    W = wl.f32_to_bf16_bits((scale * g.standard_normal((V, d)) / math.sqrt(d)).astype(np.float32))
    seeds = np.array([wl.splitmix64(seed * 1000 + r // 64) for r in range(T)], dtype=np.uint64)
    positions = (np.arange(T) % 64 + 1).astype(np.uint32)
    return h, W, seeds, positions


def _claims(h, W, seeds, positions, temperature, seed):
    honest, runner = oracle.sample_gm(h, W, seeds, positions, temperature)
    L = oracle.logits(h, W)
    g = np.random.default_rng(seed)
    T, V = h.shape[0], W.shape[0]
    tokens = honest.copy()
    k = np.arange(T)
    tokens[k % 6 == 1] = runner[k % 6 == 1]
    tokens[k % 6 == 3] = g.integers(0, V, size=T)[k % 6 == 3]
    third = np.argsort(-L, axis=1)[:, 2]  # a high-logit id that was not sampled
    tokens[k % 6 == 5] = third[k % 6 == 5]
    return tokens.astype(np.int32)


def _run(dev, tokens, temperature, sigma, top_k, top_p, s):
    out = difr.DifrOut.allocate(dev.T, dev.d, dev.V, sigma, EPS)
    out.workspace = torch.empty(difr.difr_filtered_workspace_bytes(dev.T, dev.d, dev.V), dtype=torch.uint8, device="cuda")
    out.cutoff = torch.full((dev.T,), float("nan"), dtype=torch.float32, device="cuda")
    out.rank = torch.full((dev.T,), -5, dtype=torch.int32, device="cuda")
    out.score.fill_(float("nan"))
    difr.difr_score_gm_filtered(dev.h, dev.W, to_dev(np.asarray(tokens, dtype=np.int32)), dev.seeds, dev.positions,
                                f32(temperature), top_k, top_p, s, out)
    torch.cuda.synchronize()
    assert int(out.device_status.item()) == 0
    return out


def test_one_competitor_and_no_filter_is_the_plain_estimator():
    T, d, V = 200, 64, 3000
    h, W, seeds, positions = _small(T, d, V, 51)
    tokens = _claims(h, W, seeds, positions, f32(1.0), 52)
    tokens[9] = -3
    dev = Device(h, W, seeds, positions)
    for sigma in (0.5, 0.05):
        plain = dev.score("gm", tokens, 1.0, sigma, EPS)
        out = _run(dev, tokens, 1.0, sigma, 0, 1.0, 1)
        np.testing.assert_allclose(out.score.cpu().numpy(), plain["score"], rtol=0, atol=2e-5)
        assert np.all(np.isneginf(out.cutoff.cpu().numpy()))
        assert np.array_equal(out.argmax.cpu().numpy(), plain["argmax"])
        assert np.array_equal(out.row_status.cpu().numpy(), plain["row_status"])


@pytest.mark.parametrize("T,d,V,scale,temperature,sigma,top_k,top_p,s", [
    (96, 64, 3000, 2.0, 1.0, 0.3, 50, 0.95, 4),     # the paper's sampling setting; every id is a candidate (V < 16384)
    (96, 64, 3000, 2.0, 0.7, 0.05, 8, 1.0, 2),      # top-k only, narrow noise
    (64, 72, 20000, 3.0, 1.0, 0.5, 20, 0.9, 8),     # candidate lists bounded from the first pass (V >= 16384)
    (64, 72, 20000, 1.0, 1.0, 1.0, 0, 1.0, 8),      # no filter, many competitors, flat logits
    (64, 72, 20000, 3.0, 1.0, 0.3, 100, 0.98, 3),   # a top-k and a nucleus beyond 64 ids
    (48, 64, 9000, 2.0, 1.0, 0.3, 128, 1.0, 2),     # the largest top-k
    (40, 64, 40, 2.0, 1.0, 0.4, 64, 0.8, 3),        # top_k beyond the vocabulary: the nucleus acts on all of it
    (48, 64, 300000, 3.0, 1.0, 0.3, 50, 0.95, 4),   # more vocabulary tiles than 128 strips of eight: longer strips
])
def test_full_estimator_matches_the_oracle(T, d, V, scale, temperature, sigma, top_k, top_p, s):
    h, W, seeds, positions = _small(T, d, V, 61, scale)
    tokens = _claims(h, W, seeds, positions, f32(temperature), 62)
    tokens[5] = V + 1
    dev = Device(h, W, seeds, positions)
    out = _run(dev, tokens, temperature, sigma, top_k, top_p, s)
    want, pi, cut = filtered.score_gm_filtered(h, W, tokens, seeds, positions, f32(temperature), f32(sigma), f32(EPS),
                                               top_k, f32(top_p), s)
    got, got_cut = out.score.cpu().numpy(), out.cutoff.cpu().numpy().astype(np.float64)
    assert np.all(out.row_status.cpu().numpy() & 4 == 0)  # no candidate list overflowed
    # the cutoff is one of the row's logits: equal up to fp32 rounding, except where two prefixes of the nucleus
    # differ by less than rounding (then the neighbouring logit is as good an answer)
    same_cut = np.isclose(got_cut, cut, rtol=0, atol=1e-5) | (np.isneginf(got_cut) & np.isneginf(cut))
    assert same_cut.mean() >= 0.97
    np.testing.assert_allclose(got[same_cut], want[same_cut], rtol=0, atol=SCORE_TOL)
    assert got[5] == pytest.approx(math.log(EPS), abs=1e-5)
    # the raw-logit rank rides on the second pass: the very counts of the plain call's rank mode
    plain_out = difr.DifrOut.allocate(T, d, V, sigma, EPS)
    plain_out.rank = torch.full((T,), -5, dtype=torch.int32, device="cuda")
    difr.difr_score_gm(dev.h, dev.W, to_dev(tokens), dev.seeds, dev.positions, f32(temperature), plain_out)
    torch.cuda.synchronize()
    assert torch.equal(out.rank, plain_out.rank) and int(out.rank[5]) == V
    ref_rank = oracle.score_gm(h, W, tokens, seeds, positions, f32(temperature), f32(sigma), f32(EPS)).rank
    assert np.array_equal(out.rank.cpu().numpy(), ref_rank)
    # the estimate is not degenerate: the filter and the extra competitors move it
    if top_k or s > 1:
        plain = dev.score("gm", tokens, temperature, sigma, EPS)["score"]
        assert np.abs(got - plain).max() > 0.05


def test_full_estimator_at_full_size_on_sampled_rows():
    w = wl.WORKLOADS["llama3b"]
    inp = wl.make_inputs(w)
    dev = Device(inp.h, inp.W, inp.seeds, inp.positions)
    rows = wl.sample_rows(w, 12, salt=3)
    temperature, sigma, top_k, top_p, s = 1.0, 0.3, 50, 0.95, 4
    g = np.random.default_rng(5)
    tokens = g.integers(0, w.V, size=w.T).astype(np.int32)
    hs = np.ascontiguousarray(inp.h[rows])
    tokens[rows] = _claims(hs, inp.W, inp.seeds[rows], inp.positions[rows], f32(temperature), 6)
    out = _run(dev, tokens, temperature, sigma, top_k, top_p, s)
    want, _, cut = filtered.score_gm_filtered(hs, inp.W, tokens[rows], inp.seeds[rows], inp.positions[rows],
                                              f32(temperature), f32(sigma), f32(EPS), top_k, f32(top_p), s)
    got, got_cut = out.score.cpu().numpy(), out.cutoff.cpu().numpy()
    np.testing.assert_allclose(got_cut[rows], cut, rtol=0, atol=1e-5)
    np.testing.assert_allclose(got[rows], want, rtol=0, atol=SCORE_TOL)
    assert np.all(out.row_status.cpu().numpy() == 0)
    assert np.all(np.isfinite(got)) and np.all(got <= 1e-6)
    # the rank counted by the second pass: the oracle's on the sampled rows
    ref_rank = oracle.score_gm(hs, inp.W, tokens[rows], inp.seeds[rows], inp.positions[rows], f32(temperature),
                               f32(sigma), f32(EPS)).rank
    got_rank = out.rank.cpu().numpy()
    assert np.array_equal(got_rank[rows], ref_rank)
    assert got_rank.min() >= 0 and got_rank.max() < w.V


def test_results_do_not_depend_on_the_order_work_is_handed_out():
    """Work units are taken on demand and candidates are appended with atomics, so the order of work differs from
    launch to launch; the results must not."""
    T, d, V = 700, 128, 9000
    h, W, seeds, positions = _small(T, d, V, 81, 2.0)
    tokens = _claims(h, W, seeds, positions, f32(1.0), 82)
    dev = Device(h, W, seeds, positions)
    first = _run(dev, tokens, 1.0, 0.3, 50, 0.95, 4)
    keep = {k: getattr(first, k).clone() for k in ("score", "cutoff", "margin", "argmax", "runner_up", "lse")}
    for _ in range(3):
        again = _run(dev, tokens, 1.0, 0.3, 50, 0.95, 4)
        for k, v in keep.items():
            assert torch.equal(getattr(again, k), v, ) or (k in ("score", "cutoff", "margin", "lse")
                                                            and torch.equal(torch.isnan(getattr(again, k)), torch.isnan(v))
                                                            and torch.equal(torch.nan_to_num(getattr(again, k)), torch.nan_to_num(v))), k
    plain = [dev.score("gm", tokens, 1.0, 0.3, EPS) for _ in range(3)]
    for other in plain[1:]:
        for k in ("score", "margin", "argmax", "runner_up", "lse"):
            assert np.array_equal(plain[0][k], other[k], equal_nan=True) if plain[0][k].dtype.kind == "f" else \
                np.array_equal(plain[0][k], other[k]), k


@pytest.mark.parametrize("T,d,V,scale,temperature,sigma,top_k,top_p", [
    (96, 64, 3000, 2.0, 1.0, 0.1, 50, 0.95),
    (80, 72, 20000, 3.0, 0.7, 0.05, 20, 0.9),
    (64, 64, 20000, 1.0, 1.0, 1.0, 64, 1.0),
    (64, 64, 50000, 1.0, 1.0, 0.3, 128, 0.9),   # flat logits and the largest top-k: the longest lists
    (40, 64, 40, 2.0, 1.3, 0.2, 64, 0.8),
])
def test_ipt_estimator_under_the_filter_matches_the_oracle(T, d, V, scale, temperature, sigma, top_k, top_p):
    h, W, seeds, positions = _small(T, d, V, 91, scale)
    L = oracle.logits(h, W)
    mu = np.array([oracle.ipt_uniform(int(s), int(p)) for s, p in zip(seeds, positions)])
    tokens = np.array([filtered.ipt_sample_filtered(L[r], f32(temperature), top_k, f32(top_p), mu[r]) for r in range(T)],
                      dtype=np.int32)                                    # honest claims of the filtered sampler
    k = np.arange(T)
    tokens[k % 5 == 1] = np.argsort(-L, axis=1)[k % 5 == 1, 1]           # a likely id that was not drawn
    tokens[k % 5 == 3] = np.argmin(L, axis=1)[k % 5 == 3]                # an id the filter removes
    tokens[7] = V + 3
    dev = Device(h, W, seeds, positions)
    out = difr.DifrOut.allocate(T, d, V, sigma, EPS)
    out.workspace = torch.empty(difr.difr_filtered_workspace_bytes(T, d, V), dtype=torch.uint8, device="cuda")
    out.cutoff = torch.full((T,), float("nan"), dtype=torch.float32, device="cuda")
    for name in ("score", "p_claimed", "cdf_lo", "u"):
        getattr(out, name).fill_(float("nan"))
    difr.difr_score_ipt_filtered(dev.h, dev.W, to_dev(tokens), dev.seeds, dev.positions, f32(temperature), top_k, top_p, out)
    torch.cuda.synchronize()
    assert int(out.device_status.item()) == 0
    want, pt, a, mu_ref, cut = filtered.score_ipt_filtered(h, W, tokens, seeds, positions, f32(temperature), f32(sigma),
                                                           f32(EPS), top_k, f32(top_p))
    got = out.score.cpu().numpy()
    got_cut = out.cutoff.cpu().numpy().astype(np.float64)
    same_cut = np.isclose(got_cut, cut, rtol=0, atol=1e-5)
    assert same_cut.mean() >= 0.97
    ok = same_cut & (np.arange(T) != 7)
    np.testing.assert_allclose(got[ok], want[ok], rtol=0, atol=SCORE_TOL)
    np.testing.assert_allclose(out.p_claimed.cpu().numpy()[ok], pt[ok], rtol=2e-4, atol=1e-9)
    np.testing.assert_allclose(out.cdf_lo.cpu().numpy()[ok], a[ok], rtol=2e-4, atol=2e-6)
    np.testing.assert_allclose(out.u.cpu().numpy(), mu_ref, rtol=0, atol=1e-7)
    assert got[7] == pytest.approx(math.log(EPS), abs=1e-5)
    removed = ok & (k % 5 == 3) & (pt == 0.0)
    assert removed.sum() > 3 and np.allclose(got[removed], math.log(EPS), atol=1e-5)
    assert np.all(out.row_status.cpu().numpy() & 4 == 0)


def _nucleus_sizes(h, W, temperature, top_p):
    """Per row: how many ids the nucleus over the whole vocabulary keeps, and by how much (in mass) the prefix
    one shorter / the kept prefix misses / passes top_p (the distance of the decision from a tie)."""
    L = oracle.logits(h, W)
    sizes, slack = [], []
    for l in L:
        z = np.sort(l)[::-1] / temperature
        c = np.cumsum(np.exp(z - z[0]))
        c /= c[-1]
        n = int(np.searchsorted(c, top_p, side="left")) + 1
        sizes.append(n)
        near = [abs(c[n - 1] - top_p)] + ([abs(c[n - 2] - top_p)] if n >= 2 else [])
        if len(c) >= 128:
            near.append(abs(c[127] - top_p))
        slack.append(min(near))
    return np.array(sizes), np.array(slack)


@pytest.mark.parametrize("T,d,V,scale,temperature,sigma,top_p,s", [
    (96, 72, 20000, 4.0, 1.0, 0.3, 0.9, 4),   # peaked rows: most nuclei hold a handful of ids, some more than 128
    (96, 64, 3000, 3.0, 0.9, 0.1, 0.85, 2),   # every id is a candidate (V < 16384)
    (40, 64, 40, 2.0, 1.0, 0.4, 0.8, 3),      # the whole vocabulary is resolved: never flagged
])
def test_nucleus_over_the_whole_vocabulary(T, d, V, scale, temperature, sigma, top_p, s):
    """top_k = 0 with top_p < 1 given per row: the nucleus takes its mass from the whole row and is resolved among
    the row's 128 largest logits.  Rows whose nucleus fits agree with the oracle; the others carry row_status bit 4
    and the 128th largest logit as cutoff.  (With one policy for the call the selection path resolves any size:
    test_filters_of_any_size_match_the_oracle.)"""
    h, W, seeds, positions = _small(T, d, V, 71, scale)
    tokens = _claims(h, W, seeds, positions, f32(temperature), 72)
    dev = Device(h, W, seeds, positions)
    sizes, slack = _nucleus_sizes(h, W, f32(temperature), f32(top_p))
    clear = slack > 1e-4                      # the kernel's mass comes from fp32 sums: leave near-ties out
    fits = sizes <= min(128, V)
    assert fits.sum() >= 10 and (V <= 128 or (~fits).sum() >= 3)
    L = oracle.logits(h, W)
    kth = np.sort(L, axis=1)[:, ::-1][:, min(128, V) - 1]

    k_rows = torch.zeros(T, dtype=torch.int32, device="cuda")
    p_rows = torch.full((T,), top_p, dtype=torch.float32, device="cuda")
    out = _run(dev, tokens, temperature, sigma, k_rows, p_rows, s)
    flagged = (out.row_status.cpu().numpy() & 16) != 0
    assert np.array_equal(flagged[clear], ~fits[clear])
    want, _, cut = filtered.score_gm_filtered(h, W, tokens, seeds, positions, f32(temperature), f32(sigma), f32(EPS),
                                              0, f32(top_p), s)
    got, got_cut = out.score.cpu().numpy(), out.cutoff.cpu().numpy().astype(np.float64)
    ok = clear & fits
    np.testing.assert_allclose(got_cut[ok], cut[ok], rtol=0, atol=1e-5)
    np.testing.assert_allclose(got[ok], want[ok], rtol=0, atol=SCORE_TOL)
    over = clear & ~fits
    np.testing.assert_allclose(got_cut[over], kth[over], rtol=0, atol=1e-5)

    # the IPT estimator under the same nucleus
    o2 = difr.DifrOut.allocate(T, d, V, 0.1, EPS)
    o2.workspace = torch.empty(difr.difr_filtered_workspace_bytes(T, d, V), dtype=torch.uint8, device="cuda")
    o2.cutoff = torch.full((T,), float("nan"), dtype=torch.float32, device="cuda")
    difr.difr_score_ipt_filtered(dev.h, dev.W, to_dev(tokens), dev.seeds, dev.positions, f32(temperature), k_rows, p_rows, o2)
    torch.cuda.synchronize()
    assert int(o2.device_status.item()) == 0
    want2, pt, a, _, cut2 = filtered.score_ipt_filtered(h, W, tokens, seeds, positions, f32(temperature), f32(0.1),
                                                        f32(EPS), 0, f32(top_p))
    flagged2 = (o2.row_status.cpu().numpy() & 16) != 0
    assert np.array_equal(flagged2[clear], ~fits[clear])
    np.testing.assert_allclose(o2.cutoff.cpu().numpy()[ok], cut2[ok], rtol=0, atol=1e-5)
    np.testing.assert_allclose(o2.score.cpu().numpy()[ok], want2[ok], rtol=0, atol=SCORE_TOL)
    np.testing.assert_allclose(o2.p_claimed.cpu().numpy()[ok], pt[ok], rtol=2e-4, atol=1e-9)
    np.testing.assert_allclose(o2.cdf_lo.cpu().numpy()[ok], a[ok], rtol=2e-4, atol=2e-6)


def test_one_sampling_policy_per_row():
    """Requests with their own temperature, top_k and top_p in one batch: every row equals, bit for bit, the row
    of a call that applies its policy to the whole batch; rows with unusable values are NaN and carry bit 3."""
    T, d, V, s, sigma = 96, 72, 9000, 3, 0.3
    h, W, seeds, positions = _small(T, d, V, 81, 4.0)
    tokens = _claims(h, W, seeds, positions, f32(1.0), 82)
    dev = Device(h, W, seeds, positions)
    policies = [(1.0, 50, 0.95), (0.7, 8, 1.0), (1.3, 0, 0.9), (1.0, 0, 1.0), (0.0, 50, 0.95), (1.0, 130, 0.9),
                (1.0, 20, 1.5)]
    valid = [0, 1, 2, 3]
    group = np.arange(T) % len(policies)
    temps = torch.tensor([policies[g][0] for g in group], dtype=torch.float32, device="cuda")
    ks = torch.tensor([policies[g][1] for g in group], dtype=torch.int32, device="cuda")
    ps = torch.tensor([policies[g][2] for g in group], dtype=torch.float32, device="cuda")
    tok_dev = to_dev(tokens)

    def fresh():
        out = difr.DifrOut.allocate(T, d, V, sigma, EPS)
        out.workspace = torch.empty(difr.difr_filtered_workspace_bytes(T, d, V), dtype=torch.uint8, device="cuda")
        out.cutoff = torch.full((T,), float("nan"), dtype=torch.float32, device="cuda")
        return out

    for fn, extra in ((difr.difr_score_gm_filtered, (s,)), (difr.difr_score_ipt_filtered, ())):
        mixed = fresh()
        mixed.temperatures = temps
        fn(dev.h, dev.W, tok_dev, dev.seeds, dev.positions, 1.0, ks, ps, *extra, mixed)
        torch.cuda.synchronize()
        assert int(mixed.device_status.item()) == 0
        got, cut, st = mixed.score.cpu().numpy(), mixed.cutoff.cpu().numpy(), mixed.row_status.cpu().numpy()
        for g in valid:
            temp, k, p = policies[g]
            rows = group == g
            if fn is difr.difr_score_ipt_filtered and k == 0 and p == 1.0:
                # a row whose policy filters nothing keeps the unfiltered score
                ref = dev.score("ipt", tokens, temp, sigma, EPS)["score"]
                # (up to the last digits: the plain call also swaps the claimed token's fp32 softmax term for
                # the fp64 one, the filtered call's first pass keeps another statistic in that record word)
                np.testing.assert_allclose(got[rows], ref[rows], rtol=0, atol=2e-5)
                assert np.all(np.isneginf(cut[rows]))
                continue
            one = fresh()  # the same policy for every row, given per row like the mixed call's
            k_all = torch.full((T,), k, dtype=torch.int32, device="cuda")
            p_all = torch.full((T,), p, dtype=torch.float32, device="cuda")
            fn(dev.h, dev.W, tok_dev, dev.seeds, dev.positions, f32(temp), k_all, p_all, *extra, one)
            torch.cuda.synchronize()
            assert np.array_equal(got[rows], one.score.cpu().numpy()[rows], equal_nan=True), (fn.__name__, g)
            assert np.array_equal(cut[rows], one.cutoff.cpu().numpy()[rows], equal_nan=True), (fn.__name__, g)
            assert np.all(np.isfinite(got[rows])) and np.all(st[rows] & 8 == 0)
        bad = group >= len(valid)
        assert np.all(np.isnan(got[bad])) and np.all(st[bad] & 8 != 0)
        # the policies differ where they should: the same claims score differently under different filters
        assert np.unique(np.round(cut[~bad & np.isfinite(cut)], 3)).size > 10


@pytest.mark.parametrize("T,d,V,scale,temperature,sigma,top_k,top_p,min_p,s", [
    (96, 72, 20000, 4.0, 1.0, 0.3, 0, 1.0, 0.05, 3),     # min-p alone (the largest logit is all the filter needs)
    (96, 64, 3000, 3.0, 0.8, 0.05, 0, 1.0, 0.3, 2),      # every id is a candidate (V < 16384), a strict bar
    (64, 72, 20000, 4.0, 1.0, 0.3, 50, 0.95, 0.02, 4),   # behind top-k and top-p: the stricter bound decides
    (64, 72, 20000, 2.0, 1.2, 0.5, 100, 1.0, 0.2, 1),
])
def test_min_p_filter_matches_the_oracle(T, d, V, scale, temperature, sigma, top_k, top_p, min_p, s):
    """min-p keeps the ids whose probability is at least min_p times the largest: the cutoff is the larger of the
    top-k / top-p cutoff and l_max + Temp ln(min_p), with l_max re-evaluated in fp64."""
    h, W, seeds, positions = _small(T, d, V, 93, scale)
    tokens = _claims(h, W, seeds, positions, f32(temperature), 94)
    tokens[5] = V + 1
    dev = Device(h, W, seeds, positions)
    out = difr.DifrOut.allocate(T, d, V, sigma, EPS)
    out.workspace = torch.empty(difr.difr_filtered_workspace_bytes(T, d, V), dtype=torch.uint8, device="cuda")
    out.cutoff = torch.full((T,), float("nan"), dtype=torch.float32, device="cuda")
    out.score.fill_(float("nan"))
    difr.difr_score_gm_filtered(dev.h, dev.W, to_dev(tokens), dev.seeds, dev.positions, f32(temperature), top_k, top_p,
                                s, out, min_p=f32(min_p))
    torch.cuda.synchronize()
    assert int(out.device_status.item()) == 0
    want, _, cut = filtered.score_gm_filtered(h, W, tokens, seeds, positions, f32(temperature), f32(sigma), f32(EPS),
                                              top_k, f32(top_p), s, f32(min_p))
    got, got_cut = out.score.cpu().numpy(), out.cutoff.cpu().numpy().astype(np.float64)
    same_cut = np.isclose(got_cut, cut, rtol=0, atol=1e-5)
    assert same_cut.mean() >= 0.97
    np.testing.assert_allclose(got[same_cut], want[same_cut], rtol=0, atol=SCORE_TOL)
    assert got[5] == pytest.approx(math.log(EPS), abs=1e-5)
    # the bar really is the binding part of the filter on some rows, and the rank filter on others (when both act)
    L = oracle.logits(h, W)
    bar = L.max(axis=1) + f32(temperature) * math.log(f32(min_p))
    assert np.isclose(cut, bar, atol=1e-9).sum() > 5
    if top_k and top_p < 1.0:
        assert (~np.isclose(cut, bar, atol=1e-9)).sum() > 5
    # without min-p the same call gives other scores
    plain = _run(dev, tokens, temperature, sigma, top_k, top_p, s).score.cpu().numpy()
    assert np.abs(plain - got)[np.isfinite(plain)].max() > 0.01


@pytest.mark.parametrize("T,d,V,scale,temperature,sigma,top_k,top_p,min_p", [
    (96, 72, 20000, 5.0, 1.0, 0.1, 0, 1.0, 0.05),    # min-p alone: the survivors are found among the 128 largest logits
    (80, 64, 3000, 4.0, 0.8, 0.05, 40, 0.9, 0.1),
    (40, 64, 40, 2.0, 1.0, 0.2, 0, 1.0, 0.3),
])
def test_ipt_estimator_under_min_p_matches_the_oracle(T, d, V, scale, temperature, sigma, top_k, top_p, min_p):
    h, W, seeds, positions = _small(T, d, V, 95, scale)
    L = oracle.logits(h, W)
    mu = np.array([oracle.ipt_uniform(int(s), int(p)) for s, p in zip(seeds, positions)])
    tokens = np.array([filtered.ipt_sample_filtered(L[r], f32(temperature), top_k, f32(top_p), mu[r], f32(min_p))
                       for r in range(T)], dtype=np.int32)
    k = np.arange(T)
    tokens[k % 5 == 1] = np.argsort(-L, axis=1)[k % 5 == 1, 1]
    tokens[k % 5 == 3] = np.argmin(L, axis=1)[k % 5 == 3]
    dev = Device(h, W, seeds, positions)
    out = difr.DifrOut.allocate(T, d, V, sigma, EPS)
    out.workspace = torch.empty(difr.difr_filtered_workspace_bytes(T, d, V), dtype=torch.uint8, device="cuda")
    out.cutoff = torch.full((T,), float("nan"), dtype=torch.float32, device="cuda")
    difr.difr_score_ipt_filtered(dev.h, dev.W, to_dev(tokens), dev.seeds, dev.positions, f32(temperature), top_k, top_p,
                                 out, min_p=f32(min_p))
    torch.cuda.synchronize()
    assert int(out.device_status.item()) == 0
    want, pt, a, _, cut = filtered.score_ipt_filtered(h, W, tokens, seeds, positions, f32(temperature), f32(sigma),
                                                      f32(EPS), top_k, f32(top_p), f32(min_p))
    n_kept = np.array([len(filtered.filter_kept(L[r], f32(temperature), top_k, f32(top_p), f32(min_p)))
                       for r in range(T)])
    status = out.row_status.cpu().numpy()
    resolved = n_kept < min(128, V) if not top_k else np.ones(T, dtype=bool)
    assert resolved.sum() >= T // 2
    assert np.all(status[resolved] & 16 == 0)
    got_cut = out.cutoff.cpu().numpy().astype(np.float64)
    ok = resolved & np.isclose(got_cut, cut, rtol=0, atol=1e-5)
    assert ok.sum() >= 0.95 * resolved.sum()
    np.testing.assert_allclose(out.score.cpu().numpy()[ok], want[ok], rtol=0, atol=SCORE_TOL)
    np.testing.assert_allclose(out.p_claimed.cpu().numpy()[ok], pt[ok], rtol=2e-4, atol=1e-9)
    np.testing.assert_allclose(out.cdf_lo.cpu().numpy()[ok], a[ok], rtol=2e-4, atol=2e-6)
    assert (n_kept[resolved] > 1).sum() > 5  # the bar keeps more than the top id on some rows


def _filtered_call(fn, dev, tokens, temperature, sigma, top_k, top_p, min_p, s=None):
    T, d, V = dev.T, dev.d, dev.V
    out = difr.DifrOut.allocate(T, d, V, sigma, EPS)
    out.workspace = torch.empty(difr.difr_filtered_workspace_bytes(T, d, V), dtype=torch.uint8, device="cuda")
    out.cutoff = torch.full((T,), float("nan"), dtype=torch.float32, device="cuda")
    for name in ("score", "p_claimed", "cdf_lo", "u"):
        getattr(out, name).fill_(float("nan"))
    args = (dev.h, dev.W, to_dev(np.asarray(tokens, dtype=np.int32)), dev.seeds, dev.positions, f32(temperature),
            top_k, top_p)
    if s is None:
        fn(*args, out, min_p=f32(min_p))
    else:
        fn(*args, s, out, min_p=f32(min_p))
    torch.cuda.synchronize()
    assert int(out.device_status.item()) == 0
    return out


def _cutoff_agrees(l_row, temperature, top_k, top_p, min_p, got_cut, want_cut, tol_mass=3e-5):
    """The kernel's cutoff is the oracle's, or the logit at a neighbouring position of the sorted row where the
    nucleus decision "does this prefix hold top_p of the mass" lies within tol_mass of a tie (the kernel sums
    masses of fp32 logits).  Returns (acceptable, identical)."""
    if (np.isneginf(got_cut) and np.isneginf(want_cut)) or abs(got_cut - want_cut) <= 1e-5:
        return True, True
    if not top_p < 1.0:
        return False, False
    V = l_row.shape[0]
    z = np.sort(l_row)[::-1]
    k = top_k if 0 < top_k < V else V
    e = np.exp((z[:k] - z[0]) / temperature)
    c = np.cumsum(e) / e.sum()
    q = int(np.argmin(np.abs(z[:k] - got_cut)))
    if abs(z[q] - got_cut) > 1e-5:
        return False, False
    n = int(np.searchsorted(c, top_p, side="left")) + 1
    if q + 1 < n:   # the kernel stopped earlier: it saw the mass of its prefix reach top_p
        return bool(top_p - c[q] <= tol_mass), False
    return bool(c[q - 1] - top_p <= tol_mass), False   # it stopped later: it saw the shorter prefix fall short


@pytest.mark.parametrize("T,d,V,scale,temperature,sigma,top_k,top_p,min_p,s", [
    (64, 72, 20000, 1.0, 1.0, 0.3, 0, 0.95, 0.0, 3),      # flat logits: the nucleus holds most of the vocabulary
    (64, 72, 20000, 3.0, 1.0, 0.3, 0, 0.9, 0.0, 2),       # peaked rows: nuclei from a handful to thousands of ids
    (48, 64, 9000, 2.0, 0.8, 0.1, 1000, 1.0, 0.0, 4),     # a top-k above the lists' reach
    (48, 64, 9000, 2.0, 1.0, 0.3, 2000, 0.9, 0.0, 2),     # both: the nucleus inside a large top-k
    (48, 64, 9000, 2.0, 1.0, 0.3, 500, 0.97, 0.05, 2),    # ... with a min-p bound behind them
    (40, 64, 300, 2.0, 1.0, 0.4, 200, 0.9, 0.0, 3),       # one vocabulary tile, ragged
])
def test_filters_of_any_size_match_the_oracle(T, d, V, scale, temperature, sigma, top_k, top_p, min_p, s):
    """One policy for the whole call with a kept set beyond the candidate lists (top_k > 128, a nucleus over the
    whole vocabulary): the kept prefix is found by selection over the rows' logits.  The cutoff is the oracle's
    (or its neighbour in the sorted row where the nucleus decision is within 3e-5 of a tie in relative mass),
    the score the oracle's on every row."""
    h, W, seeds, positions = _small(T, d, V, 97, scale)
    tokens = _claims(h, W, seeds, positions, f32(temperature), 98)
    tokens[5] = V + 1
    dev = Device(h, W, seeds, positions)
    out = _filtered_call(difr.difr_score_gm_filtered, dev, tokens, temperature, sigma, top_k, top_p, min_p, s)
    want, _, cut = filtered.score_gm_filtered(h, W, tokens, seeds, positions, f32(temperature), f32(sigma), f32(EPS),
                                              top_k, f32(top_p), s, f32(min_p))
    L = oracle.logits(h, W)
    got, got_cut = out.score.cpu().numpy(), out.cutoff.cpu().numpy().astype(np.float64)
    status = out.row_status.cpu().numpy()
    assert np.all(status & (4 | 8 | 16) == 0)  # nothing unresolved, nothing overflowed
    bar = L.max(axis=1) + f32(temperature) * math.log(f32(min_p)) if min_p > 0 else np.full(T, -np.inf)
    agree = [_cutoff_agrees(L[r], f32(temperature), top_k, f32(top_p), f32(min_p), max(got_cut[r], -np.inf),
                            cut[r]) if not (min_p > 0 and np.isclose(cut[r], bar[r], atol=1e-9))
             else (bool(abs(got_cut[r] - cut[r]) <= 1e-5),) * 2 for r in range(T)]
    ok = np.array([a[0] for a in agree])
    same = np.array([a[1] for a in agree])
    assert ok.all(), np.nonzero(~ok)[0]
    assert same.mean() > 0.8
    np.testing.assert_allclose(got, want, rtol=0, atol=SCORE_TOL)
    assert got[5] == pytest.approx(math.log(EPS), abs=1e-5)
    # the kept sets really are large
    n_kept = np.array([len(filtered.filter_kept(L[r], f32(temperature), top_k, f32(top_p), f32(min_p))) for r in range(T)])
    assert n_kept.max() > 128 or V <= 300

    # Token-IPT-DiFR on the same filtered distribution
    mu = np.array([oracle.ipt_uniform(int(sd), int(ps)) for sd, ps in zip(seeds, positions)])
    tok2 = np.array([filtered.ipt_sample_filtered(L[r], f32(temperature), top_k, f32(top_p), mu[r], f32(min_p))
                     for r in range(T)], dtype=np.int32)
    k = np.arange(T)
    tok2[k % 5 == 1] = np.argsort(-L, axis=1)[k % 5 == 1, 1]
    tok2[k % 5 == 3] = np.argmin(L, axis=1)[k % 5 == 3]
    o2 = _filtered_call(difr.difr_score_ipt_filtered, dev, tok2, temperature, 0.1, top_k, top_p, min_p)
    want2, pt, a, _, cut2 = filtered.score_ipt_filtered(h, W, tok2, seeds, positions, f32(temperature), f32(0.1),
                                                        f32(EPS), top_k, f32(top_p), f32(min_p))
    assert np.all(o2.row_status.cpu().numpy() & (8 | 16) == 0)
    cut_ipt = o2.cutoff.cpu().numpy().astype(np.float64)
    same2 = np.isclose(cut_ipt, cut2, rtol=0, atol=1e-5)   # the same kept set (compared where it is)
    assert same2.mean() > 0.8
    np.testing.assert_allclose(o2.score.cpu().numpy()[same2], want2[same2], rtol=0, atol=SCORE_TOL)
    np.testing.assert_allclose(o2.p_claimed.cpu().numpy()[same2], pt[same2], rtol=2e-4, atol=1e-9)
    np.testing.assert_allclose(o2.cdf_lo.cpu().numpy()[same2], a[same2], rtol=2e-4, atol=2e-6)


def test_min_p_set_of_any_size_for_the_ipt_estimator():
    """min-p alone on flat logits keeps thousands of ids: with one policy for the call the IPT estimator's kept
    set is summed by the selection, none is left unresolved."""
    T, d, V, temperature, min_p = 64, 72, 20000, 1.0, 0.05
    h, W, seeds, positions = _small(T, d, V, 99, 1.0)
    L = oracle.logits(h, W)
    mu = np.array([oracle.ipt_uniform(int(sd), int(ps)) for sd, ps in zip(seeds, positions)])
    tokens = np.array([filtered.ipt_sample_filtered(L[r], f32(temperature), 0, 1.0, mu[r], f32(min_p)) for r in range(T)],
                      dtype=np.int32)
    tokens[::4] = np.argmin(L, axis=1)[::4]
    dev = Device(h, W, seeds, positions)
    out = _filtered_call(difr.difr_score_ipt_filtered, dev, tokens, temperature, 0.1, 0, 1.0, min_p)
    want, pt, a, _, cut = filtered.score_ipt_filtered(h, W, tokens, seeds, positions, f32(temperature), f32(0.1), f32(EPS),
                                                      0, 1.0, f32(min_p))
    n_kept = np.array([len(filtered.filter_kept(L[r], f32(temperature), 0, 1.0, f32(min_p))) for r in range(T)])
    assert n_kept.min() > 128
    # ids whose logit lies within fp32 rounding of the bound may fall on either side: leave those rows out
    bar = L.max(axis=1, keepdims=True) + f32(temperature) * math.log(f32(min_p))
    clear = np.abs(L - bar).min(axis=1) > 2e-5
    assert clear.mean() > 0.8
    assert np.all(out.row_status.cpu().numpy() & (8 | 16) == 0)
    np.testing.assert_allclose(out.cutoff.cpu().numpy()[clear], cut[clear], rtol=0, atol=1e-5)
    np.testing.assert_allclose(out.score.cpu().numpy()[clear], want[clear], rtol=0, atol=SCORE_TOL)
    np.testing.assert_allclose(out.cdf_lo.cpu().numpy()[clear], a[clear], rtol=2e-4, atol=2e-6)


def test_filters_of_any_size_at_full_size_on_sampled_rows():
    """llama3b at full size with the nucleus taken over the whole vocabulary (flat synthetic logits: it holds about
    three quarters of the ids) and with a top-k of 1000: the logits go through the selection three blocks of rows
    at a time; sampled rows against the oracle, twice (the results are the same bits on every run)."""
    w = wl.WORKLOADS["llama3b"]
    inp = wl.make_inputs(w)
    dev = Device(inp.h, inp.W, inp.seeds, inp.positions)
    rows = wl.sample_rows(w, 10, salt=4)
    temperature, sigma, s = 1.0, 0.3, 2
    g = np.random.default_rng(7)
    tokens = g.integers(0, w.V, size=w.T).astype(np.int32)
    hs = np.ascontiguousarray(inp.h[rows])
    tokens[rows] = _claims(hs, inp.W, inp.seeds[rows], inp.positions[rows], f32(temperature), 8)
    L = oracle.logits(hs, inp.W)
    for top_k, top_p in ((0, 0.95), (1000, 1.0)):
        out = _filtered_call(difr.difr_score_gm_filtered, dev, tokens, temperature, sigma, top_k, top_p, 0.0, s)
        again = _filtered_call(difr.difr_score_gm_filtered, dev, tokens, temperature, sigma, top_k, top_p, 0.0, s)
        assert torch.equal(out.score.view(torch.int32), again.score.view(torch.int32))
        assert torch.equal(out.cutoff.view(torch.int32), again.cutoff.view(torch.int32))
        want, _, cut = filtered.score_gm_filtered(hs, inp.W, tokens[rows], inp.seeds[rows], inp.positions[rows],
                                                  f32(temperature), f32(sigma), f32(EPS), top_k, f32(top_p), s)
        got, got_cut = out.score.cpu().numpy(), out.cutoff.cpu().numpy().astype(np.float64)
        for i, r in enumerate(rows):
            ok, _ = _cutoff_agrees(L[i], f32(temperature), top_k, f32(top_p), 0.0, got_cut[r], cut[i])
            assert ok, (top_k, top_p, int(r), got_cut[r], cut[i])
        np.testing.assert_allclose(got[rows], want, rtol=0, atol=SCORE_TOL)
        assert np.all(out.row_status.cpu().numpy() & (4 | 8 | 16) == 0)
        assert np.all(np.isfinite(got)) and np.all(got <= 1e-6)
        assert np.all(np.isfinite(got_cut))


def test_per_row_policies_of_any_size():
    """Requests with their own sampling parameters in one batch, some of them beyond the candidate lists' reach
    (a top-k of 700, a whole-vocabulary nucleus, min-p for the IPT estimator), some within it, some without a
    filter: with `any_size` every row is resolved by the selection and matches the oracle run on the rows of each
    policy by themselves."""
    T, d, V = 60, 64, 9000
    h, W, seeds, positions = _small(T, d, V, 131, 2.0)
    # (top_k, top_p, min_p, temperature)
    policies = [(700, 1.0, 0.0, 1.0), (0, 0.93, 0.0, 1.0), (40, 0.9, 0.0, 0.8), (0, 1.0, 0.0, 0.8),
                (1500, 0.95, 0.02, 1.0), (V, 1.0, 0.0, 1.0)]
    which = np.arange(T) % len(policies)
    k_rows = np.array([policies[w][0] for w in which], dtype=np.int32)
    p_rows = np.array([policies[w][1] for w in which], dtype=np.float32)
    m_rows = np.array([policies[w][2] for w in which], dtype=np.float32)
    t_rows = np.array([policies[w][3] for w in which], dtype=np.float32)
    dev = Device(h, W, seeds, positions)
    L = oracle.logits(h, W)
    sigma, s = 0.3, 3

    def call(fn, tokens, sig, s_arg=None):
        out = difr.DifrOut.allocate(T, d, V, sig, EPS)
        out.workspace = torch.empty(difr.difr_filtered_workspace_bytes(T, d, V), dtype=torch.uint8, device="cuda")
        out.cutoff = torch.full((T,), float("nan"), dtype=torch.float32, device="cuda")
        out.temperatures = to_dev(t_rows)
        args = (dev.h, dev.W, to_dev(tokens), dev.seeds, dev.positions, 1.0, to_dev(k_rows), to_dev(p_rows))
        if s_arg is None:
            fn(*args, out, min_p=to_dev(m_rows), any_size=True)
        else:
            fn(*args, s_arg, out, min_p=to_dev(m_rows), any_size=True)
        torch.cuda.synchronize()
        assert int(out.device_status.item()) == 0
        return out

    # Token-DiFR
    tokens = np.empty(T, dtype=np.int32)
    for w, (k, p, m, t) in enumerate(policies):
        rows = np.nonzero(which == w)[0]
        tokens[rows] = _claims(h[rows], W, seeds[rows], positions[rows], f32(t), 140 + w)
    out = call(difr.difr_score_gm_filtered, tokens, sigma, s)
    got, got_cut = out.score.cpu().numpy(), out.cutoff.cpu().numpy().astype(np.float64)
    assert np.all(out.row_status.cpu().numpy() & (4 | 8 | 16) == 0)
    for w, (k, p, m, t) in enumerate(policies):
        rows = np.nonzero(which == w)[0]
        want, _, cut = filtered.score_gm_filtered(h[rows], W, tokens[rows], seeds[rows], positions[rows], f32(t),
                                                  f32(sigma), f32(EPS), k, f32(p), s, f32(m))
        for j, r in enumerate(rows):
            bar = L[r].max() + f32(t) * math.log(f32(m)) if m > 0 else -np.inf
            if m > 0 and np.isclose(cut[j], bar, atol=1e-9):
                assert abs(got_cut[r] - cut[j]) <= 1e-5
            else:
                assert _cutoff_agrees(L[r], f32(t), k, f32(p), f32(m), got_cut[r], cut[j])[0], (w, r)
        np.testing.assert_allclose(got[rows], want, rtol=0, atol=SCORE_TOL, err_msg=f"policy {w}")

    # Token-IPT-DiFR on the rows' filtered distributions
    mu = np.array([oracle.ipt_uniform(int(sd), int(ps)) for sd, ps in zip(seeds, positions)])
    tok2 = np.array([filtered.ipt_sample_filtered(L[r], f32(t_rows[r]), int(k_rows[r]), f32(p_rows[r]), mu[r],
                                                  f32(m_rows[r])) for r in range(T)], dtype=np.int32)
    tok2[np.arange(T) % 7 == 2] = np.argsort(-L, axis=1)[np.arange(T) % 7 == 2, 1]
    o2 = call(difr.difr_score_ipt_filtered, tok2, 0.1)
    assert np.all(o2.row_status.cpu().numpy() & (8 | 16) == 0)
    cut_ipt = o2.cutoff.cpu().numpy().astype(np.float64)
    n_same = 0
    for w, (k, p, m, t) in enumerate(policies):
        rows = np.nonzero(which == w)[0]
        want2, pt, a, _, cut2 = filtered.score_ipt_filtered(h[rows], W, tok2[rows], seeds[rows], positions[rows],
                                                            f32(t), f32(0.1), f32(EPS), k, f32(p), f32(m))
        same = np.isclose(cut_ipt[rows], cut2, rtol=0, atol=1e-5) | (np.isneginf(cut_ipt[rows]) & np.isneginf(cut2))
        n_same += int(same.sum())
        np.testing.assert_allclose(o2.score.cpu().numpy()[rows][same], want2[same], rtol=0, atol=SCORE_TOL,
                                   err_msg=f"policy {w}")
        np.testing.assert_allclose(o2.p_claimed.cpu().numpy()[rows][same], pt[same], rtol=2e-4, atol=1e-9)
        np.testing.assert_allclose(o2.cdf_lo.cpu().numpy()[rows][same], a[same], rtol=0, atol=2e-5)
    assert n_same > 0.8 * T


@pytest.mark.parametrize("any_size", [False, True])
def test_calls_beyond_a_block_of_stored_logits_equal_their_blocks(any_size):
    """A filtered call with more rows than the workspace's block of stored logits holds (2 GiB: 4096 rows at
    V = 128256) is worked off block by block: every output equals, bit for bit, what separate calls on the row
    ranges give (per-row policies, temperatures, the rank and the cutoff all travel with their rows)."""
    d, V = 64, 128256
    block = ((2**31) // (4 * V)) & ~255
    T = block + 700
    g = np.random.default_rng(171)
    h = torch.from_numpy(g.standard_normal((T, d)).astype(np.float32)).cuda().to(torch.bfloat16)
    W = torch.from_numpy((g.standard_normal((V, d)) * (2.0 / math.sqrt(d))).astype(np.float32)).cuda().to(torch.bfloat16)
    tokens = to_dev(g.integers(0, V, size=T).astype(np.int32))
    seeds = to_dev(g.integers(1, 2**62, size=T).astype(np.int64))
    positions = to_dev((np.arange(T) % 512 + 1).astype(np.int32))
    k_rows = to_dev(np.where(np.arange(T) % 3 == 0, 40, 0).astype(np.int32))
    p_rows = to_dev(np.where(np.arange(T) % 2 == 0, 0.9, 1.0).astype(np.float32))
    m_rows = to_dev(np.where(np.arange(T) % 5 == 0, 0.01, 0.0).astype(np.float32))
    t_rows = to_dev(np.where(np.arange(T) % 4 == 0, 0.8, 1.0).astype(np.float32))

    def run(lo, hi):
        n = hi - lo
        out = difr.DifrOut.allocate(n, d, V, 0.3, EPS)
        out.workspace = torch.empty(difr.difr_filtered_workspace_bytes(n, d, V), dtype=torch.uint8, device="cuda")
        out.cutoff = torch.full((n,), float("nan"), dtype=torch.float32, device="cuda")
        out.rank = torch.full((n,), -7, dtype=torch.int32, device="cuda")
        out.temperatures = t_rows[lo:hi].contiguous()
        difr.difr_score_gm_filtered(h[lo:hi].contiguous(), W, tokens[lo:hi].contiguous(), seeds[lo:hi].contiguous(),
                                    positions[lo:hi].contiguous(), 1.0, k_rows[lo:hi].contiguous(),
                                    p_rows[lo:hi].contiguous(), 3, out, min_p=m_rows[lo:hi].contiguous(),
                                    any_size=any_size)
        torch.cuda.synchronize()
        assert int(out.device_status.item()) == 0
        return out

    whole, first, second = run(0, T), run(0, block), run(block, T)
    for name in ("score", "cutoff", "margin", "argmax", "runner_up", "lse", "rank", "row_status"):
        a = getattr(whole, name)
        b = torch.cat([getattr(first, name), getattr(second, name)])
        assert torch.equal(a.view(torch.int32), b.view(torch.int32)), name
    assert torch.isfinite(whole.score).all()
