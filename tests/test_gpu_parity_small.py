"""GPU-vs-oracle parity on shapes the oracle finishes in seconds: the library's
Philox, the tensor-core logits, both scores and detection, element by element."""
import math

import numpy as np
import pytest
import torch

import oracle
import workloads as wl
from gpu_util import SEQ_STATS_DTYPE, Device, f32, to_bf16, to_dev

import paper_2511_02620_b200 as difr

pytestmark = pytest.mark.gpu

SCORE_TOL = 2e-3  # absolute, on the log-scores
LSE_RTOL = 1e-3
ARGMAX_MARGIN = 1e-3  # ids may differ only where the oracle's top-2 margin is below this
EPS = 1e-12


def _small(T, d, V, seed):
    g = np.random.default_rng(seed)
    h = wl.f32_to_bf16_bits(g.standard_normal((T, d)).astype(np.float32))
    W = wl.f32_to_bf16_bits((g.standard_normal((V, d)) / math.sqrt(d)).astype(np.float32))
    seeds = np.array([wl.splitmix64(seed * 1000 + r // 64) for r in range(T)], dtype=np.uint64)
    positions = (np.arange(T) % 64 + 1).astype(np.uint32)
    return h, W, seeds, positions


def _claims(h, W, seeds, positions, temperature, seed, frac=0.1):
    """Honest Gumbel-max claims with a fraction replaced: half by the runner-up, half by a random id."""
    honest, runner = oracle.sample_gm(h, W, seeds, positions, temperature)
    g = np.random.default_rng(seed)
    T, V = h.shape[0], W.shape[0]
    tokens = honest.copy()
    bad = g.random(T) < frac
    use_runner = g.random(T) < 0.5
    rnd = g.integers(0, V, size=T)
    tokens[bad & use_runner] = runner[bad & use_runner]
    tokens[bad & ~use_runner] = rnd[bad & ~use_runner]
    return tokens.astype(np.int32)


def check_gm(got, ref, tol=SCORE_TOL):
    np.testing.assert_allclose(got["score"], ref.score, rtol=0, atol=tol)
    fin = np.isfinite(ref.margin)
    np.testing.assert_allclose(got["margin"][fin], ref.margin[fin], rtol=0, atol=1e-4)
    assert np.array_equal(np.signbit(got["margin"]), np.signbit(ref.margin))
    assert np.array_equal(got["margin"][~fin], ref.margin[~fin])
    clear = ref.top2_margin >= ARGMAX_MARGIN
    assert np.array_equal(got["argmax"][clear], ref.argmax[clear])
    clear2 = clear & (ref.top23_margin >= ARGMAX_MARGIN)  # the runner-up is unique where the third is clearly behind
    assert np.array_equal(got["runner_up"][clear2], ref.runner_up[clear2])
    assert clear2.mean() > 0.9
    np.testing.assert_allclose(got["lse"], ref.lse, rtol=LSE_RTOL, atol=1e-3)
    assert np.array_equal(got["row_status"], ref.row_status)


def test_library_philox_is_bit_exact():
    g = np.random.default_rng(1)
    n = 4096
    ctr = g.integers(0, 2**32, size=(n, 4), dtype=np.uint64).astype(np.uint32)
    ctr[: n // 2, 2:] = 0  # the form the scoring epilogue uses
    ctr[:64, 0] = np.arange(64)
    key = g.integers(0, 2**32, size=(n, 2), dtype=np.uint64).astype(np.uint32)
    out = torch.zeros((n, 4), dtype=torch.int32, device="cuda")
    difr.difr_philox(to_dev(ctr), to_dev(key), out)
    got = out.cpu().numpy().view(np.uint32)
    want = np.stack([oracle.philox4x32_10(ctr[i], key[i]) for i in range(n)])
    assert np.array_equal(got, want)


# (the stores of the logits are 32, 16 or 4 bytes wide by what V and the output's address allow: every width is met)
@pytest.mark.parametrize("T,d,V,offset", [(256, 512, 4096, 0), (200, 72, 1000, 0), (130, 64, 300, 0), (90, 64, 301, 0),
                                          (200, 72, 1000, 4), (200, 72, 1000, 1)])
def test_tensor_core_logits_match_fp64(T, d, V, offset):
    h, W, _, _ = _small(T, d, V, 2)
    flat = torch.full((T * V + 8,), float("nan"), dtype=torch.float32, device="cuda")
    logits = flat[offset:offset + T * V].view(T, V)  # `offset` floats past an allocation boundary
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    difr.difr_logits(to_bf16(h), to_bf16(W), logits, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    want = oracle.logits(h, W)
    np.testing.assert_allclose(logits.cpu().numpy(), want, rtol=0, atol=2e-5 * math.sqrt(d / 64))


@pytest.mark.parametrize("temperature", [1.0, 0.7])
@pytest.mark.parametrize("sigma", [1.0, 0.05])
def test_tiny_workload_gm(temperature, sigma):
    w = wl.WORKLOADS["tiny"]
    inp = wl.make_inputs(w)
    honest, runner = oracle.sample_gm(inp.h_server, inp.W, inp.seeds, inp.positions, f32(temperature))
    tokens, _ = wl.tamper(w, honest, runner)
    ref = oracle.score_gm(inp.h, inp.W, tokens, inp.seeds, inp.positions, f32(temperature), f32(sigma), f32(EPS))
    dev = Device(inp.h, inp.W, inp.seeds, inp.positions)
    check_gm(dev.score("gm", tokens, temperature, sigma, EPS), ref)


@pytest.mark.parametrize("T,d,V", [(300, 200, 1000), (129, 64, 257), (64, 328, 5000), (1, 8, 2),
                                   (40, 8192, 3000), (24, 16392, 1500)])  # wide heads: strips of two tiles, of one
def test_ragged_shapes_gm(T, d, V):
    """Several tiles with ragged tails in T, d (not a multiple of 64) and V (not a multiple of 256 or 32)."""
    h, W, seeds, positions = _small(T, d, V, 3)
    tokens = _claims(h, W, seeds, positions, f32(0.8), 4)
    if T >= 3:
        tokens[0] = -5
        tokens[1] = V
        tokens[2] = V - 1
    ref = oracle.score_gm(h, W, tokens, seeds, positions, f32(0.8), f32(0.3), f32(EPS))
    check_gm(Device(h, W, seeds, positions).score("gm", tokens, 0.8, 0.3, EPS), ref)


def test_zero_temperature_gm():
    h, W, seeds, positions = _small(150, 128, 700, 5)
    tokens = _claims(h, W, seeds, positions, 0.0, 6)
    ref = oracle.score_gm(h, W, tokens, seeds, positions, 0.0, f32(0.2), f32(EPS))
    got = Device(h, W, seeds, positions).score("gm", tokens, 0.0, 0.2, EPS)
    np.testing.assert_allclose(got["score"], ref.score, rtol=0, atol=SCORE_TOL)
    assert np.array_equal(got["argmax"], ref.argmax)
    assert np.all(np.isnan(got["lse"]))


@pytest.mark.parametrize("temperature,sigma", [(1.0, 1.0), (0.7, 0.05)])
def test_tiny_workload_ipt(temperature, sigma):
    w = wl.WORKLOADS["tiny"]
    inp = wl.make_inputs(w)
    honest = oracle.sample_ipt(inp.h_server, inp.W, inp.seeds, inp.positions, f32(temperature))
    tokens, _ = wl.tamper(w, honest, (honest + 1) % w.V)
    ref = oracle.score_ipt(inp.h, inp.W, tokens, inp.seeds, inp.positions, f32(temperature), f32(sigma), f32(EPS))
    got = Device(inp.h, inp.W, inp.seeds, inp.positions).score("ipt", tokens, temperature, sigma, EPS)
    np.testing.assert_allclose(got["score"], ref.score, rtol=0, atol=SCORE_TOL)
    np.testing.assert_allclose(got["lse"], ref.lse, rtol=LSE_RTOL)
    np.testing.assert_allclose(got["p_claimed"], ref.p_claimed, rtol=1e-3, atol=1e-9)
    np.testing.assert_allclose(got["cdf_lo"], ref.cdf_lo, rtol=0, atol=2e-6)
    np.testing.assert_allclose(got["u"], ref.u, rtol=0, atol=1e-7)
    assert np.array_equal(got["row_status"], ref.row_status)


@pytest.mark.parametrize("T,d,V", [(300, 200, 1000), (129, 64, 257), (1, 8, 2)])
def test_ragged_shapes_ipt(T, d, V):
    h, W, seeds, positions = _small(T, d, V, 7)
    tokens = oracle.sample_ipt(h, W, seeds, positions, f32(1.2)).astype(np.int32)
    tokens[::7] = (tokens[::7] * 31 + 5) % V
    if T >= 3:
        tokens[0] = -1
        tokens[1] = V + 3
        tokens[2] = 0
    ref = oracle.score_ipt(h, W, tokens, seeds, positions, f32(1.2), f32(0.1), f32(EPS))
    got = Device(h, W, seeds, positions).score("ipt", tokens, 1.2, 0.1, EPS)
    np.testing.assert_allclose(got["score"], ref.score, rtol=0, atol=SCORE_TOL)
    ok = ref.row_status == 0
    np.testing.assert_allclose(got["cdf_lo"][ok], ref.cdf_lo[ok], rtol=0, atol=2e-6)
    assert np.array_equal(got["row_status"], ref.row_status)


def test_rows_are_equivariant_bit_for_bit():
    """Permuting the rows of a call permutes its outputs exactly."""
    h, W, seeds, positions = _small(384, 128, 2048, 8)
    tokens = _claims(h, W, seeds, positions, 1.0, 9)
    base = Device(h, W, seeds, positions).score("gm", tokens, 1.0, 0.5, EPS)
    order = np.random.default_rng(10).permutation(384)
    perm = Device(h[order], W, seeds[order], positions[order]).score("gm", tokens[order], 1.0, 0.5, EPS)
    for k in ("score", "margin", "argmax", "runner_up", "lse"):
        assert np.array_equal(perm[k], base[k][order], equal_nan=True), k


def test_detect_matches_oracle():
    g = np.random.default_rng(11)
    T = 5000
    scores = g.normal(-2, 3, size=T).astype(np.float32)
    scores[77] = np.nan
    margins = g.normal(0.3, 1, size=T).astype(np.float32)
    margins[5] = 0.0
    margins[6] = -0.0
    offs = np.array([0, 1, 1, 700, 701, 2048, 4999, 5000], dtype=np.int32)
    tau = -3.5
    ref_flags, ref_stats = oracle.detect(scores.astype(np.float64), f32(tau), margins.astype(np.float64), offs)
    flags = torch.full((T,), 9, dtype=torch.uint8, device="cuda")
    stats = torch.zeros((len(offs) - 1, 4), dtype=torch.int32, device="cuda")
    # an offset view of the score array exercises the unaligned head of the vector loop
    pad = torch.zeros(T + 1, dtype=torch.float32, device="cuda")
    pad[1:] = torch.from_numpy(scores).cuda()
    difr.difr_detect(pad[1:], tau, to_dev(margins), None, 0, to_dev(offs), flags, stats)
    torch.cuda.synchronize()
    assert np.array_equal(flags.cpu().numpy(), ref_flags)
    got = stats.cpu().numpy().view(SEQ_STATS_DTYPE).reshape(-1)
    assert np.array_equal(got["n_flagged"], ref_stats["n_flagged"])
    assert np.array_equal(got["n_match"], ref_stats["n_match"])
    np.testing.assert_allclose(got["sum"], ref_stats["sum"], rtol=1e-5, atol=1e-3, equal_nan=True)
    assert np.array_equal(got["min"], ref_stats["min"].astype(np.float32))
    # one sequence, no offsets
    stats1 = torch.zeros((1, 4), dtype=torch.int32, device="cuda")
    difr.difr_detect(to_dev(scores), tau, to_dev(margins), None, 0, None, None, stats1)
    one = stats1.cpu().numpy().view(SEQ_STATS_DTYPE).reshape(-1)
    _, ref1 = oracle.detect(scores.astype(np.float64), f32(tau), margins.astype(np.float64), None)
    assert one["n_flagged"][0] == ref1["n_flagged"][0] and one["n_match"][0] == ref1["n_match"][0]


@pytest.mark.parametrize("temperature,sigma", [(1.0, 0.05), (0.7, 1.0)])
def test_peaked_large_logits(temperature, sigma):
    """Logits as a trained head produces them: spread over tens of units with a common offset, one or two ids far
    ahead of the rest, rather than the unit-variance logits of the synthetic workloads."""
    T, d, V = 260, 256, 6000
    g = np.random.default_rng(12)
    hf = g.standard_normal((T, d)).astype(np.float32)
    Wf = (6.0 * g.standard_normal((V, d)) / math.sqrt(d)).astype(np.float32)
    bias_dir = g.standard_normal(d).astype(np.float32) / math.sqrt(d)
    hf += 4.0 * math.sqrt(d) * bias_dir            # every row carries the same strong component ...
    Wf += 7.0 * bias_dir / math.sqrt(d)            # ... that every id responds to: a common offset of about +28
    Wf[g.integers(0, V, size=40)] *= 1.8           # a few ids with much larger logits
    h, W = wl.f32_to_bf16_bits(hf), wl.f32_to_bf16_bits(Wf)
    seeds = np.array([wl.splitmix64(900 + r // 32) for r in range(T)], dtype=np.uint64)
    positions = (np.arange(T) % 32 + 1).astype(np.uint32)
    L = oracle.logits(h, W)
    assert L.mean() > 15 and L.std() > 4 and L.max() > 50
    tokens = _claims(h, W, seeds, positions, f32(temperature), 13)
    dev = Device(h, W, seeds, positions)
    ref = oracle.score_gm(h, W, tokens, seeds, positions, f32(temperature), f32(sigma), f32(EPS))
    check_gm(dev.score("gm", tokens, temperature, sigma, EPS), ref)
    itok = oracle.sample_ipt(h, W, seeds, positions, f32(temperature)).astype(np.int32)
    itok[::5] = tokens[::5]
    iref = oracle.score_ipt(h, W, itok, seeds, positions, f32(temperature), f32(0.05), f32(EPS))
    got = dev.score("ipt", itok, temperature, 0.05, EPS)
    np.testing.assert_allclose(got["score"], iref.score, rtol=0, atol=SCORE_TOL)
    np.testing.assert_allclose(got["lse"], iref.lse, rtol=LSE_RTOL)
    # logits of magnitude 50 carry about 5e-5 of fp32 accumulation error from the tensor cores, which the softmax
    # turns into a relative error of that size in every probability
    np.testing.assert_allclose(got["cdf_lo"], iref.cdf_lo, rtol=1e-4, atol=2e-6)


def test_a_wait_that_cannot_complete_gives_up_and_reports_it():
    """Every device-side wait of the library is bounded; here the bound is a millisecond and nothing ever arrives."""
    status = torch.zeros(2, dtype=torch.int32, device="cuda")
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    difr.difr_selftest_wait(status, 2_000_000)
    t1.record()
    torch.cuda.synchronize()
    assert status.cpu().tolist() == [-7, 1]  # DIFR_ERR_TIMEOUT, abort flag raised
    assert t0.elapsed_time(t1) < 100.0       # milliseconds: it really was bounded
    # the context is still usable
    assert int(torch.ones(4, device="cuda").sum().item()) == 4


def test_scores_do_not_depend_on_how_the_vocabulary_is_split():
    """The number of vocabulary strips (and with it the partial records that are merged) is a planning choice:
    argmax, runner-up and margins must not move at all (they are re-evaluated exactly), the log-sum-exp and the
    IPT statistics only by the rounding of a differently ordered sum."""
    T, d, V = 300, 128, 5000
    h, W, seeds, positions = _small(T, d, V, 14)
    tokens = _claims(h, W, seeds, positions, 1.0, 15)
    dev = Device(h, W, seeds, positions)
    results = []
    try:
        for strips, group in ((1, 1), (3, 2), (20, 1)):
            difr.difr_debug_plan_override(strips, group)
            results.append((dev.score("gm", tokens, 1.0, 0.3, EPS), dev.score("ipt", tokens, 1.0, 0.1, EPS)))
    finally:
        difr.difr_debug_plan_override()
    results.append((dev.score("gm", tokens, 1.0, 0.3, EPS), dev.score("ipt", tokens, 1.0, 0.1, EPS)))
    gm0, ipt0 = results[0]
    for gm, ipt in results[1:]:
        for k in ("score", "margin", "argmax", "runner_up"):
            assert np.array_equal(gm[k], gm0[k]), k
        np.testing.assert_allclose(gm["lse"], gm0["lse"], rtol=2e-6)
        np.testing.assert_allclose(ipt["cdf_lo"], ipt0["cdf_lo"], rtol=2e-5, atol=1e-7)
        np.testing.assert_allclose(ipt["score"], ipt0["score"], rtol=0, atol=2e-4)


def test_two_calls_in_flight_on_two_streams_keep_to_their_own_workspaces():
    """Two scoring calls enqueued back to back on different streams, each with its own workspace (its own partial
    records and work counter), give bit for bit what each gives alone."""
    a = _small(700, 96, 5000, 41)
    b = _small(300, 64, 9001, 42)
    tok_a = _claims(*a, f32(1.0), 43)
    tok_b = _claims(*b, f32(0.8), 44)
    dev_a, dev_b = Device(*a), Device(*b)
    alone_a = dev_a.score("gm", tok_a, 1.0, 0.3)
    alone_b = dev_b.score("ipt", tok_b, 0.8, 0.1)
    out_a = difr.DifrOut.allocate(dev_a.T, dev_a.d, dev_a.V, 0.3, EPS)
    out_b = difr.DifrOut.allocate(dev_b.T, dev_b.d, dev_b.V, 0.1, EPS)
    ta, tb = to_dev(tok_a), to_dev(tok_b)
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    for _ in range(3):
        difr.difr_score_gm(dev_a.h, dev_a.W, ta, dev_a.seeds, dev_a.positions, f32(1.0), out_a, stream=s1)
        difr.difr_score_ipt(dev_b.h, dev_b.W, tb, dev_b.seeds, dev_b.positions, f32(0.8), out_b, stream=s2)
    torch.cuda.synchronize()
    assert int(out_a.device_status.item()) == 0 and int(out_b.device_status.item()) == 0
    for k in ("score", "margin", "argmax", "runner_up", "lse"):
        assert np.array_equal(getattr(out_a, k).cpu().numpy(), alone_a[k], equal_nan=True), k
    for k in ("score", "p_claimed", "cdf_lo", "u", "lse"):
        assert np.array_equal(getattr(out_b, k).cpu().numpy(), alone_b[k], equal_nan=True), k


def test_rows_with_non_finite_logits_are_never_scored_as_safe():
    """A NaN or an infinity in a row of h makes every logit of that row non-finite, one in a row of W makes one
    logit of every row non-finite: the oracle marks exactly those rows (row_status bit 1), and so must the library,
    whose scores there are NaN (flagged by the detection step) whatever the claim."""
    T, d, V = 200, 64, 3000
    h, W, seeds, positions = _small(T, d, V, 51)
    tokens = _claims(h, W, seeds, positions, f32(1.0), 52)
    h = h.copy()
    h[3, 5] = 0x7FC0    # NaN
    h[40, 0] = 0x7F80   # +inf
    h[41, 63] = 0xFF80  # -inf
    for W_case in ("clean", "nan_in_W"):
        Wc = W.copy()
        if W_case == "nan_in_W":
            Wc[2999, 7] = 0x7FC0
        dev = Device(h, Wc, seeds, positions)
        ref = oracle.score_gm(h, Wc, tokens, seeds, positions, f32(1.0), f32(0.3), f32(EPS))
        marked = (ref.row_status & 2) != 0
        assert marked.sum() == (3 if W_case == "clean" else T)
        for kind in ("gm", "ipt"):
            got = dev.score(kind, tokens, 1.0, 0.3, EPS)
            assert np.array_equal((got["row_status"] & 2) != 0, marked), (W_case, kind)
            assert np.all(np.isnan(got["score"][marked])), (W_case, kind)
            assert np.all(np.isfinite(got["score"][~marked])), (W_case, kind)
        if W_case == "clean":
            ok = ~marked
            np.testing.assert_allclose(dev.score("gm", tokens, 1.0, 0.3, EPS)["score"][ok], ref.score[ok], rtol=0, atol=SCORE_TOL)
        flags, _ = difr.difr_detect(to_dev(dev.score("gm", tokens, 1.0, 0.3, EPS)["score"]), -20.0,
                                    flags=torch.zeros(T, dtype=torch.uint8, device="cuda"))
        torch.cuda.synchronize()
        assert np.all(flags.cpu().numpy()[marked] == 1)


@pytest.mark.parametrize("tied", [(37, 1301), (1301, 37, 700), (8999, 5000, 37, 700, 1301, 4096, 4111),
                                  (4098, 4100, 4111), (4111, 4097, 4103, 4100, 8990),   # three and more in one 16-id group
                                  (37, 4098, 4100, 4111), (36, 37, 39, 44, 47)])
def test_exact_ties_go_to_the_lowest_id(tied):
    """Greedy replay with identical rows of W that hold the largest logit of every row: the lowest id is the
    sample, the next lowest the runner-up, and a claim of any other tied id is a mismatch by the tie-break alone
    (margin -0.0), as in the oracle.  The tied ids lie in different 16-id groups, tiles and strips, or several of
    them inside one aligned group of 16 ids (where the fused kernel ranks equal keys by column and marks the
    record, and the finalize kernel walks the group)."""
    T, d, V = 64, 64, 9000
    h, W, seeds, positions = _small(T, d, V, 61)
    # one direction that dominates every row's logits: h gets a large common component, the tied rows point along it
    h = wl.f32_to_bf16_bits(wl.bf16_bits_to_f32(h) + 4.0 * np.sign(np.arange(d) % 2 - 0.5).astype(np.float32))
    W = W.copy()
    along = wl.f32_to_bf16_bits((np.sign(np.arange(d) % 2 - 0.5)).astype(np.float32))
    for v in tied:
        W[v] = along
    order = sorted(tied)
    tokens = np.array([tied[r % len(tied)] for r in range(T)], dtype=np.int32)
    ref = oracle.score_gm(h, W, tokens, seeds, positions, 0.0, f32(0.2), f32(EPS))
    assert np.all(ref.argmax == order[0]) and np.all(ref.runner_up == order[1]) and np.all(ref.top2_margin == 0.0)
    got = Device(h, W, seeds, positions).score("gm", tokens, 0.0, 0.2, EPS)
    assert np.array_equal(got["argmax"], ref.argmax) and np.array_equal(got["runner_up"], ref.runner_up)
    assert np.all(got["margin"] == 0.0) and np.array_equal(np.signbit(got["margin"]), np.signbit(ref.margin))
    assert np.array_equal(np.signbit(got["margin"]), tokens != order[0])
    np.testing.assert_allclose(got["score"], ref.score, rtol=0, atol=1e-6)


@pytest.mark.parametrize("sigma", [0.01, 0.001])
def test_near_ties_below_the_fused_kernels_ranking_noise_are_resolved_exactly(sigma):
    """Three ids in different strips whose logits differ by 7.5e-6 (far below what the fused kernel's fp32 keys
    can tell apart) hold the top of every row under greedy replay.  The finalize kernel re-evaluates every
    candidate inside the ranking noise of the second best in fp64, so the sample, the runner-up and the claimed
    token's competitor are the oracle's; at sigma 0.001 the wrong competitor would move the score by 4e-3."""
    T, d, V = 96, 64, 9000
    h, W, seeds, positions = _small(T, d, V, 67)
    hf = wl.bf16_bits_to_f32(h) * np.float32(0.25)
    hf[:, 0] = 1.0
    hf[:, 1] = 2.0 ** -10
    Wf = wl.bf16_bits_to_f32(W).copy()
    Wf[:, 0] = 0.0
    Wf[:, 1] = 0.0
    ids = (37, 3001, 8800)  # ascending logits: the highest id is the exact maximum
    for k, v in enumerate(ids):
        Wf[v] = 0.0
        Wf[v, 0] = 8.0
        Wf[v, 1] = k * 2.0 ** -7
    h, W = wl.f32_to_bf16_bits(hf), wl.f32_to_bf16_bits(Wf)
    tokens = np.array([ids[r % 3] for r in range(T)], dtype=np.int32)
    ref = oracle.score_gm(h, W, tokens, seeds, positions, 0.0, f32(sigma), f32(EPS))
    assert np.all(ref.argmax == ids[2]) and np.all(ref.runner_up == ids[1])
    assert np.all(ref.top2_margin < 1e-5) and np.all(ref.top2_margin > 0) and np.all(ref.top23_margin < 1e-5)
    got = Device(h, W, seeds, positions).score("gm", tokens, 0.0, sigma, EPS)
    assert np.array_equal(got["argmax"], ref.argmax) and np.array_equal(got["runner_up"], ref.runner_up)
    np.testing.assert_allclose(got["margin"], ref.margin, rtol=1e-6, atol=1e-9)
    np.testing.assert_allclose(got["score"], ref.score, rtol=0, atol=SCORE_TOL)
    # the three claims score differently, by more than the tolerance at the smaller widths
    assert len(np.unique(np.round(ref.score[:3] / (2 * SCORE_TOL)))) >= (3 if sigma <= 0.001 else 2)


@pytest.mark.parametrize("T,d,V,temperature", [(256, 512, 4096, 1.0), (300, 200, 1000, 0.7), (129, 64, 5000, 1.0)])
@pytest.mark.parametrize("sigma", [0.01, 0.001])
def test_small_noise_widths_of_the_papers_sweep(T, d, V, temperature, sigma):
    """The paper sweeps the estimator's noise width down to 0.001, where 1e-5 of margin is 1e-2 of score: the
    scores still agree with the oracle to 2e-3 on every row, ragged shapes included."""
    h, W, seeds, positions = _small(T, d, V, 71)
    tokens = _claims(h, W, seeds, positions, f32(temperature), 72, frac=0.3)
    ref = oracle.score_gm(h, W, tokens, seeds, positions, f32(temperature), f32(sigma), f32(EPS))
    got = Device(h, W, seeds, positions).score("gm", tokens, temperature, sigma, EPS)
    np.testing.assert_allclose(got["score"], ref.score, rtol=0, atol=SCORE_TOL)
    np.testing.assert_allclose(got["margin"], ref.margin, rtol=2e-6, atol=1e-6)
    clear = ref.top2_margin >= 1e-6
    assert np.array_equal(got["argmax"][clear], ref.argmax[clear])


@pytest.mark.parametrize("d,kind", [(512, "peaked"), (5120, "unit"), (5120, "peaked")])
def test_ipt_score_holds_its_tolerance_over_widths_and_logit_magnitudes(d, kind):
    """The IPT estimator divides by sigma^2: at sigma 0.01 an error of 1e-7 in a CDF value is 1e-3 of score.  The
    softmax sums come from the tensor cores' fp32 logits; the claimed token's own term is swapped for the fp64
    one in the finalize kernel.  Unit-variance logits at d = 5120 and heads whose logits reach +-200 (one or two
    ids far ahead) stay within 2e-3 for sigma from 0.2 down to 0.01."""
    T, V = 128, 8192
    g = np.random.default_rng(12)
    hf = g.standard_normal((T, d)).astype(np.float32)
    if kind == "unit":
        Wf = (g.standard_normal((V, d)) / math.sqrt(d)).astype(np.float32)
    else:
        Wf = (6.0 * g.standard_normal((V, d)) / math.sqrt(d)).astype(np.float32)
        bias_dir = g.standard_normal(d).astype(np.float32) / math.sqrt(d)
        hf += 4.0 * math.sqrt(d) * bias_dir
        Wf += 7.0 * bias_dir / math.sqrt(d)
        Wf[g.integers(0, V, size=40)] *= 1.8
    h, W = wl.f32_to_bf16_bits(hf), wl.f32_to_bf16_bits(Wf)
    seeds = np.array([wl.splitmix64(900 + r // 32) for r in range(T)], dtype=np.uint64)
    positions = (np.arange(T) % 32 + 1).astype(np.uint32)
    itok = oracle.sample_ipt(h, W, seeds, positions, 1.0).astype(np.int32)
    itok[::5] = g.integers(0, V, size=len(itok[::5]))
    if kind == "peaked":
        assert np.abs(oracle.logits(h[:8], W)).max() > 100
    dev = Device(h, W, seeds, positions)
    for sigma in (0.2, 0.05, 0.01):
        ref = oracle.score_ipt(h, W, itok, seeds, positions, 1.0, f32(sigma), f32(EPS))
        got = dev.score("ipt", itok, 1.0, sigma, EPS)
        np.testing.assert_allclose(got["score"], ref.score, rtol=0, atol=SCORE_TOL, err_msg=f"sigma {sigma}")
        np.testing.assert_allclose(got["lse"], ref.lse, rtol=LSE_RTOL)
        np.testing.assert_allclose(got["p_claimed"], ref.p_claimed, rtol=2e-4, atol=1e-12)
