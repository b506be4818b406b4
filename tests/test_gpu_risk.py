"""GPU-vs-oracle parity of the widened path: raw-logit rank and the three risk
classes, both estimators from one pass, admissible-set sizes and the
information bound.  The integers (a rank, a set size) must be the oracle's on
every row: the fused kernel counts what fp32 can decide and lists the ids it
cannot, and a finalize kernel decides those in fp64."""
import math

import numpy as np
import pytest
import torch

import oracle
import workloads as wl
from gpu_util import Device, f32, to_dev

import paper_2511_02620_b200 as difr

pytestmark = pytest.mark.gpu

EPS = 1e-12
SCORE_TOL = 2e-3


def _small(T, d, V, seed):
    g = np.random.default_rng(seed)
    h = wl.f32_to_bf16_bits(g.standard_normal((T, d)).astype(np.float32))
    W = wl.f32_to_bf16_bits((g.standard_normal((V, d)) / math.sqrt(d)).astype(np.float32))
    seeds = np.array([wl.splitmix64(seed * 1000 + r // 64) for r in range(T)], dtype=np.uint64)
    positions = (np.arange(T) % 64 + 1).astype(np.uint32)
    return h, W, seeds, positions


def _claims(h, W, seeds, positions, temperature, seed):
    honest, runner = oracle.sample_gm(h, W, seeds, positions, temperature)
    g = np.random.default_rng(seed)
    T, V = h.shape[0], W.shape[0]
    tokens = honest.copy()
    k = np.arange(T)
    tokens[k % 5 == 1] = runner[k % 5 == 1]
    rnd = g.integers(0, V, size=T)
    tokens[k % 5 == 3] = rnd[k % 5 == 3]
    return tokens.astype(np.int32)


def _score(dev, fn, tokens, temperature, sigma, want_rank=False, sigma_ipt=0.0):
    out = difr.DifrOut.allocate(dev.T, dev.d, dev.V, sigma, EPS)
    f = lambda: torch.full((dev.T,), float("nan"), dtype=torch.float32, device="cuda")
    out.y_max, out.y_second = f(), f()
    if want_rank:
        out.rank = torch.full((dev.T,), -7, dtype=torch.int32, device="cuda")
    if sigma_ipt:
        out.sigma_ipt, out.score_ipt = sigma_ipt, f()
    fn(dev.h, dev.W, to_dev(np.asarray(tokens, dtype=np.int32)), dev.seeds, dev.positions, f32(temperature), out)
    torch.cuda.synchronize()
    assert int(out.device_status.item()) == 0
    return out


@pytest.mark.parametrize("T,d,V,temperature", [(300, 128, 3000, 1.0), (130, 72, 777, 0.7)])
def test_rank_and_three_classes(T, d, V, temperature):
    h, W, seeds, positions = _small(T, d, V, 21)
    tokens = _claims(h, W, seeds, positions, f32(temperature), 22)
    tokens[7] = V + 5  # an id outside the vocabulary
    dev = Device(h, W, seeds, positions)
    sigma = 0.3
    out = _score(dev, difr.difr_score_gm, tokens, temperature, sigma, want_rank=True)
    plain = _score(dev, difr.difr_score_gm, tokens, temperature, sigma)
    assert torch.equal(out.score, plain.score) and torch.equal(out.argmax, plain.argmax)  # asking for ranks changes nothing else
    ref = oracle.score_gm(h, W, tokens, seeds, positions, f32(temperature), f32(sigma), f32(EPS))
    got = out.rank.cpu().numpy()
    ok = (tokens >= 0) & (tokens < V)
    assert np.array_equal(got, ref.rank)
    assert np.all(got[~ok] == V)
    assert got[ok].max() > V // 2 and got[ok].min() < 10  # both ends of the range are exercised
    assert np.all(out.row_status.cpu().numpy() & 32 == 0)  # no list of undecided ids overflowed

    # three classes: decided wherever the score does not sit on the threshold
    score = out.score.cpu().numpy()
    np.testing.assert_allclose(score, ref.score, rtol=0, atol=SCORE_TOL)
    tau = -1.5
    for R in (1, 8, 200):
        want = oracle.classify(ref.score, tau, ref.rank, R)
        flags = torch.full((T,), 9, dtype=torch.uint8, device="cuda")
        difr.difr_detect(out.score, tau, out.margin, out.rank, R, None, flags, None)
        torch.cuda.synchronize()
        decided = np.abs(ref.score - tau) > 2 * SCORE_TOL
        assert decided.mean() > 0.95
        assert np.array_equal(flags.cpu().numpy()[decided], want[decided])
    assert set(np.unique(want[decided])) == {0, 1, 2}


def test_rank_is_exact_among_logits_closer_than_fp32_can_tell():
    """Rows of W that differ from the claimed token's row in one small component give logits 4e-6 apart around
    the claimed logit, well inside the tensor cores' rounding: the fused kernel lists them, the finalize kernel
    compares them in fp64, and identical rows (equal logits) do not count as larger."""
    T, d, V = 64, 128, 3000
    h, W, seeds, positions = _small(T, d, V, 23)
    hf = wl.bf16_bits_to_f32(h).copy()
    hf[:, 0] = 2.0 ** -9
    Wf = wl.bf16_bits_to_f32(W).copy()
    Wf[:, 0] = 0.0
    claimed = 1500
    near = [3, 700, 1499, 1501, 2222, 2999, 40, 41]           # same row as the claim, component 0 changed
    for k, v in enumerate(near):
        Wf[v] = Wf[claimed]
        Wf[v, 0] = (k - 3) * 2.0 ** -9   # logit differences (k - 3) * 2^-18: three below, one equal, four above
    h, W = wl.f32_to_bf16_bits(hf), wl.f32_to_bf16_bits(Wf)
    tokens = np.full(T, claimed, dtype=np.int32)
    dev = Device(h, W, seeds, positions)
    out = _score(dev, difr.difr_score_gm, tokens, 1.0, 0.3, want_rank=True)
    ref = oracle.score_gm(h, W, tokens, seeds, positions, f32(1.0), f32(0.3), f32(EPS))
    logits = oracle.logits(h, W)
    assert np.all(np.abs(logits[:, near] - logits[:, [claimed]]) < 2e-5)
    assert np.array_equal(out.rank.cpu().numpy(), ref.rank)
    assert len(np.unique(ref.rank)) > 4  # the rows differ in how many other ids lie above


def test_both_scores_from_one_pass_equal_the_two_separate_calls():
    T, d, V = 260, 136, 2100
    h, W, seeds, positions = _small(T, d, V, 31)
    tokens = _claims(h, W, seeds, positions, f32(0.7), 32)
    dev = Device(h, W, seeds, positions)
    both = _score(dev, difr.difr_score_both, tokens, 0.7, 0.3, sigma_ipt=0.05)
    gm = _score(dev, difr.difr_score_gm, tokens, 0.7, 0.3)
    ipt = _score(dev, difr.difr_score_ipt, tokens, 0.7, 0.05)
    for name in ("score", "margin", "argmax", "runner_up", "y_max", "y_second"):
        assert torch.equal(getattr(both, name), getattr(gm, name)), name
    assert torch.equal(both.score_ipt, ipt.score)
    for name in ("p_claimed", "cdf_lo", "u", "lse"):
        assert torch.equal(getattr(both, name), getattr(ipt, name)), name
    ref_gm = oracle.score_gm(h, W, tokens, seeds, positions, f32(0.7), f32(0.3), f32(EPS))
    ref_ipt = oracle.score_ipt(h, W, tokens, seeds, positions, f32(0.7), f32(0.05), f32(EPS))
    np.testing.assert_allclose(both.score.cpu().numpy(), ref_gm.score, rtol=0, atol=SCORE_TOL)
    np.testing.assert_allclose(both.score_ipt.cpu().numpy(), ref_ipt.score, rtol=0, atol=SCORE_TOL)
    # y_max / y_second are the two largest noisy logits
    np.testing.assert_allclose(both.y_max.cpu().numpy() - both.y_second.cpu().numpy(), ref_gm.top2_margin, atol=1e-4)


@pytest.mark.parametrize("T,d,V,temperature,sigma", [(150, 64, 1200, 1.0, 1.0), (140, 72, 520, 0.7, 0.3),
                                                     (130, 64, 700, 0.0, 0.5)])  # the last: greedy decoding, no noise
def test_admissible_set_sizes_and_information_bound(T, d, V, temperature, sigma):
    h, W, seeds, positions = _small(T, d, V, 41)
    dev = Device(h, W, seeds, positions)
    tokens = _claims(h, W, seeds, positions, f32(temperature), 42)
    scored = _score(dev, difr.difr_score_gm, tokens, temperature, sigma, want_rank=True)
    taus = [f32(-0.9), f32(-3.0), f32(-9.0), f32(math.log(EPS))]  # the last: every id is admissible
    counts = torch.full((len(taus), T), -1, dtype=torch.int32, device="cuda")
    difr.difr_admissible(dev.h, dev.W, dev.seeds, dev.positions, f32(temperature), scored, taus, counts)
    one = torch.full((1, T), -1, dtype=torch.int32, device="cuda")
    difr.difr_admissible(dev.h, dev.W, dev.seeds, dev.positions, f32(temperature), scored, taus[1:2], one)
    none = torch.full((1, T), -1, dtype=torch.int32, device="cuda")
    difr.difr_admissible(dev.h, dev.W, dev.seeds, dev.positions, f32(temperature), scored, [f32(0.5)], none)
    torch.cuda.synchronize()
    assert int(scored.device_status.item()) == 0
    got = counts.cpu().numpy()
    assert np.array_equal(one.cpu().numpy()[0], got[1])  # one bound or four: the same count
    assert np.all(none.cpu().numpy() == 0)               # no score reaches a threshold above ln(1 + eps)

    # the oracle's sets: every count is the oracle's
    status = torch.full((T,), 0x7fffffff, dtype=torch.int32, device="cuda")
    again = torch.full((len(taus), T), -1, dtype=torch.int32, device="cuda")
    difr.difr_admissible(dev.h, dev.W, dev.seeds, dev.positions, f32(temperature), scored, taus, again, status)
    torch.cuda.synchronize()
    assert torch.equal(again, counts) and int(status.max().item()) == 0
    for j, tau in enumerate(taus):
        want = oracle.admissible_count(h, W, seeds, positions, f32(temperature), f32(sigma), tau, f32(EPS))
        assert np.array_equal(got[j], want), (j, np.nonzero(got[j] != want)[0][:8])
    assert np.all(got[3] == V) and got[0].max() < V and got[2].max() > got[0].max()

    # information bound per token and per sequence
    tau, R = taus[1], 8
    flags = torch.empty(T, dtype=torch.uint8, device="cuda")
    difr.difr_detect(scored.score, tau, scored.margin, scored.rank, R, None, flags, None)
    seq_offsets = np.array([0, T // 3, T // 3, T], dtype=np.int32)  # one empty sequence
    bits = torch.full((T,), float("nan"), dtype=torch.float32, device="cuda")
    seq_bits = torch.full((3,), float("nan"), dtype=torch.float32, device="cuda")
    difr.difr_exfiltratable_bits(flags, counts[1], R, V, to_dev(seq_offsets), bits, seq_bits)
    torch.cuda.synchronize()
    want_bits, want_seq = oracle.exfiltratable_bits(flags.cpu().numpy(), got[1], R, V, seq_offsets)
    np.testing.assert_allclose(bits.cpu().numpy(), want_bits, rtol=1e-6, atol=1e-6)
    np.testing.assert_allclose(seq_bits.cpu().numpy(), want_seq, rtol=1e-5)
    assert seq_bits.cpu().numpy()[1] == 0.0


def test_per_row_temperatures_equal_one_call_per_temperature():
    """Requests with their own sampling temperature in one batch: every row must come out exactly as in a call
    that uses its temperature for the whole batch."""
    T, d, V = 300, 128, 2600
    h, W, seeds, positions = _small(T, d, V, 71)
    temps = np.where(np.arange(T) % 3 == 0, 0.7, 1.0).astype(np.float32)
    temps[T // 2:] = np.where(np.arange(T - T // 2) % 4 == 0, 1.3, temps[T // 2:])
    tokens = np.empty(T, dtype=np.int32)
    for t in np.unique(temps):
        sel = temps == t
        tokens[sel] = _claims(h[sel], W, seeds[sel], positions[sel], float(t), 72)
    dev = Device(h, W, seeds, positions)
    bad = temps.copy()
    bad[11], bad[12] = -1.0, np.nan
    out = difr.DifrOut.allocate(T, d, V, 0.3, EPS)
    f = lambda: torch.full((T,), float("nan"), dtype=torch.float32, device="cuda")
    out.score_ipt, out.sigma_ipt, out.y_max, out.y_second = f(), 0.05, f(), f()
    out.temperatures = to_dev(bad)
    difr.difr_score_both(dev.h, dev.W, to_dev(tokens), dev.seeds, dev.positions, 123.0, out)  # the scalar is ignored
    torch.cuda.synchronize()
    assert int(out.device_status.item()) == 0
    good = np.ones(T, dtype=bool)
    good[[11, 12]] = False
    status = out.row_status.cpu().numpy()
    assert np.all(status[~good] & 8) and np.all(status[good] == 0)
    assert np.all(np.isnan(out.score.cpu().numpy()[~good])) and np.all(np.isnan(out.score_ipt.cpu().numpy()[~good]))
    for t in np.unique(temps):
        sel = (temps == t) & good
        one = _score(dev, difr.difr_score_both, tokens, float(t), 0.3, sigma_ipt=0.05)
        for name in ("score", "score_ipt", "margin", "argmax", "lse", "cdf_lo", "y_max"):
            a, b = getattr(out, name).cpu().numpy()[sel], getattr(one, name).cpu().numpy()[sel]
            assert np.array_equal(a, b), (t, name)
        ref = oracle.score_gm(h[sel], W, tokens[sel], seeds[sel], positions[sel], float(t), f32(0.3), f32(EPS))
        np.testing.assert_allclose(out.score.cpu().numpy()[sel], ref.score, rtol=0, atol=SCORE_TOL)
