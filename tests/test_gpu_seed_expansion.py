"""GPU-vs-oracle parity of the sequential randomness expansion: integer work, so every word must be equal."""
import numpy as np
import pytest
import torch

import oracle
import workloads as wl
from gpu_util import Device, to_dev
from oracle import seed_expansion as se

import paper_2511_02620_b200 as difr

pytestmark = pytest.mark.gpu


def _u64(t: torch.Tensor) -> np.ndarray:
    return t.cpu().numpy().view(np.uint64)


@pytest.mark.parametrize("T,offsets", [
    (1, [0, 1]),
    (700, [0, 700]),                                   # one sequence over several chunks of the block, ragged tail
    (1000, [0, 0, 255, 256, 513, 513, 999, 1000]),      # empty sequences, lengths around the chunk size, one row
    (2048, None),                                      # no offsets: the whole batch is one sequence
])
def test_expanded_seeds_equal_the_oracle(T, offsets):
    g = np.random.default_rng(T)
    tokens = g.integers(-3, 152064, T).astype(np.int32)  # a few out-of-range claims as well
    seeds = g.integers(0, 2**64, T, dtype=np.uint64)
    n_seq = 1 if offsets is None else len(offsets) - 1
    prompts = g.integers(0, 2**64, n_seq, dtype=np.uint64)
    off_np = np.array([0, T] if offsets is None else offsets, dtype=np.int32)
    want = se.expand_seeds(seeds, tokens, off_np, prompts)
    off_dev = None if offsets is None else to_dev(off_np)
    got = difr.difr_expand_seeds(to_dev(seeds), to_dev(tokens), off_dev, to_dev(prompts))
    torch.cuda.synchronize()
    assert np.array_equal(_u64(got), want)
    # without prompt hashes, and in place
    want0 = se.expand_seeds(seeds, tokens, off_np)
    buf = to_dev(seeds)
    difr.difr_expand_seeds(buf, to_dev(tokens), off_dev, None, expanded=buf)
    torch.cuda.synchronize()
    assert np.array_equal(_u64(buf), want0)


def test_rows_outside_every_sequence_are_left_alone():
    T = 300
    g = np.random.default_rng(5)
    tokens = g.integers(0, 1000, T).astype(np.int32)
    seeds = g.integers(0, 2**64, T, dtype=np.uint64)
    off = np.array([0, 100, 250], dtype=np.int32)  # rows 250.. belong to nothing
    out = torch.full((T,), -1, dtype=torch.int64, device="cuda")
    difr.difr_expand_seeds(to_dev(seeds), to_dev(tokens), to_dev(off), None, expanded=out)
    torch.cuda.synchronize()
    want = se.expand_seeds(seeds[:250], tokens[:250], off)
    assert np.array_equal(_u64(out)[:250], want) and bool((out[250:] == -1).all())


def test_scoring_with_expanded_seeds_replays_the_expanded_sampler():
    """The server samples with RO(seed || i || context); the verifier expands the same way on the device and
    must find every honest token again (margin >= 0), and the oracle given the oracle's expansion agrees."""
    T, d, V = 384, 64, 1000
    g = np.random.default_rng(9)
    h = wl.f32_to_bf16_bits(g.standard_normal((T, d)).astype(np.float32))
    W = wl.f32_to_bf16_bits((g.standard_normal((V, d)) / 8.0).astype(np.float32))
    positions = (np.arange(T) % 128 + 1).astype(np.uint32)
    off = np.array([0, 128, 256, 384], dtype=np.int32)
    seeds = np.repeat(g.integers(0, 2**64, 3, dtype=np.uint64), 128)
    prompts = g.integers(0, 2**64, 3, dtype=np.uint64)
    # the server's loop: each token is drawn with the context of the tokens before it
    tokens = np.zeros(T, dtype=np.int32)
    for r in range(T):
        q, o = divmod(r, 128)[0], (r // 128) * 128
        exp_r = se.expand_seeds(seeds[o : r + 1], tokens[o : r + 1], [0, r + 1 - o], prompts[q : q + 1])[-1:]
        tok, _ = oracle.sample_gm(h[r : r + 1], W, exp_r, positions[r : r + 1], 1.0)
        tokens[r] = tok[0]
    dev = Device(h, W, seeds, positions)
    dev.seeds = difr.difr_expand_seeds(dev.seeds, to_dev(tokens), to_dev(off), to_dev(prompts))
    out = dev.score("gm", tokens, 1.0, 0.05)
    assert np.all(out["margin"] >= 0) and np.array_equal(out["argmax"], tokens)
    ref = oracle.score_gm(h, W, tokens, se.expand_seeds(seeds, tokens, off, prompts), positions, 1.0, 0.05)
    assert np.max(np.abs(out["score"] - ref.score)) < 2e-3
