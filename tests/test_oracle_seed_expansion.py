"""Pins for the oracle's sequential randomness expansion RO(seed || i || context).

The paper fixes no hash, so nothing printed can pin the values; what the
definition must satisfy is checked instead: a row's expanded seed depends on its
own seed, on the prompt hash and on every claimed token before it in its
sequence with its place, and on nothing else."""
import numpy as np

import oracle
import workloads as wl
from oracle import seed_expansion as se


def _case(seed=3, T=40):
    g = np.random.default_rng(seed)
    tokens = g.integers(0, 50000, T).astype(np.int32)
    seeds = g.integers(0, 2**63, T, dtype=np.uint64)
    offsets = np.array([0, 13, 13, 29, T], dtype=np.int32)  # one empty sequence
    prompts = g.integers(0, 2**63, 4, dtype=np.uint64)
    return tokens, seeds, offsets, prompts


def test_a_changed_token_changes_exactly_the_later_rows_of_its_sequence():
    tokens, seeds, offsets, prompts = _case()
    base = se.expand_seeds(seeds, tokens, offsets, prompts)
    assert len(set(base.tolist())) == len(base)
    for j in (0, 5, 12, 13, 20, 28, 29, 39):
        t2 = tokens.copy()
        t2[j] += 1
        got = se.expand_seeds(seeds, t2, offsets, prompts)
        end = int(offsets[np.searchsorted(offsets, j, side="right")])
        changed = got != base
        assert not changed[: j + 1].any() and changed[j + 1 : end].all() and not changed[end:].any(), j


def test_the_place_of_a_token_matters():
    tokens, seeds, offsets, prompts = _case()
    base = se.context_hashes(tokens, offsets, prompts)
    t2 = tokens.copy()
    t2[[3, 4]] = t2[[4, 3]]
    assert tokens[3] != tokens[4]
    got = se.context_hashes(t2, offsets, prompts)
    assert got[:4] == base[:4] and got[4] != base[4]
    assert all(a != b for a, b in zip(got[5:13], base[5:13]))  # a swap is not undone by the sum
    assert got[13:] == base[13:]


def test_seed_and_prompt_hash_enter():
    tokens, seeds, offsets, prompts = _case()
    base = se.expand_seeds(seeds, tokens, offsets, prompts)
    s2 = seeds.copy()
    s2[7] ^= np.uint64(1)
    assert ((se.expand_seeds(s2, tokens, offsets, prompts) != base) == (np.arange(len(base)) == 7)).all()
    p2 = prompts.copy()
    p2[2] += np.uint64(1)
    changed = se.expand_seeds(seeds, tokens, offsets, p2) != base
    assert changed[13:29].all() and not changed[:13].any() and not changed[29:].any()
    # no prompt hashes = all-zero prompt hashes
    assert (se.expand_seeds(seeds, tokens, offsets) == se.expand_seeds(seeds, tokens, offsets, np.zeros(4, np.uint64))).all()


def test_equal_histories_give_equal_randomness():
    """Two sequences with the same prompt hash, seed and tokens draw the same randomness, row by row;
    the first row of a sequence sees the prompt hash alone."""
    tokens = np.array([5, 9, 2, 5, 9, 7], dtype=np.int32)
    seeds = np.full(6, 1234567, dtype=np.uint64)
    offsets = np.array([0, 3, 6], dtype=np.int32)
    prompts = np.array([77, 77], dtype=np.uint64)
    ctx = se.context_hashes(tokens, offsets, prompts)
    assert ctx[0] == ctx[3] == 77 and ctx[1] == ctx[4] and ctx[2] == ctx[5]
    out = se.expand_seeds(seeds, tokens, offsets, prompts)
    assert out[0] == out[3] and out[1] == out[4] and out[2] == out[5]
    assert len({int(x) for x in out[:3]}) == 3


def test_expanded_seeds_look_uniform_and_drive_the_sampler():
    """Bits of the expanded seeds are balanced, and a Gumbel-max sample drawn with an expanded seed is
    re-found by scoring with the same expanded seed (margin >= 0), not with the raw one."""
    g = np.random.default_rng(11)
    T = 2000
    tokens = g.integers(0, 1000, T).astype(np.int32)
    seeds = np.full(T, 42, dtype=np.uint64)  # one seed for the whole batch: all variety comes from the context
    offsets = np.arange(0, T + 1, 100, dtype=np.int32)
    out = se.expand_seeds(seeds, tokens, offsets)
    assert len(set(out.tolist())) == T - 20 + 1  # only the 20 first rows (empty context) coincide
    bits = np.unpackbits(out.view(np.uint8))
    assert abs(bits.mean() - 0.5) < 0.01
    # end to end on a tiny model
    Tm, d, V = 64, 16, 64
    h = wl.f32_to_bf16_bits(g.standard_normal((Tm, d)).astype(np.float32))
    W = wl.f32_to_bf16_bits((g.standard_normal((V, d)) / 2.0).astype(np.float32))
    positions = (np.arange(Tm) % 32 + 1).astype(np.uint32)
    exp = out[:Tm]
    sampled, _ = oracle.sample_gm(h, W, exp, positions, 1.0)
    assert np.all(oracle.score_gm(h, W, sampled, exp, positions, 1.0, 0.05).margin >= 0.0)
    assert np.mean(oracle.score_gm(h, W, sampled, seeds[:Tm], positions, 1.0, 0.05).margin < 0.0) > 0.5
