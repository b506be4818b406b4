"""Sequential randomness expansion RO(seed || i || context) -- TEST INFRASTRUCTURE.

The paper asks, for one of its bounds, that the randomness of response index i
also depend on the context (the prompt and the tokens chosen so far): footnote
to the definition of honest sampling in Sec. "Sampling From Large Language
Models", and the first further measure of Sec. "Message-Sampling Secure Seed
Expansion": the next token's randomness comes from a keyed hash of the seed
and of the prompt and tokens so far.  It fixes neither that hash nor the
encoding of its input.  This file writes out the reading the
library takes, one plain loop per definition:

  element word   e(j, t)  = words 0,1 of Philox-4x32-10(counter (j, t, 0, 1), key ELEMENT_KEY)
                            for the token t (as an unsigned 32-bit value) at place j of its sequence
  context of row r        c_r = prompt_hash[q] + sum of e(j, tokens[o_q + j]) over j < r - o_q   (mod 2^64)
                            (q the sequence of row r, o_q its first row): the claimed tokens that
                            precede row r, each bound to its place, plus the caller's hash of the prompt
  expanded seed           s'_r = words 0,1 of Philox-4x32-10(counter (c_r low, c_r high, 0, 2), key seed_r)

and s'_r then takes the place of seed_r in RO(seed || i).  Parity unpinned:
nothing here is printed by the paper, so only properties pin it
(tests/test_oracle_seed_expansion.py).
"""
from __future__ import annotations

import numpy as np

from . import philox4x32_10

MASK64 = (1 << 64) - 1
ELEMENT_KEY = (0x243F6A88, 0x85A308D3)  # the first 64 fraction bits of pi


def _two_words(block) -> int:
    return int(block[0]) | (int(block[1]) << 32)


def element_word(place: int, token: int) -> int:
    return _two_words(philox4x32_10([place & 0xFFFFFFFF, token & 0xFFFFFFFF, 0, 1], list(ELEMENT_KEY)))


def context_hashes(tokens, seq_offsets, prompt_hashes=None) -> list[int]:
    """c_r for every row: what precedes row r inside its own sequence."""
    tokens = [int(t) for t in tokens]
    seq_offsets = [int(o) for o in seq_offsets]
    out = [0] * len(tokens)
    for q in range(len(seq_offsets) - 1):
        c = 0 if prompt_hashes is None else int(prompt_hashes[q]) & MASK64
        for r in range(seq_offsets[q], seq_offsets[q + 1]):
            out[r] = c
            c = (c + element_word(r - seq_offsets[q], tokens[r])) & MASK64
    return out


def expand_seeds(seeds, tokens, seq_offsets, prompt_hashes=None) -> np.ndarray:
    """s'_r for every row."""
    ctx = context_hashes(tokens, seq_offsets, prompt_hashes)
    out = np.zeros(len(ctx), dtype=np.uint64)
    for r, c in enumerate(ctx):
        seed = int(seeds[r]) & MASK64
        blk = philox4x32_10([c & 0xFFFFFFFF, c >> 32, 0, 2], [seed & 0xFFFFFFFF, seed >> 32])
        out[r] = _two_words(blk)
    return out
