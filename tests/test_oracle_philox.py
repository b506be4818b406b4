"""Pins for the oracle's random oracle RO(seed || i): Philox-4x32-10, the
uniform mapping and the Gumbel transform."""
import ctypes
import ctypes.util
import math
import os

import mpmath
import numpy as np
import pytest

import oracle

PHILOX4_32_10 = 161  # curandRngType: CURAND_RNG_PSEUDO_PHILOX4_32_10


def _curand():
    for name in ("libcurand.so.10", "/usr/local/cuda/lib64/libcurand.so.10", ctypes.util.find_library("curand")):
        if not name:
            continue
        try:
            return ctypes.CDLL(name)
        except OSError:
            continue
    pytest.skip("cuRAND host library not found")


def _curand_words(lib, seed, offset, n):
    gen = ctypes.c_void_p()
    assert lib.curandCreateGeneratorHost(ctypes.byref(gen), PHILOX4_32_10) == 0
    try:
        assert lib.curandSetPseudoRandomGeneratorSeed(gen, ctypes.c_ulonglong(seed)) == 0
        assert lib.curandSetGeneratorOffset(gen, ctypes.c_ulonglong(offset)) == 0
        out = np.zeros(n, dtype=np.uint32)
        assert lib.curandGenerate(gen, out.ctypes.data_as(ctypes.c_void_p), ctypes.c_size_t(n)) == 0
        return out
    finally:
        lib.curandDestroyGenerator(gen)


def test_philox_matches_curand_host_generator():
    """cuRAND's host Philox generator is an independent implementation of the
    published algorithm.  It interleaves 65536 subsequences: the B-th block of
    four output words is the block of subsequence B mod 65536 at counter
    B div 65536.  Key words, counter words 0..2 and all four output lanes are
    exercised; a wrong constant, a swapped multiplier or a mis-ordered output
    word fails."""
    lib = _curand()
    rng = np.random.default_rng(7)
    n_blocks = 48
    for trial in range(40):
        seed = int(rng.integers(0, 2**64, dtype=np.uint64))
        first = int(rng.integers(0, 2**61)) if trial % 2 else int(rng.integers(0, 2**24))
        words = _curand_words(lib, seed, 4 * first, 4 * n_blocks).reshape(n_blocks, 4)
        key = [seed & 0xFFFFFFFF, seed >> 32]
        for j in range(n_blocks):
            counter, sub = divmod(first + j, 65536)
            mine = oracle.philox4x32_10([counter & 0xFFFFFFFF, counter >> 32, sub, 0], key)
            assert np.array_equal(mine, words[j]), (hex(seed), first, j)


def test_philox_known_answer_vectors():
    """Three stored vectors (all-zero, all-one and pi-digit inputs); unlike the cuRAND comparison this needs no
    library.  The fixture's header says where they come from: the cuRAND comparison above is the authority."""
    path = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")
    rows = [ln.split() for ln in open(path) if ln.strip() and not ln.startswith("#")]
    assert len(rows) == 3
    for words in rows:
        w = [int(x, 16) for x in words]
        assert len(w) == 10
        out = oracle.philox4x32_10(w[0:4], w[4:6])
        assert [int(x) for x in out] == w[6:10]


def test_philox_is_a_bijection_of_the_counter_low_bits():
    """A counter-mode block cipher never maps two counters to one block."""
    key = [0xDEADBEEF, 0x12345678]
    seen = set()
    for c in range(2048):
        seen.add(tuple(int(x) for x in oracle.philox4x32_10([c, 5, 0, 0], key)))
    assert len(seen) == 2048


def test_ro_word_layout():
    """Noise id v reads word v & 3 of the block at counter (v >> 2, position, tag, 0)."""
    seed, pos = 0x0123456789ABCDEF, 77
    key = [seed & 0xFFFFFFFF, seed >> 32]
    for tag in (0, 1):
        for v in (0, 1, 2, 3, 4, 7, 1023, 128255, 151935):
            blk = oracle.philox4x32_10([v >> 2, pos, tag, 0], key)
            assert oracle.ro_word(seed, pos, tag, v) == int(blk[v & 3])


def test_uniform_is_the_exact_midpoint_rational():
    for word in (0, 1, 511, 512, 0x7FFFFFFF, 0x80000000, 0xFFFFFE00, 0xFFFFFFFF, 123456789):
        u = oracle.uniform23(word)
        assert u == (2 * (word >> 9) + 1) / 2**24  # exact in binary floating point
        assert 0.0 < u < 1.0
        mu = oracle.uniform32(word)
        assert mu == (2 * word + 1) / 2**33
        assert 0.0 < mu < 1.0


def test_gumbel_matches_50_digit_arithmetic():
    mpmath.mp.dps = 50
    words = [0, 511, 512, 1 << 20, 0x7FFFFFFF, 0x80000000, 0xFFFFFDFF, 0xFFFFFE00, 0xFFFFFFFF, 0xC0FFEE00]
    for word in words:
        u = mpmath.mpf(2 * (word >> 9) + 1) / 2**24
        want = -mpmath.log(-mpmath.log(u))
        got = oracle.gumbel(word)
        assert abs(got - float(want)) <= 1e-13 * max(1.0, abs(float(want))), word
    assert oracle.gumbel(0) == pytest.approx(-math.log(-math.log(2.0**-24)), rel=1e-15)
    assert -2.82 < oracle.gumbel(0) < -2.80
    assert 16.6 < oracle.gumbel(0xFFFFFFFF) < 16.7


def test_gumbel_moments_over_the_seeded_stream():
    """Mean Euler-Mascheroni, variance pi^2/6 for Gumbel(0,1)."""
    g = oracle.gumbel_noise_row(0xABCDEF0123456789, 3, 200_000)
    assert abs(g.mean() - 0.5772156649) < 4 * math.sqrt(math.pi**2 / 6 / g.size)
    assert abs(g.var() - math.pi**2 / 6) < 0.03
    u = np.exp(-np.exp(-g))  # back to the uniform: should fill (0,1) evenly
    hist, _ = np.histogram(u, bins=20, range=(0, 1))
    chi2 = float(((hist - g.size / 20) ** 2 / (g.size / 20)).sum())
    assert chi2 < 50.0  # 19 dof, p ~ 1e-4


def test_streams_differ_by_seed_position_and_tag():
    a = [oracle.ro_word(1, 1, 0, v) for v in range(64)]
    assert a != [oracle.ro_word(2, 1, 0, v) for v in range(64)]
    assert a != [oracle.ro_word(1, 2, 0, v) for v in range(64)]
    assert a != [oracle.ro_word(1, 1, 1, v) for v in range(64)]
    assert a != [oracle.ro_word(1 << 32, 1, 0, v) for v in range(64)]
