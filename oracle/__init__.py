"""fp64 CPU oracle for the verifier's token-scoring path -- TEST INFRASTRUCTURE.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import
this package.  It shares nothing with the CUDA path: `difr_oracle.c` is plain C
compiled with gcc, `posterior.py` is plain numpy.

`build()` compiles the C file next to it; `lib()` loads it.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "difr_oracle.c")
_SO = os.path.join(_HERE, "libdifr_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle (gcc -O2 -fopenmp); returns the path of the library."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-Wall", "-Wextra", "-o", _SO, _SRC, "-lm"]
        )
    return _SO


class _GmOut(ctypes.Structure):
    _fields_ = [
        ("score", ctypes.c_void_p), ("margin", ctypes.c_void_p), ("argmax", ctypes.c_void_p),
        ("runner_up", ctypes.c_void_p), ("top2_margin", ctypes.c_void_p), ("lse", ctypes.c_void_p),
        ("y_claimed", ctypes.c_void_p), ("logit_claimed", ctypes.c_void_p), ("rank", ctypes.c_void_p),
        ("match", ctypes.c_void_p), ("row_status", ctypes.c_void_p), ("top23_margin", ctypes.c_void_p),
    ]


class _IptOut(ctypes.Structure):
    _fields_ = [
        ("score", ctypes.c_void_p), ("p_claimed", ctypes.c_void_p), ("cdf_lo", ctypes.c_void_p),
        ("u", ctypes.c_void_p), ("lse", ctypes.c_void_p), ("mass", ctypes.c_void_p),
        ("sampled", ctypes.c_void_p), ("row_status", ctypes.c_void_p),
    ]


SEQ_STATS_DTYPE = np.dtype([("n_flagged", "<i4"), ("n_match", "<i4"), ("sum", "<f8"), ("min", "<f8")])


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        L.oracle_ro_word.restype = ctypes.c_uint32
        L.oracle_ro_word.argtypes = [ctypes.c_uint64, ctypes.c_uint32, ctypes.c_uint32, ctypes.c_uint32]
        for name in ("oracle_uniform23", "oracle_uniform32", "oracle_gumbel"):
            getattr(L, name).restype = ctypes.c_double
            getattr(L, name).argtypes = [ctypes.c_uint32]
        L.oracle_gumbel_noise.restype = ctypes.c_double
        L.oracle_gumbel_noise.argtypes = [ctypes.c_uint64, ctypes.c_uint32, ctypes.c_uint32]
        L.oracle_gumbel_row.restype = None
        L.oracle_gumbel_row.argtypes = [ctypes.c_uint64, ctypes.c_uint32, ctypes.c_int64, ctypes.c_void_p]
        L.oracle_ipt_uniform.restype = ctypes.c_double
        L.oracle_ipt_uniform.argtypes = [ctypes.c_uint64, ctypes.c_uint32]
        L.oracle_normal_cdf.restype = ctypes.c_double
        L.oracle_normal_cdf.argtypes = [ctypes.c_double]
        L.oracle_normal_interval_mass.restype = ctypes.c_double
        L.oracle_normal_interval_mass.argtypes = [ctypes.c_double, ctypes.c_double]
        L.oracle_gm_pi.restype = ctypes.c_double
        L.oracle_gm_pi.argtypes = [ctypes.c_double, ctypes.c_double]
        L.oracle_gm_score.restype = ctypes.c_double
        L.oracle_gm_score.argtypes = [ctypes.c_double, ctypes.c_double, ctypes.c_double]
        L.oracle_ipt_mass.restype = ctypes.c_double
        L.oracle_ipt_mass.argtypes = [ctypes.c_double] * 4
        L.oracle_ipt_score.restype = ctypes.c_double
        L.oracle_ipt_score.argtypes = [ctypes.c_double] * 5
        L.oracle_philox4x32_10.restype = None
        L.oracle_philox4x32_10.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
        L.oracle_logits.restype = ctypes.c_int
        L.oracle_logits.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64,
                                    ctypes.c_int64, ctypes.c_void_p]
        common = [ctypes.c_void_p] * 5 + [ctypes.c_double] * 3 + [ctypes.c_int64] * 3
        L.oracle_score_gm.restype = ctypes.c_int
        L.oracle_score_gm.argtypes = common + [ctypes.c_void_p, ctypes.POINTER(_GmOut)]
        L.oracle_score_ipt.restype = ctypes.c_int
        L.oracle_score_ipt.argtypes = common + [ctypes.POINTER(_IptOut)]
        L.oracle_score_both.restype = ctypes.c_int
        L.oracle_score_both.argtypes = [ctypes.c_void_p] * 6 + [ctypes.c_double] * 4 + [ctypes.c_int64] * 3 + [
            ctypes.POINTER(_GmOut), ctypes.POINTER(_IptOut)]
        L.oracle_detect.restype = ctypes.c_int
        L.oracle_detect.argtypes = [ctypes.c_void_p, ctypes.c_double, ctypes.c_void_p, ctypes.c_void_p,
                                    ctypes.c_int64, ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p]
        L.oracle_classify.restype = ctypes.c_int
        L.oracle_classify.argtypes = [ctypes.c_void_p, ctypes.c_double, ctypes.c_void_p, ctypes.c_int32,
                                      ctypes.c_int64, ctypes.c_void_p]
        L.oracle_admissible_count.restype = ctypes.c_int
        L.oracle_admissible_count.argtypes = [ctypes.c_void_p] * 4 + [ctypes.c_double] * 4 + [ctypes.c_int64] * 3 + [
            ctypes.c_void_p]
        L.oracle_exfiltratable_bits.restype = ctypes.c_int
        L.oracle_exfiltratable_bits.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64,
                                                ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64, ctypes.c_void_p,
                                                ctypes.c_void_p]
        L.oracle_num_threads.restype = ctypes.c_int
        _lib = L
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _bf16_bits(a, shape):
    a = np.ascontiguousarray(a)
    if a.dtype != np.uint16 or a.shape != tuple(shape):
        raise ValueError(f"expected bf16 bit patterns as uint16 with shape {shape}, got {a.dtype} {a.shape}")
    return a


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def philox4x32_10(ctr, key) -> np.ndarray:
    c = np.ascontiguousarray(ctr, dtype=np.uint32)
    k = np.ascontiguousarray(key, dtype=np.uint32)
    out = np.zeros(4, dtype=np.uint32)
    lib().oracle_philox4x32_10(_p(c), _p(k), _p(out))
    return out


def ro_word(seed: int, position: int, tag: int, idx: int) -> int:
    return int(lib().oracle_ro_word(seed, position, tag, idx))


def uniform23(word: int) -> float:
    return float(lib().oracle_uniform23(word))


def uniform32(word: int) -> float:
    return float(lib().oracle_uniform32(word))


def gumbel(word: int) -> float:
    return float(lib().oracle_gumbel(word))


def gumbel_noise(seed: int, position: int, idx: int) -> float:
    return float(lib().oracle_gumbel_noise(seed, position, idx))


def gumbel_noise_row(seed: int, position: int, V: int) -> np.ndarray:
    out = np.zeros(V, dtype=np.float64)
    lib().oracle_gumbel_row(int(seed), int(position), int(V), _p(out))
    return out


def ipt_uniform(seed: int, position: int) -> float:
    return float(lib().oracle_ipt_uniform(seed, position))


def gm_pi(A: float, sigma: float) -> float:
    return float(lib().oracle_gm_pi(A, sigma))


def gm_score(A: float, sigma: float, eps: float) -> float:
    return float(lib().oracle_gm_score(A, sigma, eps))


def ipt_mass(a: float, b: float, mu: float, sigma: float) -> float:
    return float(lib().oracle_ipt_mass(a, b, mu, sigma))


def ipt_score(a: float, b: float, mu: float, sigma: float, eps: float) -> float:
    return float(lib().oracle_ipt_score(a, b, mu, sigma, eps))


def normal_interval_mass(za: float, zb: float) -> float:
    return float(lib().oracle_normal_interval_mass(za, zb))


def logits(h_bits, W_bits) -> np.ndarray:
    """All T x V logits in fp64 (small shapes only)."""
    T, d = h_bits.shape
    V = W_bits.shape[0]
    h_bits = _bf16_bits(h_bits, (T, d))
    W_bits = _bf16_bits(W_bits, (V, d))
    out = np.zeros((T, V), dtype=np.float64)
    rc = lib().oracle_logits(_p(h_bits), _p(W_bits), T, d, V, _p(out))
    if rc != 0:
        raise RuntimeError(f"oracle_logits failed: {rc}")
    return out


@dataclass
class GmResult:
    score: np.ndarray
    margin: np.ndarray
    argmax: np.ndarray
    runner_up: np.ndarray
    top2_margin: np.ndarray
    lse: np.ndarray
    y_claimed: np.ndarray
    logit_claimed: np.ndarray
    rank: np.ndarray
    match: np.ndarray
    row_status: np.ndarray
    top23_margin: np.ndarray


@dataclass
class IptResult:
    score: np.ndarray
    p_claimed: np.ndarray
    cdf_lo: np.ndarray
    u: np.ndarray
    lse: np.ndarray
    mass: np.ndarray
    sampled: np.ndarray
    row_status: np.ndarray


def _row_inputs(tokens, seeds, positions, T):
    tokens = np.ascontiguousarray(tokens, dtype=np.int32)
    seeds = np.ascontiguousarray(seeds, dtype=np.uint64)
    positions = np.ascontiguousarray(positions, dtype=np.uint32)
    if tokens.shape != (T,) or seeds.shape != (T,) or positions.shape != (T,):
        raise ValueError("tokens, seeds and positions must have shape (T,)")
    return tokens, seeds, positions


def score_gm(h_bits, W_bits, tokens, seeds, positions, temperature, sigma, eps=1e-12, noise_id=None) -> GmResult:
    """Token-DiFR (Gumbel-max) scores of every row, one competitor, Gaussian noise."""
    T, d = h_bits.shape
    V = W_bits.shape[0]
    h_bits = _bf16_bits(h_bits, (T, d))
    W_bits = _bf16_bits(W_bits, (V, d))
    tokens, seeds, positions = _row_inputs(tokens, seeds, positions, T)
    if noise_id is not None:
        noise_id = np.ascontiguousarray(noise_id, dtype=np.int32)
        assert noise_id.shape == (V,)
    f8 = lambda: np.zeros(T, dtype=np.float64)
    i4 = lambda: np.zeros(T, dtype=np.int32)
    res = GmResult(f8(), f8(), i4(), i4(), f8(), f8(), f8(), f8(), i4(), i4(), np.zeros(T, dtype=np.uint32), f8())
    out = _GmOut(*[_p(getattr(res, name)) for name, _ in _GmOut._fields_])
    rc = lib().oracle_score_gm(_p(h_bits), _p(W_bits), _p(tokens), _p(seeds), _p(positions), float(temperature),
                               float(sigma), float(eps), T, d, V, _p(noise_id), ctypes.byref(out))
    if rc != 0:
        raise RuntimeError(f"oracle_score_gm failed: {rc}")
    return res


def sample_gm(h_bits, W_bits, seeds, positions, temperature):
    """The Gumbel-max sampler on every row: (sampled token, runner-up token)."""
    T = h_bits.shape[0]
    res = score_gm(h_bits, W_bits, np.zeros(T, dtype=np.int32), seeds, positions, temperature, 1.0)
    return res.argmax.copy(), res.runner_up.copy()


def score_ipt(h_bits, W_bits, tokens, seeds, positions, temperature, sigma, eps=1e-12) -> IptResult:
    """Token-IPT-DiFR scores of every row."""
    T, d = h_bits.shape
    V = W_bits.shape[0]
    h_bits = _bf16_bits(h_bits, (T, d))
    W_bits = _bf16_bits(W_bits, (V, d))
    tokens, seeds, positions = _row_inputs(tokens, seeds, positions, T)
    f8 = lambda: np.zeros(T, dtype=np.float64)
    res = IptResult(f8(), f8(), f8(), f8(), f8(), f8(), np.zeros(T, dtype=np.int32), np.zeros(T, dtype=np.uint32))
    out = _IptOut(*[_p(getattr(res, name)) for name, _ in _IptOut._fields_])
    rc = lib().oracle_score_ipt(_p(h_bits), _p(W_bits), _p(tokens), _p(seeds), _p(positions), float(temperature),
                                float(sigma), float(eps), T, d, V, ctypes.byref(out))
    if rc != 0:
        raise RuntimeError(f"oracle_score_ipt failed: {rc}")
    return res


def score_both(h_bits, W_bits, tokens_gm, tokens_ipt, seeds, positions, temperature, sigma_gm, sigma_ipt,
               eps=1e-12):
    """`score_gm` on tokens_gm and `score_ipt` on tokens_ipt from one evaluation of each row's logits."""
    T, d = h_bits.shape
    V = W_bits.shape[0]
    h_bits = _bf16_bits(h_bits, (T, d))
    W_bits = _bf16_bits(W_bits, (V, d))
    tokens_gm, seeds, positions = _row_inputs(tokens_gm, seeds, positions, T)
    tokens_ipt = np.ascontiguousarray(tokens_ipt, dtype=np.int32)
    if tokens_ipt.shape != (T,):
        raise ValueError("tokens_ipt must have shape (T,)")
    f8 = lambda: np.zeros(T, dtype=np.float64)
    i4 = lambda: np.zeros(T, dtype=np.int32)
    gm = GmResult(f8(), f8(), i4(), i4(), f8(), f8(), f8(), f8(), i4(), i4(), np.zeros(T, dtype=np.uint32), f8())
    ipt = IptResult(f8(), f8(), f8(), f8(), f8(), f8(), i4(), np.zeros(T, dtype=np.uint32))
    gm_out = _GmOut(*[_p(getattr(gm, name)) for name, _ in _GmOut._fields_])
    ipt_out = _IptOut(*[_p(getattr(ipt, name)) for name, _ in _IptOut._fields_])
    rc = lib().oracle_score_both(_p(h_bits), _p(W_bits), _p(tokens_gm), _p(tokens_ipt), _p(seeds), _p(positions),
                                 float(temperature), float(sigma_gm), float(sigma_ipt), float(eps), T, d, V,
                                 ctypes.byref(gm_out), ctypes.byref(ipt_out))
    if rc != 0:
        raise RuntimeError(f"oracle_score_both failed: {rc}")
    return gm, ipt


def sample_ipt(h_bits, W_bits, seeds, positions, temperature) -> np.ndarray:
    """The inverse-probability-transform sampler on every row."""
    T = h_bits.shape[0]
    return score_ipt(h_bits, W_bits, np.zeros(T, dtype=np.int32), seeds, positions, temperature, 1.0).sampled.copy()


def detect(scores, threshold, margins=None, seq_offsets=None):
    """Threshold flags and per-sequence pooled statistics."""
    scores = np.ascontiguousarray(scores, dtype=np.float64)
    T = scores.shape[0]
    if margins is not None:
        margins = np.ascontiguousarray(margins, dtype=np.float64)
    n_seq = 1
    if seq_offsets is not None:
        seq_offsets = np.ascontiguousarray(seq_offsets, dtype=np.int32)
        n_seq = seq_offsets.shape[0] - 1
    flags = np.zeros(T, dtype=np.uint8)
    stats = np.zeros(n_seq, dtype=SEQ_STATS_DTYPE)
    rc = lib().oracle_detect(_p(scores), float(threshold), _p(margins), _p(seq_offsets), n_seq, T, _p(flags),
                             _p(stats))
    if rc != 0:
        raise RuntimeError(f"oracle_detect failed: {rc}")
    return flags, stats


def classify(scores, threshold, ranks=None, rank_cutoff=0) -> np.ndarray:
    """Risk class per token: 0 safe, 1 suspicious, 2 dangerous (Alg. "Per-Token Risk Classification")."""
    scores = np.ascontiguousarray(scores, dtype=np.float64)
    T = scores.shape[0]
    if ranks is not None:
        ranks = np.ascontiguousarray(ranks, dtype=np.int32)
    classes = np.zeros(T, dtype=np.uint8)
    rc = lib().oracle_classify(_p(scores), float(threshold), _p(ranks), int(rank_cutoff), T, _p(classes))
    if rc != 0:
        raise RuntimeError(f"oracle_classify failed: {rc}")
    return classes


def admissible_count(h_bits, W_bits, seeds, positions, temperature, sigma, tau, eps=1e-12) -> np.ndarray:
    """|A_t(tau)| per row: how many vocabulary ids would score >= tau if they were the claim."""
    T, d = h_bits.shape
    V = W_bits.shape[0]
    h_bits = _bf16_bits(h_bits, (T, d))
    W_bits = _bf16_bits(W_bits, (V, d))
    seeds = np.ascontiguousarray(seeds, dtype=np.uint64)
    positions = np.ascontiguousarray(positions, dtype=np.uint32)
    counts = np.zeros(T, dtype=np.int32)
    rc = lib().oracle_admissible_count(_p(h_bits), _p(W_bits), _p(seeds), _p(positions), float(temperature),
                                       float(sigma), float(eps), float(tau), T, d, V, _p(counts))
    if rc != 0:
        raise RuntimeError(f"oracle_admissible_count failed: {rc}")
    return counts


def exfiltratable_bits(classes, counts, rank_cutoff, V, seq_offsets=None):
    """(bits per token, bits per sequence) from the risk classes and admissible-set sizes."""
    classes = np.ascontiguousarray(classes, dtype=np.uint8)
    counts = np.ascontiguousarray(counts, dtype=np.int32)
    T = classes.shape[0]
    n_seq = 1
    if seq_offsets is not None:
        seq_offsets = np.ascontiguousarray(seq_offsets, dtype=np.int32)
        n_seq = seq_offsets.shape[0] - 1
    bits = np.zeros(T, dtype=np.float64)
    seq_bits = np.zeros(n_seq, dtype=np.float64)
    rc = lib().oracle_exfiltratable_bits(_p(classes), _p(counts), int(rank_cutoff), int(V), _p(seq_offsets), n_seq,
                                         T, _p(bits), _p(seq_bits))
    if rc != 0:
        raise RuntimeError(f"oracle_exfiltratable_bits failed: {rc}")
    return bits, seq_bits
