"""Seeded synthetic workloads for the token-scoring path.

This module only draws random inputs of the right shape and distribution; it
holds none of the method's arithmetic.  Whoever needs claimed tokens passes in a
sampler (the tests pass the CPU oracle's, the benchmark its own), so the same
generators serve every consumer.

The five workloads stand in for the paper's evaluation set-up (500-token
generations from four instruction-tuned models, Sec. "Experimental Set up"), whose
prompts and weights are not available: hidden states h ~ N(0,1) and LM-head rows
W ~ N(0, 1/d), both rounded to bf16, give unit-variance logits over vocabularies
of the same sizes as those models.
"""
from __future__ import annotations

import os
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, field, replace

import numpy as np

_CHUNK = 1 << 22


@dataclass(frozen=True)
class Workload:
    name: str
    index: int            # 1..5, enters every generator seed
    T: int                # token rows
    d: int                # hidden size
    V: int                # vocabulary size
    seq_len: int          # tokens per sequence; T is a multiple of it
    temperatures: tuple   # sampling temperatures the workload is run at
    h_noise_var: float    # variance of the inference-side perturbation of h (0: none)
    tamper_frac: float    # fraction of rows whose claim is replaced
    tamper_kind: str      # "uniform" | "runner_up" | "mixed"
    single_seed: bool = False
    sweep_T: tuple = field(default_factory=tuple)


WORKLOADS = {
    "tiny": Workload("tiny", 1, 256, 512, 4096, 256, (1.0,), 0.0, 0.05, "uniform", single_seed=True),
    "llama3b": Workload("llama3b", 2, 4096, 3072, 128256, 512, (0.7, 1.0), 1e-3, 0.02, "uniform"),
    "llama8b": Workload("llama8b", 3, 16384, 4096, 128256, 512, (1.0,), 1e-3, 0.01, "runner_up"),
    "moe30b": Workload("moe30b", 4, 65536, 2048, 151936, 512, (0.7,), 2e-3, 0.005, "mixed"),
    "longstream": Workload("longstream", 5, 4096, 5120, 152064, 1024, (1.0,), 0.0, 0.001, "uniform",
                           sweep_T=(4096, 32768, 131072, 262144)),
}

TINY_SEED = 0x9E3779B97F4A7C15


def with_T(w: Workload, T: int) -> Workload:
    """The same workload with another number of rows (whole sequences)."""
    if T % w.seq_len:
        raise ValueError("T must be a whole number of sequences")
    return replace(w, T=T)


def stream_seed(w: Workload, stream: int) -> int:
    """Generator seeds: 1000*stream + workload index (1 h, 2 W, 3 tamper, 4 seeds, 5 perturbation)."""
    return 1000 * stream + w.index


def splitmix64(x: int) -> int:
    m = (1 << 64) - 1
    z = (x + 0x9E3779B97F4A7C15) & m
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & m
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & m
    return z ^ (z >> 31)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even conversion of finite float32 values to bf16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _normal_chunk(args):
    seed, idx, n, std, out = args
    g = np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, idx])))
    x = g.standard_normal(n, dtype=np.float32)
    if std != 1.0:
        x *= np.float32(std)
    out[idx * _CHUNK: idx * _CHUNK + n] = x


def normal_f32(n: int, std: float, seed: int) -> np.ndarray:
    """n draws of N(0, std^2); the result does not depend on the thread count."""
    out = np.empty(n, dtype=np.float32)
    jobs = [(seed, i, min(_CHUNK, n - i * _CHUNK), std, out) for i in range((n + _CHUNK - 1) // _CHUNK)]
    workers = min(len(jobs), os.cpu_count() or 1, 32)
    if workers <= 1:
        for j in jobs:
            _normal_chunk(j)
    else:
        with ThreadPoolExecutor(workers) as ex:
            list(ex.map(_normal_chunk, jobs))
    return out


def normal_bf16(shape, std: float, seed: int) -> np.ndarray:
    n = int(np.prod(shape))
    return f32_to_bf16_bits(normal_f32(n, std, seed)).reshape(shape)


@dataclass
class Inputs:
    workload: Workload
    h: np.ndarray            # uint16 [T, d]: bf16 bits the verifier scores
    W: np.ndarray            # uint16 [V, d]
    h_server: np.ndarray     # uint16 [T, d]: what the inference server saw (h plus its perturbation)
    seeds: np.ndarray        # uint64 [T]
    positions: np.ndarray    # uint32 [T]: response index within the sequence, from 1
    seq_offsets: np.ndarray  # int32 [n_seq + 1]


def make_W(w: Workload) -> np.ndarray:
    return normal_bf16((w.V, w.d), float(1.0 / np.sqrt(w.d)), stream_seed(w, 2))


def make_row_metadata(w: Workload):
    n_seq = w.T // w.seq_len
    if w.single_seed:
        per_seq = np.full(n_seq, TINY_SEED, dtype=np.uint64)
    else:
        base = stream_seed(w, 4)
        per_seq = np.array([splitmix64(base + s) for s in range(n_seq)], dtype=np.uint64)
    seeds = np.repeat(per_seq, w.seq_len)
    positions = np.tile(np.arange(1, w.seq_len + 1, dtype=np.uint32), n_seq)
    seq_offsets = (np.arange(n_seq + 1, dtype=np.int64) * w.seq_len).astype(np.int32)
    return seeds, positions, seq_offsets


def make_inputs(w: Workload, W: np.ndarray | None = None) -> Inputs:
    h = normal_bf16((w.T, w.d), 1.0, stream_seed(w, 1))
    if W is None:
        W = make_W(w)
    if w.h_noise_var > 0.0:
        noise = normal_f32(w.T * w.d, float(np.sqrt(w.h_noise_var)), stream_seed(w, 5)).reshape(w.T, w.d)
        h_server = f32_to_bf16_bits(bf16_bits_to_f32(h) + noise)
    else:
        h_server = h
    seeds, positions, seq_offsets = make_row_metadata(w)
    return Inputs(w, h, W, h_server, seeds, positions, seq_offsets)


def tamper(w: Workload, honest: np.ndarray, runner_up: np.ndarray):
    """Replace a seeded fraction of the honest claims; returns (tokens, tampered mask).

    "uniform": a uniformly random *other* id; "runner_up": the sampler's second
    choice under the seeded noise; "mixed": alternately one and the other."""
    T = honest.shape[0]
    g = np.random.Generator(np.random.PCG64(np.random.SeedSequence([stream_seed(w, 3)])))
    n_bad = int(round(w.tamper_frac * T))
    rows = np.sort(g.choice(T, size=n_bad, replace=False)) if n_bad else np.zeros(0, dtype=np.int64)
    other = (honest[rows] + 1 + g.integers(0, w.V - 1, size=n_bad)) % w.V
    tokens = honest.astype(np.int32).copy()
    if w.tamper_kind == "uniform":
        tokens[rows] = other
    elif w.tamper_kind == "runner_up":
        tokens[rows] = runner_up[rows]
    elif w.tamper_kind == "mixed":
        pick = (np.arange(n_bad) % 2) == 0
        tokens[rows] = np.where(pick, runner_up[rows], other)
    else:
        raise ValueError(w.tamper_kind)
    mask = np.zeros(T, dtype=bool)
    mask[rows] = True
    return tokens, mask


def sample_rows(w: Workload, n: int, salt: int = 0) -> np.ndarray:
    """A seeded, sorted subset of row indices (for checks that cannot afford every row)."""
    g = np.random.Generator(np.random.PCG64(np.random.SeedSequence([stream_seed(w, 6), salt])))
    n = min(n, w.T)
    return np.sort(g.choice(w.T, size=n, replace=False))
