"""Thin binding of libdifr.so, the B200 token-scoring library.

The functions carry the names of the C entry points in include/difr.h and only
marshal arguments: torch supplies device memory and streams, every step of the
scoring path runs in the library's CUDA kernels.  There is no CPU fallback: a
missing or unloadable library raises.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "csrc", "libdifr.so")

DIFR_OK = 0
STATUS_NAMES = {0: "DIFR_OK", -1: "DIFR_ERR_INVALID_ARG", -2: "DIFR_ERR_SHAPE", -3: "DIFR_ERR_ALIGN",
                -4: "DIFR_ERR_WORKSPACE", -5: "DIFR_ERR_CUDA", -6: "DIFR_ERR_ARCH", -7: "DIFR_ERR_TIMEOUT"}

EXPORTS = ("difr_workspace_bytes", "difr_filtered_workspace_bytes", "difr_score_gm", "difr_score_ipt",
           "difr_score_both", "difr_score_gm_filtered", "difr_score_ipt_filtered", "difr_score_gm_static",
           "difr_admissible", "difr_exfiltratable_bits", "difr_detect", "difr_expand_seeds", "difr_logits", "difr_philox",
           "difr_selftest_wait", "difr_debug_plan_override", "difr_status_string", "difr_version")
STATIC_SCRATCH_BYTES = 16 << 20  # DIFR_STATIC_SCRATCH_BYTES


class DifrError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)}")


class _COut(ctypes.Structure):
    _fields_ = [
        ("sigma", ctypes.c_float), ("eps", ctypes.c_float),
        ("score", ctypes.c_void_p), ("margin", ctypes.c_void_p), ("argmax", ctypes.c_void_p),
        ("runner_up", ctypes.c_void_p), ("lse", ctypes.c_void_p), ("p_claimed", ctypes.c_void_p),
        ("cdf_lo", ctypes.c_void_p), ("u", ctypes.c_void_p), ("row_status", ctypes.c_void_p),
        ("workspace", ctypes.c_void_p), ("workspace_bytes", ctypes.c_size_t), ("device_status", ctypes.c_void_p),
        ("event_fused_start", ctypes.c_void_p), ("event_fused_stop", ctypes.c_void_p),
        ("rank", ctypes.c_void_p), ("y_max", ctypes.c_void_p), ("y_second", ctypes.c_void_p),
        ("sigma_ipt", ctypes.c_float), ("score_ipt", ctypes.c_void_p), ("cutoff", ctypes.c_void_p),
        ("temperatures", ctypes.c_void_p),
    ]


class _CFilter(ctypes.Structure):
    _fields_ = [("top_k", ctypes.c_int32), ("top_p", ctypes.c_float), ("s", ctypes.c_int32),
                ("top_k_rows", ctypes.c_void_p), ("top_p_rows", ctypes.c_void_p),
                ("min_p", ctypes.c_float), ("min_p_rows", ctypes.c_void_p), ("any_size", ctypes.c_int32)]


_lib = None


def lib() -> ctypes.CDLL:
    """Loads csrc/libdifr.so (built by paper_2511_02620_b200.build.build())."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_2511_02620_b200.build` "
                              "(there is no fallback path)")
        L = ctypes.CDLL(LIB_PATH)
        L.difr_workspace_bytes.restype = ctypes.c_size_t
        L.difr_workspace_bytes.argtypes = [ctypes.c_int64] * 3
        score_args = [ctypes.c_void_p] * 5 + [ctypes.c_float] + [ctypes.c_int64] * 3 + [ctypes.POINTER(_COut),
                                                                                      ctypes.c_void_p]
        for name in ("difr_score_gm", "difr_score_ipt", "difr_score_both", "difr_score_gm_static"):
            getattr(L, name).restype = ctypes.c_int
            getattr(L, name).argtypes = score_args
        L.difr_detect.restype = ctypes.c_int
        L.difr_detect.argtypes = [ctypes.c_void_p, ctypes.c_float, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int32,
                                  ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p,
                                  ctypes.c_void_p]
        L.difr_filtered_workspace_bytes.restype = ctypes.c_size_t
        L.difr_filtered_workspace_bytes.argtypes = [ctypes.c_int64] * 3
        for name in ("difr_score_gm_filtered", "difr_score_ipt_filtered"):
            getattr(L, name).restype = ctypes.c_int
            getattr(L, name).argtypes = ([ctypes.c_void_p] * 5 + [ctypes.c_float] + [ctypes.c_int64] * 3
                                         + [ctypes.POINTER(_CFilter), ctypes.POINTER(_COut), ctypes.c_void_p])
        L.difr_admissible.restype = ctypes.c_int
        L.difr_admissible.argtypes = ([ctypes.c_void_p] * 4 + [ctypes.c_float] + [ctypes.c_int64] * 3
                                      + [ctypes.c_void_p] * 4 + [ctypes.c_float] * 2
                                      + [ctypes.POINTER(ctypes.c_float), ctypes.c_int32, ctypes.c_void_p,
                                         ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p,
                                         ctypes.c_void_p])
        L.difr_exfiltratable_bits.restype = ctypes.c_int
        L.difr_exfiltratable_bits.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64,
                                              ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64, ctypes.c_void_p,
                                              ctypes.c_void_p, ctypes.c_void_p]
        L.difr_expand_seeds.restype = ctypes.c_int
        L.difr_expand_seeds.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64,
                                        ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p]
        L.difr_logits.restype = ctypes.c_int
        L.difr_logits.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64, ctypes.c_int64,
                                  ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
        L.difr_philox.restype = ctypes.c_int
        L.difr_philox.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p]
        L.difr_selftest_wait.restype = ctypes.c_int
        L.difr_selftest_wait.argtypes = [ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p]
        L.difr_debug_plan_override.restype = ctypes.c_int
        L.difr_debug_plan_override.argtypes = [ctypes.c_int32] * 3
        L.difr_status_string.restype = ctypes.c_char_p
        L.difr_status_string.argtypes = [ctypes.c_int]
        L.difr_version.restype = ctypes.c_int
        _lib = L
    return _lib


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream):
    import torch

    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _check(t, dtype, shape, name):
    import torch

    if not isinstance(t, torch.Tensor) or not t.is_cuda or not t.is_contiguous():
        raise TypeError(f"{name} must be a contiguous CUDA tensor")
    if t.dtype != dtype or tuple(t.shape) != tuple(shape):
        raise TypeError(f"{name}: expected {dtype} {tuple(shape)}, got {t.dtype} {tuple(t.shape)}")


def difr_workspace_bytes(T: int, d: int, V: int) -> int:
    return int(lib().difr_workspace_bytes(T, d, V))


def difr_version() -> int:
    return int(lib().difr_version())


def difr_status_string(status: int) -> str:
    return lib().difr_status_string(status).decode()


@dataclass
class DifrOut:
    """Estimator parameters and output tensors of a scoring call (mirrors `difr_out`)."""
    sigma: float
    eps: float
    score: "object"
    margin: "object" = None
    argmax: "object" = None
    runner_up: "object" = None
    lse: "object" = None
    p_claimed: "object" = None
    cdf_lo: "object" = None
    u: "object" = None
    row_status: "object" = None
    workspace: "object" = None
    device_status: "object" = None
    event_fused_start: int = 0  # raw cudaEvent_t handles (0: none)
    event_fused_stop: int = 0
    rank: "object" = None       # int32 [T]: ask for the raw-logit rank of the claimed token (GM calls)
    y_max: "object" = None      # float [T]: largest / second largest l + Temp*G (GM calls); difr_admissible needs them
    y_second: "object" = None
    sigma_ipt: float = 0.0      # difr_score_both: width of the IPT estimator
    score_ipt: "object" = None  # difr_score_both: float [T]
    cutoff: "object" = None     # difr_score_gm_filtered: float [T], the filter's cutoff per row
    temperatures: "object" = None  # float [T]: one temperature per row instead of the call's scalar

    @staticmethod
    def allocate(T: int, d: int, V: int, sigma: float, eps: float = 1e-12, device="cuda"):
        import torch

        f = lambda: torch.empty(T, dtype=torch.float32, device=device)
        i = lambda: torch.empty(T, dtype=torch.int32, device=device)
        nbytes = max(difr_workspace_bytes(T, d, V), 16)
        return DifrOut(sigma, eps, f(), f(), i(), i(), f(), f(), f(), f(), i(),
                       torch.empty(nbytes, dtype=torch.uint8, device=device),
                       torch.zeros(1, dtype=torch.int32, device=device))

    def _c(self) -> _COut:
        ws = self.workspace
        return _COut(float(self.sigma), float(self.eps), _ptr(self.score), _ptr(self.margin), _ptr(self.argmax),
                     _ptr(self.runner_up), _ptr(self.lse), _ptr(self.p_claimed), _ptr(self.cdf_lo), _ptr(self.u),
                     _ptr(self.row_status), _ptr(ws), 0 if ws is None else ws.numel() * ws.element_size(),
                     _ptr(self.device_status), ctypes.c_void_p(self.event_fused_start or None),
                     ctypes.c_void_p(self.event_fused_stop or None), _ptr(self.rank), _ptr(self.y_max),
                     _ptr(self.y_second), float(self.sigma_ipt), _ptr(self.score_ipt), _ptr(self.cutoff),
                     _ptr(self.temperatures))


def _score(fn_name, h, W, tokens, seeds, positions, temperature, out: DifrOut, stream):
    import torch

    T, d = h.shape
    V = W.shape[0]
    _check(h, torch.bfloat16, (T, d), "h")
    _check(W, torch.bfloat16, (V, d), "W")
    _check(tokens, torch.int32, (T,), "tokens")
    _check(seeds, torch.int64, (T,), "seeds")  # uint64 bit patterns carried in int64 storage
    _check(positions, torch.int32, (T,), "positions")  # uint32 bit patterns
    c = out._c()
    rc = getattr(lib(), fn_name)(_ptr(h), _ptr(W), _ptr(tokens), _ptr(seeds), _ptr(positions), float(temperature),
                                 T, d, V, ctypes.byref(c), _stream(stream))
    if rc != DIFR_OK:
        raise DifrError(rc, fn_name)
    return out


def difr_score_gm(h, W, tokens, seeds, positions, temperature, out: DifrOut, stream=None) -> DifrOut:
    """Token-DiFR (Gumbel-max) scores; see include/difr.h."""
    return _score("difr_score_gm", h, W, tokens, seeds, positions, temperature, out, stream)


def difr_score_ipt(h, W, tokens, seeds, positions, temperature, out: DifrOut, stream=None) -> DifrOut:
    """Token-IPT-DiFR scores; see include/difr.h."""
    return _score("difr_score_ipt", h, W, tokens, seeds, positions, temperature, out, stream)


def difr_score_both(h, W, tokens, seeds, positions, temperature, out: DifrOut, stream=None) -> DifrOut:
    """Token-DiFR and Token-IPT-DiFR scores from one pass (`out.sigma_ipt`, `out.score_ipt`); see include/difr.h."""
    return _score("difr_score_both", h, W, tokens, seeds, positions, temperature, out, stream)


def difr_filtered_workspace_bytes(T: int, d: int, V: int) -> int:
    return int(lib().difr_filtered_workspace_bytes(T, d, V))


def difr_score_ipt_filtered(h, W, tokens, seeds, positions, temperature, top_k, top_p, out: DifrOut, stream=None,
                            min_p=0.0, any_size=False):
    """Token-IPT-DiFR on the filtered distribution; workspace as for difr_score_gm_filtered."""
    return difr_score_gm_filtered(h, W, tokens, seeds, positions, temperature, top_k, top_p, 1, out, stream,
                                  _fn="difr_score_ipt_filtered", min_p=min_p, any_size=any_size)


def difr_score_gm_filtered(h, W, tokens, seeds, positions, temperature, top_k, top_p, s, out: DifrOut, stream=None,
                           _fn="difr_score_gm_filtered", min_p=0.0, any_size=False):
    """Alg. Token-DiFR in full: top-k / top-p cutoff, B_i terms, s competitors; `out.workspace` must hold
    difr_filtered_workspace_bytes(T, d, V) bytes.  `top_k` (int32) and `top_p` (float32) may be device tensors
    of T values, one per row (`min_p` likewise), and `out.temperatures` one temperature per row; `any_size`
    lets such per-row values go beyond 128 kept ids.
    See include/difr.h."""
    import torch

    T, d = h.shape
    V = W.shape[0]
    _check(h, torch.bfloat16, (T, d), "h")
    _check(W, torch.bfloat16, (V, d), "W")
    _check(tokens, torch.int32, (T,), "tokens")
    _check(seeds, torch.int64, (T,), "seeds")
    _check(positions, torch.int32, (T,), "positions")
    c = out._c()
    k_rows = top_k if isinstance(top_k, torch.Tensor) else None
    p_rows = top_p if isinstance(top_p, torch.Tensor) else None
    if k_rows is not None:
        _check(k_rows, torch.int32, (T,), "top_k")
    if p_rows is not None:
        _check(p_rows, torch.float32, (T,), "top_p")
    m_rows = min_p if isinstance(min_p, torch.Tensor) else None
    if m_rows is not None:
        _check(m_rows, torch.float32, (T,), "min_p")
    f = _CFilter(0 if k_rows is not None else int(top_k), 1.0 if p_rows is not None else float(top_p), int(s),
                 _ptr(k_rows), _ptr(p_rows), 0.0 if m_rows is not None else float(min_p), _ptr(m_rows),
                 1 if any_size else 0)
    rc = getattr(lib(), _fn)(_ptr(h), _ptr(W), _ptr(tokens), _ptr(seeds), _ptr(positions),
                             float(temperature), T, d, V, ctypes.byref(f), ctypes.byref(c), _stream(stream))
    if rc != DIFR_OK:
        raise DifrError(rc, _fn)
    return out


def difr_admissible(h, W, seeds, positions, temperature, scored: DifrOut, taus, counts, row_status=None, stream=None):
    """Admissible-set sizes |A_t(tau)| for up to four thresholds; `scored` holds argmax, runner_up, y_max, y_second,
    sigma, eps and the workspace of a difr_score_gm call on the same inputs; `counts` is int32 [len(taus), T];
    `row_status` (uint32 bits in an int32 [T] tensor, optional) receives bit 5 for rows whose list overflowed."""
    import torch

    T, d = h.shape
    V = W.shape[0]
    taus = [float(t) for t in taus]
    _check(counts, torch.int32, (len(taus), T), "counts")
    arr = (ctypes.c_float * len(taus))(*taus)
    ws = scored.workspace
    rc = lib().difr_admissible(_ptr(h), _ptr(W), _ptr(seeds), _ptr(positions), float(temperature), T, d, V,
                               _ptr(scored.argmax), _ptr(scored.runner_up), _ptr(scored.y_max), _ptr(scored.y_second),
                               float(scored.sigma), float(scored.eps), arr, len(taus), _ptr(counts), _ptr(row_status),
                               _ptr(ws), ws.numel() * ws.element_size(), _ptr(scored.device_status), _stream(stream))
    if rc != DIFR_OK:
        raise DifrError(rc, "difr_admissible")
    return counts


def difr_exfiltratable_bits(classes, counts, rank_cutoff, V, seq_offsets=None, bits=None, seq_bits=None, stream=None):
    """Per-token / per-sequence information bound from the risk classes and admissible-set sizes."""
    T = classes.shape[0]
    n_seq = 1 if seq_offsets is None else seq_offsets.shape[0] - 1
    rc = lib().difr_exfiltratable_bits(_ptr(classes), _ptr(counts), int(rank_cutoff), int(V), _ptr(seq_offsets), n_seq,
                                       T, _ptr(bits), _ptr(seq_bits), _stream(stream))
    if rc != DIFR_OK:
        raise DifrError(rc, "difr_exfiltratable_bits")
    return bits, seq_bits


def difr_expand_seeds(seeds, tokens, seq_offsets=None, prompt_hashes=None, expanded=None, stream=None):
    """Sequential randomness expansion: per-row seeds (int64 tensor holding the uint64 words) that also depend
    on the prompt hash of the row's sequence and on the claimed tokens before it.  `expanded` may be `seeds`."""
    T = seeds.shape[0]
    n_seq = 1 if seq_offsets is None else seq_offsets.shape[0] - 1
    if expanded is None:
        import torch
        expanded = torch.empty_like(seeds)
    rc = lib().difr_expand_seeds(_ptr(seeds), _ptr(tokens), _ptr(seq_offsets), n_seq, _ptr(prompt_hashes), T,
                                 _ptr(expanded), _stream(stream))
    if rc != DIFR_OK:
        raise DifrError(rc, "difr_expand_seeds")
    return expanded


def difr_score_gm_static(h, W, tokens, seeds, positions, temperature, out: DifrOut, stream=None) -> DifrOut:
    """difr_score_gm for callers that cannot allocate scratch memory: `out.workspace` is ignored (it may be
    None) and the library's built-in 16 MiB array is used instead.  Raises DifrError(DIFR_ERR_WORKSPACE) for
    problems that need more.  Calls on one device share that array, so do not let two of them overlap."""
    return _score("difr_score_gm_static", h, W, tokens, seeds, positions, temperature, out, stream)


def difr_detect(scores, threshold, margins=None, ranks=None, rank_cutoff=0, seq_offsets=None, flags=None,
                seq_stats=None, stream=None):
    """Threshold flags and per-sequence statistics; `seq_stats` is an int32 [n_seq, 4] tensor whose rows are
    (n_flagged, n_match, bits of float sum, bits of float min)."""
    T = scores.shape[0]
    n_seq = 1 if seq_offsets is None else seq_offsets.shape[0] - 1
    rc = lib().difr_detect(_ptr(scores), float(threshold), _ptr(margins), _ptr(ranks), int(rank_cutoff),
                           _ptr(seq_offsets), n_seq, T, _ptr(flags), _ptr(seq_stats), _stream(stream))
    if rc != DIFR_OK:
        raise DifrError(rc, "difr_detect")
    return flags, seq_stats


def difr_logits(h, W, logits, device_status=None, stream=None):
    T, d = h.shape
    V = W.shape[0]
    rc = lib().difr_logits(_ptr(h), _ptr(W), T, d, V, _ptr(logits), _ptr(device_status), _stream(stream))
    if rc != DIFR_OK:
        raise DifrError(rc, "difr_logits")
    return logits


def difr_selftest_wait(status2, limit_cycles, stream=None):
    """Runs the bounded-wait self-test; `status2` is an int32 [2] CUDA tensor."""
    rc = lib().difr_selftest_wait(_ptr(status2), int(limit_cycles), _stream(stream))
    if rc != DIFR_OK:
        raise DifrError(rc, "difr_selftest_wait")
    return status2


def difr_debug_plan_override(strips: int = 0, group: int = 0, l2_mb: int = 0) -> None:
    """Validation aid: fixes the planner's strip count / raster group / L2 share for later calls (0: its own)."""
    rc = lib().difr_debug_plan_override(int(strips), int(group), int(l2_mb))
    if rc != DIFR_OK:
        raise DifrError(rc, "difr_debug_plan_override")


def difr_philox(ctr, key, out, stream=None):
    rc = lib().difr_philox(_ptr(ctr), _ptr(key), ctr.shape[0], _ptr(out), _stream(stream))
    if rc != DIFR_OK:
        raise DifrError(rc, "difr_philox")
    return out
