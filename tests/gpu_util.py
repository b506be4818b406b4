"""Helpers shared by the GPU parity tests: move the seeded numpy inputs to the
device bit-for-bit and run the library through its binding."""
import numpy as np
import torch

import paper_2511_02620_b200 as difr

SEQ_STATS_DTYPE = np.dtype([("n_flagged", "<i4"), ("n_match", "<i4"), ("sum", "<f4"), ("min", "<f4")])


def to_bf16(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def to_dev(a: np.ndarray) -> torch.Tensor:
    a = np.ascontiguousarray(a)
    if a.dtype == np.uint64:
        a = a.view(np.int64)
    elif a.dtype == np.uint32:
        a = a.view(np.int32)
    return torch.from_numpy(a).cuda()


class Device:
    """h, W and the row metadata of one problem, resident on the GPU."""

    def __init__(self, h_bits, W_bits, seeds, positions):
        self.h = to_bf16(h_bits)
        self.W = to_bf16(W_bits)
        self.seeds = to_dev(seeds)
        self.positions = to_dev(positions)
        self.T, self.d = h_bits.shape
        self.V = W_bits.shape[0]

    def score(self, kind, tokens, temperature, sigma, eps=1e-12):
        out = difr.DifrOut.allocate(self.T, self.d, self.V, sigma, eps)
        # poison the outputs so that a row the kernels skip cannot pass by accident
        for name in ("score", "margin", "lse", "p_claimed", "cdf_lo", "u"):
            getattr(out, name).fill_(float("nan"))
        out.argmax.fill_(-7)
        out.runner_up.fill_(-7)
        fn = difr.difr_score_gm if kind == "gm" else difr.difr_score_ipt
        fn(self.h, self.W, to_dev(np.asarray(tokens, dtype=np.int32)), self.seeds, self.positions,
           float(np.float32(temperature)), out)
        torch.cuda.synchronize()
        assert int(out.device_status.item()) == 0, "device-side wait timed out"
        return {k: getattr(out, k).cpu().numpy() for k in
                ("score", "margin", "argmax", "runner_up", "lse", "p_claimed", "cdf_lo", "u", "row_status")}


def f32(x) -> float:
    """The double value of the float32 nearest to x (what the C ABI receives)."""
    return float(np.float32(x))
