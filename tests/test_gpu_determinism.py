"""Repeated launches on fixed inputs must give bit-identical outputs: the fused kernel hands its work units out on
demand, so which CTA pair computes which unit changes from launch to launch, and candidate lists fill in a
different order every time; none of it may show in the results.  (A race in the pipeline or the scheduler would
show here as a word that differs once in many launches.)"""
import numpy as np
import pytest
import torch

import paper_2511_02620_b200 as difr

pytestmark = pytest.mark.gpu


def _problem(T, d, V, seed):
    g = torch.Generator(device="cuda").manual_seed(seed)
    h = torch.randn(T, d, device="cuda", generator=g).to(torch.bfloat16)
    W = (2.0 * torch.randn(V, d, device="cuda", generator=g) / d**0.5).to(torch.bfloat16)
    tokens = torch.randint(0, V, (T,), device="cuda", dtype=torch.int32, generator=g)
    seeds = torch.randint(0, 2**62, (T,), device="cuda", dtype=torch.int64, generator=g)
    pos = (torch.arange(T, device="cuda", dtype=torch.int32) % 512) + 1
    return h, W, tokens, seeds, pos


@pytest.mark.parametrize("kind,T,d,V,iters", [
    ("gm", 4096, 3072, 128256, 300),     # the benchmark's workload: ten rounds of units on every pair
    ("ipt", 4096, 3072, 128256, 200),
    ("gm", 1000, 520, 50001, 1500),      # ragged everywhere, fewer units than pairs
    ("gm_filtered", 2048, 1024, 128256, 100),
    ("ipt_filtered", 2048, 1024, 128256, 100),
])
def test_repeated_launches_are_bit_identical(kind, T, d, V, iters):
    h, W, tokens, seeds, pos = _problem(T, d, V, 3)
    out = difr.DifrOut.allocate(T, d, V, 0.05)
    out.workspace = torch.empty(difr.difr_filtered_workspace_bytes(T, d, V), dtype=torch.uint8, device="cuda")
    out.cutoff = torch.empty(T, dtype=torch.float32, device="cuda")
    call, names = {
        "gm": (lambda: difr.difr_score_gm(h, W, tokens, seeds, pos, 1.0, out),
               ("score", "margin", "argmax", "runner_up", "lse", "row_status")),
        "ipt": (lambda: difr.difr_score_ipt(h, W, tokens, seeds, pos, 1.0, out),
                ("score", "p_claimed", "cdf_lo", "u", "lse", "row_status")),
        "gm_filtered": (lambda: difr.difr_score_gm_filtered(h, W, tokens, seeds, pos, 1.0, 50, 0.95, 4, out),
                        ("score", "cutoff", "margin", "argmax", "row_status")),
        "ipt_filtered": (lambda: difr.difr_score_ipt_filtered(h, W, tokens, seeds, pos, 1.0, 50, 0.95, out),
                         ("score", "cutoff", "p_claimed", "cdf_lo", "row_status")),
    }[kind]
    call()
    torch.cuda.synchronize()
    ref = [getattr(out, n).clone() for n in names]
    differing = torch.zeros(1, dtype=torch.int64, device="cuda")
    for _ in range(iters):
        call()
        for n, r in zip(names, ref):
            differing += (getattr(out, n).view(torch.int32) != r.view(torch.int32)).sum()
    torch.cuda.synchronize()
    assert int(out.device_status.item()) == 0
    assert int(differing.item()) == 0
    assert np.isfinite(ref[0].cpu().numpy()).all()
