#!/usr/bin/env python
"""Benchmark of the token-scoring path: verified tokens per second.

One step = one pass of the whole path over one synthetic batch: the fused
LM-head + Token-DiFR kernel, the split-V finalize kernel and the detection
kernel (`difr_score_gm` + `difr_detect`).  Prints one JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

With N > 1 (launched by torch.distributed.run, one rank per GPU) every rank
scores its own batch of the same shape with W replicated: rows are independent,
so there is no data-path collective (weak scaling).  `--impl reference` times
the fp64 CPU oracle instead, on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import ctypes
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import workloads as wl  # noqa: E402

METRIC = "verified_tokens_per_sec"
UNIT = "tokens/s"
L2_BYTES = 126 * 2**20
# dram__bytes_read.sum + dram__bytes_write.sum of the fused kernel per launch, from the
# ncu captures summarised under profiles/ (bytes; None until captured for that workload)
FUSED_TRAFFIC = {"llama3b": 962.3e6}  # profiles/k1_fused_score_llama3b.md


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"bf16_tflops": float(p["bf16_tflops"]), "bf16_tflops_sustained": float(p["bf16_tflops_sustained"]),
                "hbm_gbs": float(p["hbm_gbs"]), "source": "measured"}
    return {"bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "hbm_gbs": 6650.0, "source": "fallback"}


def pick_workload(args):
    w = wl.WORKLOADS[args.workload]
    if args.T:
        w = wl.with_T(w, args.T)
    return w


# ------------------------------------------------------------------ multi-rank
def rank_info():
    return int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))


def reduce_max(values, device=None):
    """Max over ranks of a list of floats (each rank times its own replica; the job is as slow as the slowest)."""
    import torch
    import torch.distributed as dist

    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.cpu()]


def whole_job_rate(world, rows_per_rank, steps, elapsed_ms):
    """Rows are sharded across ranks with no exchange: the job's rate is all ranks' rows over the slowest rank's time."""
    return world * rows_per_rank * steps / (elapsed_ms * 1e-3)


# --------------------------------------------------------------------- clocks
class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
               0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting"}

    def __init__(self, torch_device_index):
        super().__init__(daemon=True)
        self.samples, self.reason_bits, self.max_mhz, self.ok = [], 0, None, False
        self._stop_evt = threading.Event()
        try:
            import pynvml
            import torch

            pynvml.nvmlInit()
            self.nv = pynvml
            uuid = getattr(torch.cuda.get_device_properties(torch_device_index), "uuid", None)
            try:
                self.handle = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + str(uuid)).encode())
            except Exception:
                vis = os.environ.get("CUDA_VISIBLE_DEVICES", "")
                idx = int(vis.split(",")[torch_device_index]) if vis and vis.split(",")[0].isdigit() else torch_device_index
                self.handle = pynvml.nvmlDeviceGetHandleByIndex(idx)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.handle, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception as e:  # pragma: no cover
            self.err = repr(e)

    def run(self):
        if not self.ok:
            return
        while not self._stop_evt.is_set():
            try:
                self.samples.append(int(self.nv.nvmlDeviceGetClockInfo(self.handle, self.nv.NVML_CLOCK_SM)))
                self.reason_bits |= int(self.nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.handle))
            except Exception:
                pass
            time.sleep(0.02)

    def finish(self):
        self._stop_evt.set()
        if self.is_alive():
            self.join()
        if not self.ok or not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": ["unavailable"]}
        reasons = [name for bit, name in self.REASONS.items() if self.reason_bits & bit]
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz, "reasons": reasons,
                "samples": len(self.samples)}


# --------------------------------------------------------------- CPU baseline
def oracle_throughput(w, inp, tokens, temperature, sigma, budget_s, rows_override=None):
    """Times the oracle, as it stands, on a seeded subset of rows; returns (tokens/s, rows, seconds, cores)."""
    import oracle

    cores = oracle.num_threads()
    rows_all = wl.sample_rows(w, w.T, salt=7)
    one = rows_all[:1]
    t0 = time.perf_counter()
    oracle.score_gm(inp.h[one], inp.W, tokens[one], inp.seeds[one], inp.positions[one], temperature, sigma)
    t_row = time.perf_counter() - t0
    n = rows_override or int(max(cores, min(w.T, budget_s * cores / max(t_row, 1e-6))))
    n = max(1, min(n, w.T))
    rows = rows_all[:n]
    t0 = time.perf_counter()
    oracle.score_gm(np.ascontiguousarray(inp.h[rows]), inp.W, tokens[rows], inp.seeds[rows], inp.positions[rows],
                    temperature, sigma)
    dt = time.perf_counter() - t0
    return n / dt, n, dt, cores


def run_reference(args):
    if rank_info()[0] != 0:
        return  # under torchrun rank 0 alone times the oracle
    import oracle

    w = pick_workload(args)
    inp = wl.make_inputs(w)
    temperature = float(np.float32(args.temperature))
    sigma = float(np.float32(args.sigma))
    g = np.random.default_rng(12345)
    tokens = g.integers(0, w.V, size=w.T).astype(np.int32)  # the oracle's cost does not depend on the claims
    cores = oracle.num_threads()
    rows_all = wl.sample_rows(w, w.T, salt=11)
    t0 = time.perf_counter()
    r1 = rows_all[:1]
    oracle.score_gm(inp.h[r1], inp.W, tokens[r1], inp.seeds[r1], inp.positions[r1], temperature, sigma)
    t_row = time.perf_counter() - t0
    budget = 150.0 / max(1, args.steps + args.warmup)
    n = int(max(1, min(w.T, budget * cores / max(t_row, 1e-6))))

    def step(i):
        rows = np.sort(rows_all[(np.arange(n) + i * n) % w.T])
        r = oracle.score_gm(np.ascontiguousarray(inp.h[rows]), inp.W, tokens[rows], inp.seeds[rows],
                            inp.positions[rows], temperature, sigma)
        oracle.detect(r.score, -4.6, r.margin, None)

    for i in range(args.warmup):
        step(i)
    t0 = time.perf_counter()
    for i in range(args.steps):
        step(args.warmup + i)
    dt = time.perf_counter() - t0
    value = n * args.steps / dt
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_dict(w, args),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": f"{n} seeded rows of {w.T} per step"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def config_dict(w, args):
    in_bytes = 2 * (w.T * w.d + w.V * w.d)
    return {"workload": w.name, "T": w.T, "d": w.d, "V": w.V, "seq_len": w.seq_len, "estimator": "token_difr_gumbel_max",
            "temperature": args.temperature, "sigma": args.sigma, "eps": 1e-12, "tamper_frac": w.tamper_frac,
            "generator_seeds": {name: wl.stream_seed(w, k) for k, name in
                                enumerate(("h", "W", "tamper", "seeds", "perturbation"), start=1)},
            "l2": ("inputs larger than L2 (h + W = %.0f MB)" % (in_bytes / 1e6)) if in_bytes > 2 * L2_BYTES
            else "L2 flushed between steps (256 MB write), per-step events"}


# ------------------------------------------------------------------- GPU arm
def run_ours(args):
    import torch
    import torch.distributed as dist

    import paper_2511_02620_b200 as difr

    rank, local_rank, world = rank_info()
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    difr.lib()  # fail loudly if the CUDA library is missing

    w = pick_workload(args)
    temperature = float(np.float32(args.temperature))
    sigma = float(np.float32(args.sigma))
    inp = wl.make_inputs(w)
    T, d, V = w.T, w.d, w.V

    def pinned(a):
        a = np.ascontiguousarray(a)
        if a.dtype == np.uint64:
            a = a.view(np.int64)
        elif a.dtype == np.uint32:
            a = a.view(np.int32)
        elif a.dtype == np.uint16:
            a = a.view(np.int16)
        return torch.from_numpy(a).pin_memory()

    h_host = pinned(inp.h)
    seeds_host, pos_host = pinned(inp.seeds), pinned(inp.positions)
    W_dev = pinned(inp.W).cuda().view(torch.bfloat16)
    h_dev = h_host.cuda().view(torch.bfloat16)
    seeds_dev, pos_dev = seeds_host.cuda(), pos_host.cuda()
    seq_dev = torch.from_numpy(inp.seq_offsets).cuda()
    n_seq = inp.seq_offsets.shape[0] - 1

    out = difr.DifrOut.allocate(T, d, V, sigma, 1e-12)
    flags = torch.empty(T, dtype=torch.uint8, device="cuda")
    stats = torch.empty((n_seq, 4), dtype=torch.int32, device="cuda")

    # Claims: the inference server's Gumbel-max sample on its own (perturbed) hidden states,
    # produced here by the library itself (untimed set-up; throughput does not depend on them),
    # then tampered as the workload prescribes.
    hs_dev = pinned(inp.h_server).cuda().view(torch.bfloat16)
    zeros = torch.zeros(T, dtype=torch.int32, device="cuda")
    difr.difr_score_gm(hs_dev, W_dev, zeros, seeds_dev, pos_dev, temperature, out)
    honest = out.argmax.clone()
    difr.difr_score_gm(hs_dev, W_dev, honest, seeds_dev, pos_dev, temperature, out)
    runner = out.runner_up.clone()
    torch.cuda.synchronize()
    del hs_dev
    tokens_np, tampered = wl.tamper(w, honest.cpu().numpy(), runner.cpu().numpy())
    tokens_host = torch.from_numpy(tokens_np).pin_memory()
    tokens_dev = tokens_host.cuda()
    tau = float(np.log(1e-3))

    cudart = ctypes.CDLL("libcudart.so.12")
    n_ev = args.steps

    def make_events(n):
        evs = []
        for _ in range(n):
            e = ctypes.c_void_p()
            assert cudart.cudaEventCreate(ctypes.byref(e)) == 0
            evs.append(e)
        return evs

    ev_a, ev_b = make_events(n_ev), make_events(n_ev)
    small = 2 * (T * d + V * d) <= 2 * L2_BYTES
    flush = torch.empty(256 * 2**20, dtype=torch.uint8, device="cuda") if small else None

    def step(i=None):
        if i is not None:
            out.event_fused_start, out.event_fused_stop = ev_a[i].value, ev_b[i].value
        else:
            out.event_fused_start = out.event_fused_stop = 0
        difr.difr_score_gm(h_dev, W_dev, tokens_dev, seeds_dev, pos_dev, temperature, out)
        difr.difr_detect(out.score, tau, out.margin, None, 0, seq_dev, flags, stats)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    barrier()
    sampler = ClockSampler(local_rank)
    sampler.start()
    t_begin, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    step_ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    t_begin.record()
    for i in range(args.steps):
        if flush is not None:
            flush.zero_()
        step_ev[i][0].record()
        step(i)
        step_ev[i][1].record()
    t_end.record()
    barrier()
    clocks = sampler.finish()
    if flush is not None:
        elapsed_ms = sum(a.elapsed_time(b) for a, b in step_ev)
    else:
        elapsed_ms = t_begin.elapsed_time(t_end)
    fused_ms = []
    for a, b in zip(ev_a, ev_b):
        ms = ctypes.c_float()
        assert cudart.cudaEventElapsedTime(ctypes.byref(ms), a, b) == 0
        fused_ms.append(ms.value)
    fused_avg_ms = float(np.mean(fused_ms))
    assert int(out.device_status.item()) == 0, "device-side wait timed out"
    n_flagged = int(flags.sum().item())
    flags_ref = flags.cpu().clone()
    stats_np = stats.cpu().numpy()

    # ---- end to end: per-step inputs start in pinned host memory, results end there
    out.event_fused_start = out.event_fused_stop = 0
    # Two input buffers and two sets of outputs: a copy stream uploads step i + 1 while the kernels of step i
    # run, and a third stream reads the results of step i back while the kernels of step i + 1 run (what a
    # serving loop does); every step's upload, kernels and read-back lie inside the timed region.
    copy_stream, back_stream, run_stream = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.current_stream()
    bufs = [(torch.empty_like(h_dev), torch.empty_like(tokens_dev), torch.empty_like(seeds_dev),
             torch.empty_like(pos_dev)) for _ in range(2)]
    outs = [out, difr.DifrOut.allocate(T, d, V, sigma, 1e-12)]
    dev_res = [(flags, stats), (torch.empty_like(flags), torch.empty_like(stats))]
    host_res = [(torch.empty(T, dtype=torch.float32).pin_memory(), torch.empty(T, dtype=torch.uint8).pin_memory(),
                 torch.empty((n_seq, 4), dtype=torch.int32).pin_memory()) for _ in range(2)]
    uploaded = [torch.cuda.Event() for _ in range(2)]
    consumed = [torch.cuda.Event() for _ in range(2)]
    scored = [torch.cuda.Event() for _ in range(2)]
    read_back = [torch.cuda.Event() for _ in range(2)]

    def upload(i):
        h_in, tok_in, seed_in, pos_in = bufs[i % 2]
        with torch.cuda.stream(copy_stream):
            copy_stream.wait_event(consumed[i % 2])  # the kernels that last read this buffer are done
            h_in.view(torch.int16).copy_(h_host, non_blocking=True)
            tok_in.copy_(tokens_host, non_blocking=True)
            seed_in.copy_(seeds_host, non_blocking=True)
            pos_in.copy_(pos_host, non_blocking=True)
            uploaded[i % 2].record(copy_stream)

    def run(i):
        h_in, tok_in, seed_in, pos_in = bufs[i % 2]
        o, (fl, st) = outs[i % 2], dev_res[i % 2]
        score_host, flags_host, stats_host = host_res[i % 2]
        run_stream.wait_event(uploaded[i % 2])
        run_stream.wait_event(read_back[i % 2])  # the results these outputs held two steps ago have been read
        difr.difr_score_gm(h_in, W_dev, tok_in, seed_in, pos_in, temperature, o)
        difr.difr_detect(o.score, tau, o.margin, None, 0, seq_dev, fl, st)
        consumed[i % 2].record(run_stream)
        scored[i % 2].record(run_stream)
        with torch.cuda.stream(back_stream):
            back_stream.wait_event(scored[i % 2])
            score_host.copy_(o.score, non_blocking=True)
            flags_host.copy_(fl, non_blocking=True)
            stats_host.copy_(st, non_blocking=True)
            read_back[i % 2].record(back_stream)

    def e2e_loop(n):
        upload(0)
        for i in range(n):
            if i + 1 < n:
                upload(i + 1)
            run(i)
        run_stream.wait_stream(back_stream)  # the last read-backs end inside the timed region

    for ev in consumed + read_back:
        ev.record(run_stream)
    e2e_loop(min(args.warmup, 3))
    barrier()
    e_begin, e_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for ev in consumed + read_back:
        ev.record(run_stream)
    e_begin.record(run_stream)
    copy_stream.wait_event(e_begin)  # the first upload starts inside the timed region
    e2e_loop(args.steps)
    e_end.record(run_stream)
    barrier()
    e2e_ms = e_begin.elapsed_time(e_end)
    assert int(outs[1].device_status.item()) == 0, "device-side wait timed out"
    last = (args.steps - 1) % 2
    score_host, flags_host, stats_host = host_res[last]
    h2d = h_host.numel() * 2 + tokens_host.numel() * 4 + seeds_host.numel() * 8 + pos_host.numel() * 4
    d2h = score_host.numel() * 4 + flags_host.numel() + stats_host.numel() * 4
    assert torch.equal(flags_host, dev_res[last][0].cpu())
    assert torch.equal(flags_host, flags_ref)

    elapsed_ms, e2e_ms, fused_avg_ms = reduce_max([elapsed_ms, e2e_ms, fused_avg_ms], device="cuda")

    # ---- the other estimator on the same resident inputs (context; the headline is Token-DiFR)
    ipt_ms = None
    if world == 1 and temperature > 0:
        n_ipt = max(1, min(args.steps, 10))
        for _ in range(2):
            difr.difr_score_ipt(h_dev, W_dev, tokens_dev, seeds_dev, pos_dev, temperature, out)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record()
        for _ in range(n_ipt):
            difr.difr_score_ipt(h_dev, W_dev, tokens_dev, seeds_dev, pos_dev, temperature, out)
            difr.difr_detect(out.score, tau, None, None, 0, seq_dev, flags, stats)
        b.record()
        torch.cuda.synchronize()
        ipt_ms = a.elapsed_time(b) / n_ipt
        assert int(out.device_status.item()) == 0, "device-side wait timed out"

    if rank == 0:
        peaks = load_peaks()
        flop = 2.0 * T * d * V
        achieved = flop / (fused_avg_ms * 1e-3) / 1e12
        value = whole_job_rate(world, T, args.steps, elapsed_ms)
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": elapsed_ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": config_dict(w, args),
            "tflops": world * flop * args.steps / (elapsed_ms * 1e-3) / 1e12,
            "clocks": clocks,
            "e2e": {"value": whole_job_rate(world, T, args.steps, e2e_ms), "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms / args.steps,
                    "note": "per-step inputs (h, tokens, seeds, positions) from pinned host memory, uploaded on a copy "
                            "stream one step ahead of the kernels; scores, flags and statistics read back on a "
                            "third stream; W resident"},
            "gpu_launches": 3 * args.steps,
            "roofline": {"kernel": "k1_fused_score", "bound": "tensor", "achieved": achieved,
                         "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": achieved / peaks["bf16_tflops"],
                         "peak_kind": "burst bf16 dense, " + peaks["source"],
                         "frac_of_sustained": achieved / peaks["bf16_tflops_sustained"],
                         "ms_per_launch": fused_avg_ms, "flop_per_launch": flop,
                         "traffic": FUSED_TRAFFIC.get(w.name)},
            "detect": {"threshold": tau, "n_flagged": n_flagged, "n_tampered": int(tampered.sum()),
                       "n_match": int(stats_np[:, 1].sum())},
        }
        if ipt_ms is not None:
            line["token_ipt_difr"] = {"value": T / (ipt_ms * 1e-3), "unit": UNIT, "ms_per_step": ipt_ms,
                                      "tflops": flop / (ipt_ms * 1e-3) / 1e12,
                                      "note": "difr_score_ipt + difr_detect, resident inputs, sigma in CDF units"}
        if args.variants:
            line["variants_ms"] = time_variants(difr, h_dev, W_dev, tokens_dev, seeds_dev, pos_dev, temperature, sigma,
                                                T, d, V)
        if world == 1 and not args.no_cpu_baseline:
            val, n, dt, cores = oracle_throughput(w, inp, tokens_np, temperature, sigma, args.cpu_seconds)
            line["cpu_baseline"] = {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle",
                                    "sample": f"{n} seeded rows of {T}, {dt:.1f} s"}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def time_variants(difr, h, W, tokens, seeds, pos, temperature, sigma, T, d, V, iters=3):
    """Milliseconds per call of the other entry points on the same resident inputs (context for the headline)."""
    import torch

    out = difr.DifrOut.allocate(T, d, V, sigma, 1e-12)
    out.workspace = torch.empty(difr.difr_filtered_workspace_bytes(T, d, V), dtype=torch.uint8, device="cuda")
    f = lambda: torch.empty(T, dtype=torch.float32, device="cuda")
    out.y_max, out.y_second, out.score_ipt, out.sigma_ipt, out.cutoff = f(), f(), f(), 0.05, f()
    rank = torch.empty(T, dtype=torch.int32, device="cuda")
    counts = torch.empty((4, T), dtype=torch.int32, device="cuda")

    def gm_rank():
        out.rank = rank
        difr.difr_score_gm(h, W, tokens, seeds, pos, temperature, out)
        out.rank = None

    calls = {
        "score_gm": lambda: difr.difr_score_gm(h, W, tokens, seeds, pos, temperature, out),
        "score_gm_with_rank": gm_rank,
        "score_ipt": lambda: difr.difr_score_ipt(h, W, tokens, seeds, pos, temperature, out),
        "score_both": lambda: difr.difr_score_both(h, W, tokens, seeds, pos, temperature, out),
        "admissible_4_thresholds": lambda: difr.difr_admissible(h, W, seeds, pos, temperature, out,
                                                                [-1.0, -3.0, -6.0, -9.0], counts),
        "score_gm_filtered_k50_p095_s4": lambda: difr.difr_score_gm_filtered(h, W, tokens, seeds, pos, temperature,
                                                                             50, 0.95, 4, out),
        "score_ipt_filtered_k50_p095": lambda: difr.difr_score_ipt_filtered(h, W, tokens, seeds, pos, temperature,
                                                                           50, 0.95, out),
    }
    res = {}
    calls["score_gm"]()
    for name, fn in calls.items():
        fn()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(iters):
            fn()
        b.record()
        torch.cuda.synchronize()
        res[name] = a.elapsed_time(b) / iters
    assert int(out.device_status.item()) == 0
    return res


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama3b", choices=sorted(wl.WORKLOADS))
    ap.add_argument("--T", type=int, default=0, help="override the number of rows (whole sequences)")
    ap.add_argument("--temperature", type=float, default=None,
                    help="sampling temperature (default: the workload's own, its last listed one)")
    ap.add_argument("--sigma", type=float, default=0.05)
    ap.add_argument("--cpu-seconds", type=float, default=15.0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--variants", action="store_true", help="also time the other entry points (extra JSON key)")
    args = ap.parse_args()
    if args.temperature is None:
        args.temperature = float(wl.WORKLOADS[args.workload].temperatures[-1])
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
