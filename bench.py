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


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"bf16_tflops": float(p["bf16_tflops"]), "bf16_tflops_sustained": float(p["bf16_tflops_sustained"]),
                "hbm_gbs": float(p["hbm_gbs"]), "source": "measured"}
    return {"bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "hbm_gbs": 6650.0, "source": "fallback"}


def pick_workload(args):
    """The benchmark's workload: by default the long stream at the largest T of its sweep."""
    w = wl.WORKLOADS[args.workload]
    T = args.T or (max(w.sweep_T) if w.sweep_T else 0)
    if T:
        w = wl.with_T(w, T)
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
def kernel_source_digest():
    """Digest of the fused kernel's sources: DRAM traffic captured under ncu is only quoted while they are unchanged."""
    import hashlib

    hsh = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_2511_02620_b200", "csrc")
    for name in ("k1_fused_score.cu", "difr_device.cuh", "difr_plan.h"):
        with open(os.path.join(csrc, name), "rb") as f:
            hsh.update(f.read())
    # of the shared header only the fused kernel's own parameter block
    with open(os.path.join(csrc, "difr_kernels.h"), "rb") as f:
        text = f.read()
    start = text.index(b"struct K1Params")
    hsh.update(text[start:text.index(b"};", start)])
    return hsh.hexdigest()[:16]


def captured_traffic(w):
    """dram__bytes_read.sum + dram__bytes_write.sum of one fused-kernel launch on this workload, from the ncu
    capture recorded in profiles/k1_fused_score_traffic.txt; None when there is no capture for the workload or
    the kernel's sources have changed since it was taken.  A capture taken at fewer rows is scaled by the rows
    (W is streamed once per group of rows, so traffic grows in proportion)."""
    path = os.path.join(ROOT, "profiles", "k1_fused_score_traffic.txt")
    if not os.path.exists(path):
        return None, "no capture"
    with open(path) as f:
        rec = json.load(f)
    if rec.get("kernel_source_digest") != kernel_source_digest():
        return None, "kernel sources changed since the capture in " + os.path.basename(path)
    for c in rec.get("captures", []):
        if c["workload"] == w.name and c["d"] == w.d and c["V"] == w.V and w.T % c["T"] == 0:
            return float(c["dram_bytes_per_launch"]) * (w.T // c["T"]), c["profile"]
    return None, "no capture for this workload"


class CudaEvents:
    """cudaEvent_t handles made through the runtime library itself, so that the library under test can be handed
    raw handles (torch's events cannot be recorded from C)."""

    def __init__(self):
        self.rt = ctypes.CDLL("libcudart.so.12")
        self.rt.cudaEventRecord.argtypes = [ctypes.c_void_p, ctypes.c_void_p]

    def make(self, n):
        evs = []
        for _ in range(n):
            e = ctypes.c_void_p()
            assert self.rt.cudaEventCreate(ctypes.byref(e)) == 0
            evs.append(e)
        return evs

    def record(self, e, stream):
        assert self.rt.cudaEventRecord(e, ctypes.c_void_p(stream)) == 0

    def ms(self, a, b):
        out = ctypes.c_float()
        assert self.rt.cudaEventElapsedTime(ctypes.byref(out), a, b) == 0
        return float(out.value)

    def free(self, evs):
        for e in evs:
            self.rt.cudaEventDestroy(e)


class Problem:
    """One workload resident on the device: inputs, claims, outputs."""

    def __init__(self, difr, w, temperature, sigma, inp=None, share=None):
        import torch

        self.difr, self.w, self.temperature, self.sigma = difr, w, temperature, sigma
        T, d, V = w.T, w.d, w.V
        if share is not None:
            # a shorter long stream: the first T rows of the resident one (the generators are prefix-stable)
            self.h_host = share.h_host[: T]
            self.W, self.h = share.W, share.h[: T]
            self.seeds_host, self.pos_host = share.seeds_host[: T], share.pos_host[: T]
            self.seeds, self.pos = share.seeds[: T], share.pos[: T]
            seq_offsets = share.seq_offsets_np[: T // w.seq_len + 1]
            hs = None
        else:
            self.h_host = pinned(inp.h)
            self.seeds_host, self.pos_host = pinned(inp.seeds), pinned(inp.positions)
            self.W = pinned(inp.W).cuda().view(torch.bfloat16)
            self.h = self.h_host.cuda().view(torch.bfloat16)
            self.seeds, self.pos = self.seeds_host.cuda(), self.pos_host.cuda()
            seq_offsets = inp.seq_offsets
            hs = None if inp.h_server is inp.h else pinned(inp.h_server).cuda().view(torch.bfloat16)
        self.seq_offsets_np = seq_offsets
        self.seq = torch.from_numpy(np.ascontiguousarray(seq_offsets)).cuda()
        self.n_seq = len(seq_offsets) - 1
        self.out = difr.DifrOut.allocate(T, d, V, sigma, 1e-12)
        self.flags = torch.empty(T, dtype=torch.uint8, device="cuda")
        self.stats = torch.empty((self.n_seq, 4), dtype=torch.int32, device="cuda")
        # Claims: the inference server's Gumbel-max sample on its own (perturbed) hidden states, produced by the
        # library itself in untimed set-up (throughput does not depend on them; the oracle would need hours at
        # these sizes), then tampered as the workload prescribes.
        src = self.h if hs is None else hs
        zeros = torch.zeros(T, dtype=torch.int32, device="cuda")
        difr.difr_score_gm(src, self.W, zeros, self.seeds, self.pos, temperature, self.out)
        honest, runner = self.out.argmax.clone(), self.out.runner_up.clone()
        torch.cuda.synchronize()
        del hs, src
        self.tokens_np, self.tampered = wl.tamper(w, honest.cpu().numpy(), runner.cpu().numpy())
        self.tokens_host = torch.from_numpy(self.tokens_np).pin_memory()
        self.tokens = self.tokens_host.cuda()
        # Detection threshold: calibrated on this batch's untampered rows for 1 % false positives
        # (Sec. "Classification via Thresholding"), from the library's own scores, in untimed set-up.
        difr.difr_score_gm(self.h, self.W, self.tokens, self.seeds, self.pos, temperature, self.out)
        benign = self.out.score[torch.from_numpy(~self.tampered).cuda()]
        k = int(0.01 * benign.numel())
        self.tau = float(torch.kthvalue(benign, k + 1).values.item())
        torch.cuda.synchronize()

    def step(self, ev=None, events=None, stream=0):
        """One pass of the whole path; `ev` = four raw events to record around the three kernels."""
        o, difr = self.out, self.difr
        if ev is not None:
            o.event_fused_start, o.event_fused_stop = ev[0].value, ev[1].value
        else:
            o.event_fused_start = o.event_fused_stop = 0
        difr.difr_score_gm(self.h, self.W, self.tokens, self.seeds, self.pos, self.temperature, o)
        if ev is not None:
            events.record(ev[2], stream)
        difr.difr_detect(o.score, self.tau, o.margin, None, 0, self.seq, self.flags, self.stats)
        if ev is not None:
            events.record(ev[3], stream)

    def detect_us_back_to_back(self, n=200):
        """Microseconds per difr_detect call when many are enqueued back to back (two events around all of them):
        what the kernel costs a stream that is kept busy, without the event records between single launches."""
        import torch

        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        o = self.out
        for _ in range(10):
            self.difr.difr_detect(o.score, self.tau, o.margin, None, 0, self.seq, self.flags, self.stats)
        torch.cuda.synchronize()
        a.record()
        for _ in range(n):
            self.difr.difr_detect(o.score, self.tau, o.margin, None, 0, self.seq, self.flags, self.stats)
        b.record()
        torch.cuda.synchronize()
        return 1e3 * a.elapsed_time(b) / n

    def host_us_per_call(self, n=8):
        """Host time of one difr_score_gm call through the raw C ABI (arguments marshalled beforehand)."""
        import torch

        lib = self.difr.lib()
        self.out.event_fused_start = self.out.event_fused_stop = 0
        c = self.out._c()
        args = (ctypes.c_void_p(self.h.data_ptr()), ctypes.c_void_p(self.W.data_ptr()),
                ctypes.c_void_p(self.tokens.data_ptr()), ctypes.c_void_p(self.seeds.data_ptr()),
                ctypes.c_void_p(self.pos.data_ptr()), ctypes.c_float(self.temperature), self.w.T, self.w.d, self.w.V,
                ctypes.byref(c), ctypes.c_void_p(torch.cuda.current_stream().cuda_stream))
        times = []
        for _ in range(n):
            t0 = time.perf_counter_ns()
            rc = lib.difr_score_gm(*args)
            times.append((time.perf_counter_ns() - t0) * 1e-3)
            assert rc == 0
        torch.cuda.synchronize()
        return float(np.median(times))


def pinned(a):
    import torch

    a = np.ascontiguousarray(a)
    view = {np.dtype(np.uint64): np.int64, np.dtype(np.uint32): np.int32, np.dtype(np.uint16): np.int16}
    return torch.from_numpy(a.view(view.get(a.dtype, a.dtype))).pin_memory()


def timed_steps(prob, steps, warmup, events, local_rank, barrier, flush=None):
    """W warm-up steps, then exactly `steps` timed ones.  Returns whole-region ms, per-kernel mean ms, clocks."""
    import torch

    for _ in range(warmup):
        prob.step()
    barrier()
    stream = torch.cuda.current_stream().cuda_stream
    evs = [events.make(4) for _ in range(steps)]
    sampler = ClockSampler(local_rank)
    sampler.start()
    t_begin, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    per_step = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    t_begin.record()
    for i in range(steps):
        if flush is not None:
            flush.zero_()
        per_step[i][0].record()
        prob.step(evs[i], events, stream)
        per_step[i][1].record()
    t_end.record()
    barrier()
    clocks = sampler.finish()
    elapsed = sum(a.elapsed_time(b) for a, b in per_step) if flush is not None else t_begin.elapsed_time(t_end)
    k1 = float(np.mean([events.ms(e[0], e[1]) for e in evs]))
    k2 = float(np.mean([events.ms(e[1], e[2]) for e in evs]))
    k3 = float(np.mean([events.ms(e[2], e[3]) for e in evs]))
    for e in evs:
        events.free(e)
    assert int(prob.out.device_status.item()) == 0, "device-side wait timed out"
    return elapsed, (k1, k2, k3), clocks


def strips_of(difr, w):
    """Partial records per row, recovered from the workspace size (records, a 256-byte tail, 540 bytes per row of
    bounds and lists for the integer outputs)."""
    T_pad = -(-w.T // 256) * 256
    return (difr.difr_workspace_bytes(w.T, w.d, w.V) - 256 - 540 * T_pad) // (32 * T_pad)


def roofline_of(difr, w, k1_ms, k2_ms, k3_ms, peaks, n_seq):
    """Roofline figures of the three kernels from their device times and their algorithmic flop / bytes."""
    flop = 2.0 * w.T * w.d * w.V
    achieved = flop / (k1_ms * 1e-3) / 1e12
    traffic, traffic_src = captured_traffic(w)
    S = strips_of(difr, w)
    # finalize: the row's records are read twice (32 B, then the 16 B of candidates), the row of h and three rows
    # of W once, 16 B of row metadata, 36 B of outputs
    k2_bytes = w.T * (48.0 * S + 8.0 * w.d + 16 + 36)
    # detect: score and margin read, one flag byte written, 16 B of statistics per sequence
    k3_bytes = w.T * 9.0 + 16.0 * n_seq
    return {
        "kernel": "k1_fused_score", "bound": "tensor", "achieved": achieved, "peak": peaks["bf16_tflops"],
        "unit": "TFLOP/s", "frac": achieved / peaks["bf16_tflops"],
        "peak_kind": "burst bf16 dense, " + peaks["source"],
        "frac_of_sustained": achieved / peaks["bf16_tflops_sustained"],
        "ms_per_launch": k1_ms, "flop_per_launch": flop, "traffic": traffic, "traffic_source": traffic_src,
        "other_kernels": {
            "k2_finalize": {"bound": "hbm", "ms_per_launch": k2_ms, "bytes_per_launch": k2_bytes,
                            "achieved": k2_bytes / (k2_ms * 1e-3) / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                            "frac": k2_bytes / (k2_ms * 1e-3) / 1e9 / peaks["hbm_gbs"]},
            "k3_detect": {"bound": "hbm", "ms_per_launch": k3_ms, "bytes_per_launch": k3_bytes,
                          "achieved": k3_bytes / (k3_ms * 1e-3) / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                          "frac": k3_bytes / (k3_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                          "note": "includes the gap between two event records (a few microseconds)"},
        },
    }


def e2e_rate(prob, steps, warmup, barrier):
    """The same step with the per-step inputs starting in pinned host memory and the results ending there.
    Two input buffers and two sets of outputs: a copy stream uploads step i + 1 while the kernels of step i run,
    and a third stream reads the results of step i back while the kernels of step i + 1 run (what a serving
    loop does); every step's upload, kernels and read-back lie inside the timed region.  W stays resident."""
    import torch

    difr, w = prob.difr, prob.w
    T, d, V = w.T, w.d, w.V
    prob.out.event_fused_start = prob.out.event_fused_stop = 0
    copy_stream, back_stream, run_stream = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.current_stream()
    bufs = [(torch.empty_like(prob.h), torch.empty_like(prob.tokens), torch.empty_like(prob.seeds),
             torch.empty_like(prob.pos)) for _ in range(2)]
    outs = [prob.out, difr.DifrOut.allocate(T, d, V, prob.sigma, 1e-12)]
    dev_res = [(prob.flags, prob.stats), (torch.empty_like(prob.flags), torch.empty_like(prob.stats))]
    host_res = [(torch.empty(T, dtype=torch.float32).pin_memory(), torch.empty(T, dtype=torch.uint8).pin_memory(),
                 torch.empty((prob.n_seq, 4), dtype=torch.int32).pin_memory()) for _ in range(2)]
    uploaded = [torch.cuda.Event() for _ in range(2)]
    consumed = [torch.cuda.Event() for _ in range(2)]
    scored = [torch.cuda.Event() for _ in range(2)]
    read_back = [torch.cuda.Event() for _ in range(2)]

    def upload(i):
        h_in, tok_in, seed_in, pos_in = bufs[i % 2]
        with torch.cuda.stream(copy_stream):
            copy_stream.wait_event(consumed[i % 2])  # the kernels that last read this buffer are done
            h_in.view(torch.int16).copy_(prob.h_host, non_blocking=True)
            tok_in.copy_(prob.tokens_host, non_blocking=True)
            seed_in.copy_(prob.seeds_host, non_blocking=True)
            pos_in.copy_(prob.pos_host, non_blocking=True)
            uploaded[i % 2].record(copy_stream)

    def run(i):
        h_in, tok_in, seed_in, pos_in = bufs[i % 2]
        o, (fl, st) = outs[i % 2], dev_res[i % 2]
        score_host, flags_host, stats_host = host_res[i % 2]
        run_stream.wait_event(uploaded[i % 2])
        run_stream.wait_event(read_back[i % 2])  # the results these outputs held two steps ago have been read
        difr.difr_score_gm(h_in, prob.W, tok_in, seed_in, pos_in, prob.temperature, o)
        difr.difr_detect(o.score, prob.tau, o.margin, None, 0, prob.seq, fl, st)
        consumed[i % 2].record(run_stream)
        scored[i % 2].record(run_stream)
        with torch.cuda.stream(back_stream):
            back_stream.wait_event(scored[i % 2])
            score_host.copy_(o.score, non_blocking=True)
            flags_host.copy_(fl, non_blocking=True)
            stats_host.copy_(st, non_blocking=True)
            read_back[i % 2].record(back_stream)

    def loop(n):
        upload(0)
        for i in range(n):
            if i + 1 < n:
                upload(i + 1)
            run(i)
        run_stream.wait_stream(back_stream)  # the last read-backs end inside the timed region

    for ev in consumed + read_back:
        ev.record(run_stream)
    loop(min(warmup, 3))
    barrier()
    e_begin, e_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for ev in consumed + read_back:
        ev.record(run_stream)
    e_begin.record(run_stream)
    copy_stream.wait_event(e_begin)  # the first upload starts inside the timed region
    loop(steps)
    e_end.record(run_stream)
    barrier()
    ms = e_begin.elapsed_time(e_end)
    assert int(outs[1].device_status.item()) == 0, "device-side wait timed out"
    last = (steps - 1) % 2
    score_host, flags_host, stats_host = host_res[last]
    h2d = prob.h_host.numel() * 2 + prob.tokens_host.numel() * 4 + prob.seeds_host.numel() * 8 + prob.pos_host.numel() * 4
    d2h = score_host.numel() * 4 + flags_host.numel() + stats_host.numel() * 4
    assert torch.equal(flags_host, dev_res[last][0].cpu())
    return ms, h2d, d2h, flags_host.clone()


def per_config_entry(difr, w, temperature, sigma, events, local_rank, barrier, peaks, inp=None, share=None):
    """One entry of the `per_config` list: the same step on another target configuration, repeated until the timed
    region is at least a second long (so that the clock record has >= 20 samples and the power cap has settled)."""
    prob = Problem(difr, w, temperature, sigma, inp=inp, share=share)
    small = 2 * (w.T * w.d + w.V * w.d) <= 2 * L2_BYTES
    assert not small, "per_config workloads are larger than L2"
    import torch

    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    prob.step()
    b.record()
    barrier()
    est_ms = max(a.elapsed_time(b), 1e-3)
    steps = int(min(2000, max(3, np.ceil(1100.0 / est_ms))))
    elapsed, (k1, k2, k3), clocks = timed_steps(prob, steps, 3, events, local_rank, barrier)
    host_us = prob.host_us_per_call()
    k3_us = prob.detect_us_back_to_back()
    roof = roofline_of(difr, w, k1, k2, k3, peaks, prob.n_seq)
    mhz = clocks.get("sm_mhz")
    entry = {
        "workload": w.name, "T": w.T, "d": w.d, "V": w.V, "temperature": temperature, "sigma": sigma,
        "steps": steps, "timed_region_s": elapsed * 1e-3, "ms_per_step": elapsed / steps,
        "value": w.T * steps / (elapsed * 1e-3), "unit": UNIT,
        "fused_tflops": roof["achieved"], "frac": roof["frac"], "frac_of_sustained": roof["frac_of_sustained"],
        "fused_ms": k1, "fused_ms_x_sm_mhz": (k1 * mhz) if mhz else None,
        "traffic": roof["traffic"], "traffic_source": roof["traffic_source"],
        "k2_finalize": {k: roof["other_kernels"]["k2_finalize"][k] for k in ("ms_per_launch", "achieved", "frac")},
        "k3_detect": dict({k: roof["other_kernels"]["k3_detect"][k] for k in ("ms_per_launch", "achieved", "frac")},
                          us_back_to_back=k3_us),
        "host_us_per_call": host_us, "clocks": clocks,
        "detect": {"threshold": prob.tau, "n_flagged": int(prob.flags.sum().item()),
                   "n_tampered": int(prob.tampered.sum())},
    }
    return entry, prob


def run_ours(args):
    import torch
    import torch.distributed as dist

    import paper_2511_02620_b200 as difr

    rank, local_rank, world = rank_info()
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    difr.lib()  # fail loudly if the CUDA library is missing

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    w = pick_workload(args)
    temperature = float(np.float32(args.temperature))
    sigma = float(np.float32(args.sigma))
    inp = wl.make_inputs(w)
    T, d, V = w.T, w.d, w.V
    events = CudaEvents()
    peaks = load_peaks()

    prob = Problem(difr, w, temperature, sigma, inp=inp)
    small = 2 * (T * d + V * d) <= 2 * L2_BYTES
    flush = torch.empty(256 * 2**20, dtype=torch.uint8, device="cuda") if small else None

    # ---- the headline: W warm-up steps, exactly K timed steps on resident inputs
    elapsed_ms, (k1_ms, k2_ms, k3_ms), clocks = timed_steps(prob, args.steps, args.warmup, events, local_rank,
                                                            barrier, flush)
    n_flagged, n_tampered, tau_used = int(prob.flags.sum().item()), int(prob.tampered.sum()), prob.tau
    flags_ref = prob.flags.cpu().clone()
    stats_np = prob.stats.cpu().numpy()
    host_us = prob.host_us_per_call()
    k3_us = prob.detect_us_back_to_back()
    k3_us_one_sequence = None
    if world == 1:
        seq_keep, stats_keep = prob.seq, prob.stats
        prob.seq, prob.stats = None, torch.empty((1, 4), dtype=torch.int32, device="cuda")
        k3_us_one_sequence = prob.detect_us_back_to_back()  # seq_offsets == NULL: all T rows are one sequence
        prob.seq, prob.stats = seq_keep, stats_keep

    # ---- end to end
    e2e_ms, h2d, d2h, e2e_flags = e2e_rate(prob, args.steps, args.warmup, barrier)
    assert torch.equal(e2e_flags, flags_ref)

    elapsed_ms, e2e_ms, k1_ms = reduce_max([elapsed_ms, e2e_ms, k1_ms], device="cuda")

    # ---- the other estimator on the same resident inputs (context; the headline is Token-DiFR)
    ipt_ms = None
    if world == 1 and temperature > 0:
        out = prob.out
        out.event_fused_start = out.event_fused_stop = 0
        n_ipt = max(1, min(args.steps, 10))
        for _ in range(2):
            difr.difr_score_ipt(prob.h, prob.W, prob.tokens, prob.seeds, prob.pos, temperature, out)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record()
        for _ in range(n_ipt):
            difr.difr_score_ipt(prob.h, prob.W, prob.tokens, prob.seeds, prob.pos, temperature, out)
            difr.difr_detect(out.score, prob.tau, None, None, 0, prob.seq, prob.flags, prob.stats)
        b.record()
        torch.cuda.synchronize()
        ipt_ms = a.elapsed_time(b) / n_ipt
        assert int(out.device_status.item()) == 0, "device-side wait timed out"

    # ---- Alg. Token-DiFR in full under a sampling filter (top-k 50, then top-p 0.95, four competitors): the fused
    #      kernel, storing the logits too, and a collecting pass over them (context; the headline has no filter)
    filt_ms = None
    if world == 1 and temperature > 0:
        fout = difr.DifrOut.allocate(T, d, V, sigma, 1e-12)
        fout.workspace = torch.empty(difr.difr_filtered_workspace_bytes(T, d, V), dtype=torch.uint8, device="cuda")
        n_f = max(1, min(args.steps, 4))
        difr.difr_score_gm_filtered(prob.h, prob.W, prob.tokens, prob.seeds, prob.pos, temperature, 50, 0.95, 4, fout)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record()
        for _ in range(n_f):
            difr.difr_score_gm_filtered(prob.h, prob.W, prob.tokens, prob.seeds, prob.pos, temperature, 50, 0.95, 4,
                                        fout)
            difr.difr_detect(fout.score, prob.tau, fout.margin, None, 0, prob.seq, prob.flags, prob.stats)
        b.record()
        torch.cuda.synchronize()
        filt_ms = a.elapsed_time(b) / n_f
        assert int(fout.device_status.item()) == 0, "device-side wait timed out"
        del fout
        torch.cuda.empty_cache()

    variants = None
    if args.variants and rank == 0:
        variants = time_variants(difr, prob.h, prob.W, prob.tokens, prob.seeds, prob.pos, temperature, sigma, T, d, V)

    # ---- the other target configurations, each timed for at least a second (1-GPU runs only)
    per_config = []
    tokens_np = prob.tokens_np
    if world == 1 and not args.no_per_config and w.name == "longstream":
        for T_other in sorted(w.sweep_T, reverse=True):
            if T_other < T:
                entry, _ = per_config_entry(difr, wl.with_T(w, T_other), temperature, sigma, events, local_rank,
                                            barrier, peaks, share=prob)
                per_config.append(entry)
        del prob, flush
        torch.cuda.empty_cache()
        for name in ("moe30b", "llama8b", "llama3b"):
            w2 = wl.WORKLOADS[name]
            inp2 = wl.make_inputs(w2)
            for temp2 in w2.temperatures:
                entry, p2 = per_config_entry(difr, w2, float(np.float32(temp2)), sigma, events, local_rank, barrier,
                                             peaks, inp=inp2)
                per_config.append(entry)
                del p2
                torch.cuda.empty_cache()
            del inp2

    if rank == 0:
        flop = 2.0 * T * d * V
        value = whole_job_rate(world, T, args.steps, elapsed_ms)
        roof = roofline_of(difr, w, k1_ms, k2_ms, k3_ms, peaks, T // w.seq_len)
        mhz = clocks.get("sm_mhz")
        roof["ms_per_launch_x_sm_mhz"] = (k1_ms * mhz) if mhz else None
        roof["other_kernels"]["k3_detect"]["us_back_to_back"] = k3_us
        roof["other_kernels"]["k3_detect"]["us_back_to_back_one_sequence"] = k3_us_one_sequence
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": elapsed_ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": config_dict(w, args),
            "tflops": world * flop * args.steps / (elapsed_ms * 1e-3) / 1e12,
            "timed_region_s": elapsed_ms * 1e-3,
            "clocks": clocks,
            "e2e": {"value": whole_job_rate(world, T, args.steps, e2e_ms), "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms / args.steps,
                    "note": "per-step inputs (h, tokens, seeds, positions) from pinned host memory, uploaded on a copy "
                            "stream one step ahead of the kernels; scores, flags and statistics read back on a "
                            "third stream; W resident"},
            "gpu_launches": 3 * args.steps,
            "host_us_per_call": host_us,
            "roofline": roof,
            "detect": {"threshold": tau_used, "calibration": "1 % of this batch's untampered rows score below it",
                       "n_flagged": n_flagged, "n_tampered": n_tampered, "n_match": int(stats_np[:, 1].sum())},
        }
        if filt_ms is not None:
            line["token_difr_filtered"] = {"value": T / (filt_ms * 1e-3), "unit": UNIT, "ms_per_step": filt_ms,
                                           "filter": {"top_k": 50, "top_p": 0.95, "s": 4},
                                           "note": "difr_score_gm_filtered + difr_detect, resident inputs; the fused "
                                                   "kernel also stores the logits, a second kernel collects the "
                                                   "candidates from them"}
        if ipt_ms is not None:
            line["token_ipt_difr"] = {"value": T / (ipt_ms * 1e-3), "unit": UNIT, "ms_per_step": ipt_ms,
                                      "tflops": flop / (ipt_ms * 1e-3) / 1e12,
                                      "note": "difr_score_ipt + difr_detect, resident inputs, sigma in CDF units"}
        if per_config:
            line["per_config"] = per_config
        if variants is not None:
            line["variants_ms"] = variants
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
        "score_gm_filtered_whole_vocabulary_nucleus_p095_s4": lambda: difr.difr_score_gm_filtered(
            h, W, tokens, seeds, pos, temperature, 0, 0.95, 4, out),
        "score_ipt_filtered_k1000": lambda: difr.difr_score_ipt_filtered(h, W, tokens, seeds, pos, temperature,
                                                                        1000, 1.0, out),
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
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="longstream", choices=sorted(wl.WORKLOADS),
                    help="default: the long stream (d 5120, V 152064) at T = 262144, the largest target configuration")
    ap.add_argument("--T", type=int, default=0, help="override the number of rows (whole sequences)")
    ap.add_argument("--no-per-config", action="store_true",
                    help="skip the per_config list (the other target configurations, a second of timed steps each)")
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
