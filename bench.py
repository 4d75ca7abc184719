#!/usr/bin/env python
"""Benchmark of the FLy verification step (one JSON line on stdout).

A "step" is one pass of the whole hot path - row reduction (entropy, argmax),
match/gate bits, deferred-window scan, token emission - over one batch of
synthetic logits and draft tokens, through the C ABI.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]
                  [--shard batch|vocab] [--launch graph|stream] [--no-extra] [--no-cpu-baseline]

Headline numbers (`value`, `ms_per_step`, `roofline.frac`) are taken in PLAIN STREAM ORDER: every step's
kernel waits for the previous kernel in the stream before its first read, which is what a decode loop
needs (each round's logits come from the kernel before it).  The same steps with `inputs_ready` (a step
may read while the step before it drains; only valid over inputs that are already complete) are reported
next to them as `overlapped`.

With one GPU and no --no-extra the line also carries `workloads`: every synthetic workload timed the
same way (serial and overlapped; the fused LM-head workload against the tensor roofline).

N > 1: launched by torch.distributed.run, one rank per GPU.  --shard batch (default): every rank verifies
its own B sequences (sequences are independent: weak scaling, no data-path collective).  --shard vocab:
every rank reduces its slice of the vocabulary, the 16-byte row states are all-gathered (NCCL) and every
rank applies the acceptance rule (a tensor-parallel LM head; strong scaling).  The job time is the max
over ranks.

--impl reference times the fp64 CPU oracle (the only "reference implementation" of this method that
exists here) on the host cores, on a bounded sample.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "loose-verify positions/s and HBM GB/s (% of B200 peak) at V=128256 bf16"
UNIT = "positions/s"
FALLBACK_HBM_GBS = 6650.0          # used only if MEASURED_PEAKS.json is absent
FALLBACK_TENSOR = (1590.0, 1400.0)
L2_BYTES = 126 * 1024 * 1024
MIN_TIMED_S = 0.05                 # every timed region lasts at least this long

# dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu captures summarised under profiles/
# (bytes), keyed by kernel; None where the kernel has changed since its counters were taken.
NCU_TRAFFIC = {
    # reduce_rows_flat, long_draft_batch (279,085,056 algorithmic bytes): 279.14 MB read + 3.83 MB written
    # (profiles/reduce_rows_flat_long_draft_batch.md); scaled to other workloads by their algorithmic bytes
    "reduce_rows_flat": {"bytes": 282.97e6, "units": 279085056},
    # lmhead_verify_kernel at V = 64000: 1.0675 GB read + 4.9 MB written (profiles/lmhead_verify_kernel_fused_lm_head.md);
    # scaled by V
    "lmhead_verify_kernel": {"bytes": 1.0724e9, "units": 64000},
}


def ncu_traffic(kernel, scale):
    t = NCU_TRAFFIC.get(kernel)
    return None if t is None else t["bytes"] * scale / t["units"]


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            d = json.load(f)
        return {"hbm": float(d["hbm_gbs"]), "burst": float(d["bf16_tflops"]),
                "sustained": float(d["bf16_tflops_sustained"]), "kind": "measured"}
    except Exception:
        return {"hbm": FALLBACK_HBM_GBS, "burst": FALLBACK_TENSOR[0], "sustained": FALLBACK_TENSOR[1], "kind": "fallback"}


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs (read-only)."""

    def __init__(self, index: int, period_s: float = 0.005):
        self.index, self.period = index, period_s
        self.sm, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thr = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _loop(self):
        nv = self.nv
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4),
        }
        while not self._stop.is_set():
            try:
                self.sm.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for k, bit in names.items():
                    if mask & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(self.period)

    def __enter__(self):
        if self.nv is not None:
            self._thr = threading.Thread(target=self._loop, daemon=True)
            self._thr.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thr is not None:
            self._thr.join(timeout=2)

    def summary(self):
        if not self.sm:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": 0}
        return {"sm_mhz": statistics.median(self.sm), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.sm)}


# ------------------------------------------------------------------------------------------------------
# timing
# ------------------------------------------------------------------------------------------------------

def time_calls(call, n_args, stream, steps, warmup, ranks, launch):
    """Device time of exactly `steps` back-to-back calls call(i % n_args): CUDA events on the launching
    stream, barrier and synchronize on both sides, max over ranks.  launch == "graph": the calls are
    captured once into CUDA graphs (one of up to 8 * n_args steps, replayed, plus one for the remainder),
    so that the host's launch cost is out of the measurement.  Returns milliseconds for all steps."""
    import torch
    from paper_2511_22972_b200 import dist as D
    with torch.cuda.stream(stream):
        for i in range(max(warmup, 3)):
            call(i % n_args)
        stream.synchronize()
        graphs = []
        if launch == "graph":
            per = min(steps, 8 * n_args)
            reps, rem = divmod(steps, per)
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                for i in range(per):
                    call(i % n_args)
            graphs = [(g, reps)]
            if rem:
                g2 = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g2, stream=stream):
                    for i in range(rem):
                        call(i % n_args)
                graphs.append((g2, 1))
            for g_, _ in graphs:
                g_.replay()
        stream.synchronize()
        D.barrier(ranks)
        torch.cuda.synchronize()
        e0 = torch.cuda.Event(enable_timing=True)
        e1 = torch.cuda.Event(enable_timing=True)
        torch.cuda.nvtx.range_push("fly_timed_region")      # lets a profiler list exactly the timed launches
        e0.record(stream)
        if graphs:
            for g_, reps in graphs:
                for _ in range(reps):
                    g_.replay()
        else:
            for i in range(steps):
                call(i % n_args)
        e1.record(stream)
        torch.cuda.nvtx.range_pop()
        stream.synchronize()
        torch.cuda.synchronize()
        D.barrier(ranks)
    return D.max_over_ranks(ranks, e0.elapsed_time(e1))


def steps_for(step_s_estimate, asked):
    """The step count of a timed region: what was asked for, else enough for MIN_TIMED_S."""
    if asked:
        return asked
    return int(min(200000, max(50, MIN_TIMED_S * 1.5 / step_s_estimate)))


def build_inputs(w, device, nbuf, near_miss=True):
    """nbuf distinct (logits, draft) pairs resident on the device.  No entropy guard here: timing does
    not need gate decisions to be precision-proof (the parity tests draw guarded inputs)."""
    import torch
    from paper_2511_22972_b200 import synthetic as S
    bufs = []
    for i in range(nbuf):
        logits = S.make_logits(w, i, device=device)
        rows = logits.view(-1, w.V)
        top = S.rank5(rows) if (near_miss and w.draft_mix[1] > 0) else rows.float().argmax(dim=1, keepdim=True)
        bufs.append((logits, S.make_draft(w, i, top)))
    torch.cuda.synchronize()
    return bufs


def bench_logits(w, ranks, device, steps, warmup, launch, peaks, near_miss=True, splits=0, library_read=False):
    """One logits-path workload: serial (plain stream order) and overlapped (inputs_ready) step times."""
    import torch
    from paper_2511_22972_b200 import FlyVerify, VerifyBuffers
    step_bytes = w.rows * w.V * w.elem_bytes
    nbuf = max(2, -(-int(2.4 * L2_BYTES) // step_bytes))     # rotate over > 2x L2 of distinct inputs
    bufs = build_inputs(w, device, nbuf, near_miss)
    out = VerifyBuffers(w.B, w.K, device)
    fv = FlyVerify(w.B, w.K, w.V, w.dtype, device=ranks.local_rank)
    fv.set_splits(splits)
    carry = w.boundary == "carry"

    def mk(l, d, ready):
        return fv.make_args(w.B, w.K, d, out.accept_len, out.out_tokens, logits=l, theta=w.theta, W=w.W,
                            boundary=w.boundary, state_in=out.state if carry else None, state_out=out.state,
                            rollback=out.rollback, target_argmax=out.target_argmax, entropy=out.entropy,
                            row_flags=out.row_flags, inputs_ready=ready)

    serial_args = [mk(l, d, False) for l, d in bufs]
    ready_args = [mk(l, d, True) for l, d in bufs]
    stream = torch.cuda.Stream(device=device)
    raw = stream.cuda_stream
    n = steps_for(max(step_bytes / (peaks["hbm"] * 1e9), 4e-6), steps)
    res = {"steps": n, "nbuf": nbuf, "step_bytes": step_bytes}
    with ClockSampler(ranks.local_rank) as clk:
        res["serial_ms"] = time_calls(lambda i: fv.run(serial_args[i], raw), nbuf, stream, n, warmup, ranks, launch) / n
        res["launches_per_step"] = fv.last_launch_count
    res["clocks"] = clk.summary()
    with ClockSampler(ranks.local_rank) as clk2:
        res["overlapped_ms"] = time_calls(lambda i: fv.run(ready_args[i], raw), nbuf, stream, n, warmup, ranks, launch) / n
    res["clocks_overlapped"] = clk2.summary()
    if library_read:
        # context only: what a LIBRARY kernel that merely reads the same bytes achieves in the same chain of dependent
        # launches (torch.amax over every row: one streaming read, one max per element, no hand-off between blocks)
        rows = [l.view(-1, w.V) for l, _ in bufs]
        tmp = torch.empty(w.rows, dtype=rows[0].dtype, device=device)
        lib_ms = time_calls(lambda i: torch.amax(rows[i], dim=1, out=tmp), nbuf, stream, n, 3, ranks, launch) / n
        res["library_read_same_bytes"] = {
            "us_per_launch": lib_ms * 1e3, "gbs": step_bytes / (lib_ms * 1e-3) / 1e9,
            "frac": step_bytes / (lib_ms * 1e-3) / 1e9 / peaks["hbm"],
            "note": "torch.amax(logits, dim=-1) over the same buffers in the same plain-stream-order chain: a library "
                    "kernel that only reads the step's bytes; context for what a launch of this size reaches alone"}
    res.update(fv=fv, bufs=bufs, stream=stream, carry=carry)
    return res


def logits_row(w, r, peaks, world):
    """The `workloads` entry of a logits-path workload."""
    gbs = lambda ms: r["step_bytes"] / (ms * 1e-3) / 1e9
    return {
        "rows_per_step": w.rows, "bytes_per_step": r["step_bytes"], "steps": r["steps"],
        "us_per_step_serial": r["serial_ms"] * 1e3, "us_per_step_overlapped": r["overlapped_ms"] * 1e3,
        "positions_per_s_serial": w.rows * world / (r["serial_ms"] * 1e-3),
        "positions_per_s_overlapped": w.rows * world / (r["overlapped_ms"] * 1e-3),
        "gbs_serial": gbs(r["serial_ms"]), "gbs_overlapped": gbs(r["overlapped_ms"]),
        "frac_serial": gbs(r["serial_ms"]) / peaks["hbm"], "frac_overlapped": gbs(r["overlapped_ms"]) / peaks["hbm"],
        "clocks": r["clocks"], "clocks_overlapped": r["clocks_overlapped"],
    }


def h2d_bandwidth(src, device, stream, copies=9):
    """Bandwidth of a pinned host -> device copy of `src` (a pinned tensor: the very buffer `e2e` copies every step),
    GB/s: `copies` single copies, each timed with its own pair of events, median.  This is what bounds `e2e`."""
    import torch
    dst = torch.empty_like(src, device=device)
    nbytes = src.numel() * src.element_size()
    rates = []
    with torch.cuda.stream(stream):
        dst.copy_(src, non_blocking=True)
        stream.synchronize()
        for _ in range(copies):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            dst.copy_(src, non_blocking=True)
            e1.record(stream)
            stream.synchronize()
            rates.append(nbytes / (e0.elapsed_time(e1) * 1e-3) / 1e9)
    return statistics.median(rates)


def e2e_logits(w, r, ranks, device, steps_hint):
    """The same metric end to end through fly_verify_run_host: logits and drafts start in pinned host
    memory every step, results end in host memory, the call synchronises.  Wall clock, max over ranks."""
    import torch
    from paper_2511_22972_b200 import VerifyBuffers, dist as D
    fv, bufs, stream, carry = r["fv"], r["bufs"], r["stream"], r["carry"]
    step_bytes = r["step_bytes"]
    host_l = [b[0].cpu().pin_memory() for b in bufs[:2]]
    host_d = [b[1].cpu().pin_memory() for b in bufs[:2]]
    h2d_gbs = h2d_bandwidth(host_l[0], device, stream)
    est = step_bytes / (h2d_gbs * 1e9) + 30e-6
    e2e_steps = int(max(10, min(400, 0.1 / est)))
    hout = VerifyBuffers(w.B, w.K, device, pinned=True)
    hargs = [fv.make_args(w.B, w.K, d, hout.accept_len, hout.out_tokens, logits=l, theta=w.theta, W=w.W,
                          boundary=w.boundary, state_in=hout.state if carry else None, state_out=hout.state,
                          rollback=hout.rollback, target_argmax=hout.target_argmax, entropy=hout.entropy,
                          row_flags=hout.row_flags) for l, d in zip(host_l, host_d)]
    raw = stream.cuda_stream
    for i in range(3):
        fv.run_host(hargs[i % 2], raw)
    D.barrier(ranks)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for i in range(e2e_steps):
        fv.run_host(hargs[i % 2], raw)          # synchronises the stream before returning
    torch.cuda.synchronize()
    e2e_s = D.max_over_ranks(ranks, time.perf_counter() - t0)
    h2d = step_bytes + w.B * w.K * 4 + (w.B * 12 if carry else 0)
    d2h = w.B * 4 * 2 + w.rows * 4 * 4 + w.B * 12
    value = w.rows * ranks.world * e2e_steps / e2e_s
    bound = w.rows * ranks.world / (h2d / (h2d_gbs * 1e9))
    return {"value": value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps,
            "us_per_step": e2e_s / e2e_steps * 1e6,
            "h2d_gbs_measured": h2d_gbs, "bound": "pcie h2d copy of the step's logits",
            "bound_value": bound, "frac_of_bound": value / bound,
            "api": "fly_verify_run_host (pinned host buffers)"}


# ------------------------------------------------------------------------------------------------------
# CPU oracle legs
# ------------------------------------------------------------------------------------------------------

_BARRIER = None


def _pool_init(barrier):
    global _BARRIER
    _BARRIER = barrier
    import torch
    torch.set_num_threads(1)


def _oracle_worker(job):
    """One worker process of the CPU baseline.  It draws its own share of the step (same recipe, its own
    seed; untimed), waits until every worker is ready, then runs the oracle as it stands.  Returns the
    system-wide monotonic clock at the start and at the end of the oracle call."""
    import numpy as np
    from oracle import fly_oracle as O
    from paper_2511_22972_b200 import synthetic as S
    ws, step = job
    logits = S.make_logits(ws, step, device="cpu")
    rows = logits.view(-1, ws.V)
    top = S.rank5(rows) if ws.draft_mix[1] > 0 else rows.float().argmax(dim=1, keepdim=True)
    d = S.make_draft(ws, step, top).numpy()
    x = logits.double().numpy()
    st = np.array([[0, 0, -1]] * ws.B) if ws.boundary == "carry" else None
    _BARRIER.wait()
    t0 = time.perf_counter()
    O.verify_batch(x, d, ws.theta, ws.W, boundary=ws.boundary, state_in=st)
    return t0, time.perf_counter()


class OraclePool:
    """The fp64 oracle on all host cores: sequences are independent, so every core verifies its own few
    sequences of the workload's recipe with the (single-threaded, untouched) oracle, all at the same time.
    One round's time is the wall clock from the first worker's start to the last worker's end."""

    def __init__(self, w, rows_per_core):
        import multiprocessing as mp
        from paper_2511_22972_b200 import synthetic as S
        cores = len(os.sched_getaffinity(0))
        self.share = max(1, min(-(-w.B // cores), rows_per_core // (w.K + 1)))   # sequences per worker and round
        self.workers = max(1, min(cores, w.B // self.share))
        self.ws = S.shrink(w, B=self.share)
        ctx = mp.get_context("forkserver")   # workers are forked from a clean server process, not from this CUDA process
        self.pool = ctx.Pool(self.workers, initializer=_pool_init, initargs=(ctx.Barrier(self.workers),))
        self.rows_per_round = self.workers * self.ws.rows
        self.w = w

    def round(self, step):
        spans = self.pool.map(_oracle_worker, [(self.ws, step * self.workers + i) for i in range(self.workers)], chunksize=1)
        return max(t1 for _, t1 in spans) - min(t0 for t0, _ in spans)

    def sample(self, rounds):
        return (f"{rounds} rounds of {self.workers} worker processes x {self.share} of {self.w.B} sequences x "
                f"{self.ws.K + 1} rows x V={self.ws.V} ({self.w.dtype} widened to fp64)")

    def close(self):
        self.pool.close()
        self.pool.join()


def oracle_rate(w, seconds_budget=12.0):
    """rows/s of the oracle on this host's cores, a description of the sample, and the cores used."""
    op = OraclePool(w, rows_per_core=40)
    try:
        op.round(10 ** 6)                                   # untimed: pages in the workers
        rows_done, t_used, rounds = 0, 0.0, 0
        while t_used < seconds_budget:
            t_used += op.round(rounds)
            rows_done += op.rows_per_round
            rounds += 1
        return rows_done / t_used, op.sample(rounds), op.workers
    finally:
        op.close()


def fused_oracle_sample(w, weight_cpu, seq, step):
    """The oracle on `seq` sequences of the fused workload (all V): exact fp64 logits, then the usual
    verification.  The product is taken in vocabulary slices so that the fp64 copy of the weight never
    exists as a whole; only the oracle calls are timed.  Returns (seconds, rows)."""
    import numpy as np
    from oracle import fly_oracle as O
    from paper_2511_22972_b200 import synthetic as S
    ws = S.shrink(w, B=seq)
    hidden = S.make_hidden(ws, step, device="cpu").double().numpy()
    draft = np.random.default_rng(step).integers(0, w.V, size=(seq, w.K)).astype(np.int32)
    t, parts = 0.0, []
    for v0 in range(0, w.V, 16032):
        wd = weight_cpu[:, v0:v0 + 16032].double().numpy()
        t0 = time.perf_counter()
        parts.append(O.lm_head_logits(hidden, wd))
        t += time.perf_counter() - t0
    t0 = time.perf_counter()
    logits = np.concatenate(parts, axis=1).reshape(seq, w.K + 1, w.V)
    O.verify_batch(logits, draft, w.theta, w.W, boundary=w.boundary)
    t += time.perf_counter() - t0
    return t, ws.rows


# ------------------------------------------------------------------------------------------------------
# fused LM-head workload
# ------------------------------------------------------------------------------------------------------

def bench_fused(w, ranks, device, steps, warmup, peaks, e2e=True, library=True):
    """hidden [B*(K+1), D] x weight [D, V] with the verification in the epilogue; tensor roofline."""
    import torch
    from paper_2511_22972_b200 import FlyVerify, VerifyBuffers, binding as Bd, dist as D, synthetic as S
    weight = S.make_weight(w, device=device)
    nbuf = 4
    hiddens = [S.make_hidden(w, i, device=device) for i in range(nbuf)]
    # synthetic drafter: the (library, fp32) argmax with p = 0.7, else uniform over V
    drafts = [S.make_draft(w, i, (h.float() @ weight.float()).argmax(dim=1, keepdim=True)) for i, h in enumerate(hiddens)]
    torch.cuda.synchronize()
    out = VerifyBuffers(w.B, w.K, device)
    fv = FlyVerify(w.B, w.K, w.V, "bf16", device=ranks.local_rank, hidden=w.hidden)
    mk = lambda h, d, o: fv.make_args(w.B, w.K, d, o.accept_len, o.out_tokens, hidden=h, weight=weight, theta=w.theta,
                                      W=w.W, boundary=w.boundary, state_out=o.state, rollback=o.rollback,
                                      target_argmax=o.target_argmax, entropy=o.entropy, row_flags=o.row_flags)
    arglist = [mk(h, d, out) for h, d in zip(hiddens, drafts)]
    stream = torch.cuda.Stream(device=device)
    raw = stream.cuda_stream
    flops = 2.0 * w.rows * w.hidden * w.V
    n = steps_for(flops / (peaks["burst"] * 1e12), steps)
    with ClockSampler(ranks.local_rank) as clk:
        ms = time_calls(lambda i: fv.run(arglist[i], raw), nbuf, stream, n, warmup, ranks, "stream") / n
        launches_per_step = fv.last_launch_count
    if fv.device_status(raw) != Bd.FLY_OK:
        raise SystemExit("a bounded device-side wait ran out: the measurement is void")
    achieved = flops / (ms * 1e-3) / 1e12
    res = {"steps": n, "ms": ms, "flops": flops, "tflops": achieved, "launches_per_step": launches_per_step,
           "clocks": clk.summary(), "frac_of_burst": achieved / peaks["burst"],
           "frac_of_sustained": achieved / peaks["sustained"],
           "hbm_gbs": (w.hidden * w.V * 2 + w.rows * w.hidden * 2) / (ms * 1e-3) / 1e9}
    if e2e:
        # end to end: hidden states and drafts come from pinned host memory every step, results go back
        e2e_steps = max(10, min(100, n // 2))
        hout = VerifyBuffers(w.B, w.K, device, pinned=True)
        hargs = [mk(h.cpu().pin_memory(), d.cpu().pin_memory(), hout) for h, d in zip(hiddens[:2], drafts[:2])]
        for i in range(3):
            fv.run_host(hargs[i % 2], raw)
        D.barrier(ranks)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for i in range(e2e_steps):
            fv.run_host(hargs[i % 2], raw)
        torch.cuda.synchronize()
        e2e_s = D.max_over_ranks(ranks, time.perf_counter() - t0)
        res["e2e"] = {"value": w.rows * ranks.world * e2e_steps / e2e_s, "unit": UNIT,
                      "h2d_bytes_per_step": w.rows * w.hidden * 2 + w.B * w.K * 4,
                      "d2h_bytes_per_step": w.B * 4 * 2 + w.rows * 4 * 4 + w.B * 12, "steps": e2e_steps,
                      "api": "fly_verify_run_host (hidden states and drafts in pinned host buffers; weight resident)"}
    if library:
        # context only: the library GEMM (torch.matmul -> cuBLAS) on the SAME shape, writing bf16 logits, same
        # number of back-to-back launches.  It does none of the verification; it shows what the shape allows.
        lib_logits = torch.empty(w.rows, w.V, dtype=torch.bfloat16, device=device)
        with torch.cuda.stream(stream):
            for _ in range(3):
                torch.matmul(hiddens[0], weight, out=lib_logits)
            stream.synchronize()
            l0, l1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            l0.record(stream)
            for i in range(n):
                torch.matmul(hiddens[i % nbuf], weight, out=lib_logits)
            l1.record(stream)
            stream.synchronize()
        lib_ms = l0.elapsed_time(l1) / n
        res["library_gemm_same_shape"] = {
            "us_per_step": lib_ms * 1e3, "tflops": flops / (lib_ms * 1e-3) / 1e12,
            "note": "torch.matmul (cuBLAS) hidden x weight -> bf16 logits only, no verification; context, "
                    "timed after the main measurement"}
        del lib_logits
    res["weight"] = weight
    fv.close()
    return res


def fused_row(w, r):
    row = {"rows_per_step": w.rows, "flops_per_step": r["flops"], "steps": r["steps"], "us_per_step": r["ms"] * 1e3,
           "positions_per_s": w.rows / (r["ms"] * 1e-3), "tflops": r["tflops"], "frac_of_burst": r["frac_of_burst"],
           "frac_of_sustained": r["frac_of_sustained"], "clocks": r["clocks"]}
    if "library_gemm_same_shape" in r:
        row["library_gemm_same_shape"] = r["library_gemm_same_shape"]
    return row


def run_fused(args, w):
    import torch
    from paper_2511_22972_b200 import dist as D
    warmup = 5 if args.warmup is None else max(args.warmup, 3)
    ranks = D.init_from_env("nccl")
    assert ranks.world == args.gpus, f"--gpus {args.gpus} but WORLD_SIZE={ranks.world}"
    torch.cuda.set_device(ranks.local_rank)
    device = torch.device("cuda", ranks.local_rank)
    peaks = measured_peaks()
    r = bench_fused(w, ranks, device, args.steps or 200, warmup, peaks)
    rows_all = w.rows * ranks.world
    line = {
        "metric": METRIC, "value": rows_all / (r["ms"] * 1e-3), "unit": UNIT, "n_gpus": ranks.world, "steps": r["steps"],
        "warmup": warmup, "ms_per_step": r["ms"], "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": w.name, "B_per_gpu": w.B, "K": w.K, "V": w.V, "hidden": w.hidden,
                   "theta_nats": w.theta, "W": w.W, "boundary": w.boundary, "parallelism": f"dp{ranks.world}",
                   "launch": "stream", "l2": f"the weight ({w.hidden * w.V * 2 / 1e9:.2f} GB, read once per step) is larger than L2"},
        "tflops": r["tflops"],
        "roofline": {"bound": "tensor", "kernel": "lmhead_verify_kernel (tcgen05 GEMM + entropy/argmax epilogue)",
                     "achieved": r["tflops"], "peak": peaks["burst"], "peak_kind": f"of {peaks['kind']} (bf16 burst)",
                     "unit": "TFLOP/s", "frac": r["tflops"] / peaks["burst"], "frac_of_sustained": r["frac_of_sustained"],
                     "flops_per_launch": r["flops"], "us_per_launch": r["ms"] * 1e3,
                     "note": "duration = whole step (GEMM kernel + fold + acceptance-scan kernels, the latter two ~3 us)",
                     "traffic": ncu_traffic("lmhead_verify_kernel", w.V)},
        "hbm_gbs": r["hbm_gbs"],
        "library_gemm_same_shape": r["library_gemm_same_shape"],
        "e2e": r["e2e"],
        "gpu_launches": r["launches_per_step"] * r["steps"],
        "clocks": r["clocks"],
    }
    if ranks.is_main and ranks.world == 1 and not args.no_cpu_baseline:
        wc = r["weight"].cpu()
        t, rows = fused_oracle_sample(w, wc, 1, 0)
        line["cpu_baseline"] = {"value": rows / t, "unit": UNIT, "cores": len(os.sched_getaffinity(0)), "kind": "oracle",
                                "sample": f"1 of {w.B} sequences ({rows} rows, all V={w.V}): fp64 matmul (BLAS threads) + verification (1 thread)"}
    if ranks.is_main:
        print(json.dumps(line), flush=True)
    D.finalize(ranks)


# ------------------------------------------------------------------------------------------------------
# vocabulary-parallel mode
# ------------------------------------------------------------------------------------------------------

def run_vocab_parallel(args, w):
    """--shard vocab: a tensor-parallel LM head leaves every rank with one slice of the vocabulary.  Per step
    every rank reduces its slice to one 16-byte state per row (fly_verify_reduce_shard), the states are
    all-gathered (one NCCL call; world 1: none) and every rank applies the rule (fly_verify_run_partials)."""
    import torch
    from paper_2511_22972_b200 import FlyVerify, VerifyBuffers, dist as D, synthetic as S
    warmup = 10 if args.warmup is None else max(args.warmup, 3)
    if args.gpus > 1:
        os.environ.setdefault("NCCL_DEBUG", "INFO")           # the communicator log shows the ranks and NVLS
        os.environ.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
    ranks = D.init_from_env("nccl")
    assert ranks.world == args.gpus, f"--gpus {args.gpus} but WORLD_SIZE={ranks.world}"
    torch.cuda.set_device(ranks.local_rank)
    device = torch.device("cuda", ranks.local_rank)
    peaks = measured_peaks()
    off, width = D.shard_vocab(w.V, ranks)
    ws = S.shrink(w, V=width)                                 # this rank's slice, drawn with the workload's recipe
    slice_bytes = w.rows * width * w.elem_bytes
    nbuf = max(2, -(-int(2.4 * L2_BYTES) // slice_bytes))
    slices = [S.make_logits(ws, 1000 * ranks.rank + i, device=device).view(w.rows, width) for i in range(nbuf)]
    draft = torch.randint(0, w.V, (w.B, w.K), device=device, dtype=torch.int32)
    out = VerifyBuffers(w.B, w.K, device)
    shard = FlyVerify(w.B, w.K, width, w.dtype, device=ranks.local_rank)
    merge = FlyVerify(w.B, w.K, w.V, w.dtype, device=ranks.local_rank)
    mine = torch.empty(w.rows, 4, dtype=torch.float32, device=device)
    margs = merge.make_args(w.B, w.K, draft, out.accept_len, out.out_tokens, theta=w.theta, W=w.W, state_out=out.state,
                            rollback=out.rollback, target_argmax=out.target_argmax, entropy=out.entropy,
                            row_flags=out.row_flags)
    stream = torch.cuda.Stream(device=device)
    raw = stream.cuda_stream

    def step(i):
        shard.reduce_shard(slices[i], off, mine, raw)
        allp = D.all_gather_partials(ranks, mine)
        merge.run_partials(margs, allp, ranks.world, w.V, raw)

    n = steps_for(max(slice_bytes / (peaks["hbm"] * 1e9), 10e-6), args.steps)
    with ClockSampler(ranks.local_rank) as clk:
        ms = time_calls(step, nbuf, stream, n, warmup, ranks, "stream") / n
    value = w.rows / (ms * 1e-3)
    achieved = slice_bytes / (ms * 1e-3) / 1e9
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": ranks.world, "steps": n, "warmup": warmup,
        "ms_per_step": ms, "higher_is_better": True, "scaling": "strong", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic",
        "config": {"workload": w.name, "B": w.B, "K": w.K, "V": w.V, "V_per_gpu": width, "logits_dtype": w.dtype,
                   "theta_nats": w.theta, "W": w.W, "boundary": "reject", "parallelism": f"tp{ranks.world}",
                   "launch": "stream", "collective": "all-gather of 16 bytes per row and rank" if ranks.world > 1 else "none (one rank)",
                   "l2": f"slices rotate over {nbuf} distinct buffers = {nbuf * slice_bytes / 1e6:.0f} MB per GPU (> 2x L2)"},
        "roofline": {"bound": "hbm", "kernel": "reduce_rows_flat (this rank's vocabulary slice)", "achieved": achieved,
                     "peak": peaks["hbm"], "peak_kind": f"of {peaks['kind']}", "unit": "GB/s", "frac": achieved / peaks["hbm"],
                     "bytes_per_launch": slice_bytes, "us_per_launch": ms * 1e3,
                     "note": "duration = whole step: slice reduction + fold + all-gather + merge + acceptance scan",
                     "traffic": ncu_traffic("reduce_rows_flat", w.rows * width * w.elem_bytes)},
        "e2e": None,
        "gpu_launches": 4 * n,
        "clocks": clk.summary(),
    }
    if ranks.is_main:
        print(json.dumps(line), flush=True)
    shard.close()
    merge.close()
    D.finalize(ranks)


# ------------------------------------------------------------------------------------------------------
# reference arm (the oracle)
# ------------------------------------------------------------------------------------------------------

def run_reference_fused(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2511_22972_b200 import synthetic as S
    weight = S.make_weight(w, device="cpu")
    for i in range(args.warmup):
        fused_oracle_sample(w, weight, 1, i)
    tot, rows = 0.0, 0
    for i in range(args.steps):
        t, r = fused_oracle_sample(w, weight, 1, 100 + i)
        tot += t
        rows += r
    value = rows / tot
    sample = f"each step = 1 of {w.B} sequences ({w.K + 1} rows, all V={w.V}), fp64 matmul + verification"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": tot / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "B": w.B, "K": w.K, "V": w.V, "hidden": w.hidden, "theta_nats": w.theta,
                   "W": w.W, "boundary": w.boundary, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": len(os.sched_getaffinity(0)), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def run_reference(args, w):
    """--impl reference: the oracle on the host cores; rank 0 only.  Each step is a bounded sample of the
    workload: a few sequences per core, all cores at once."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    op = OraclePool(w, rows_per_core=24)
    try:
        for i in range(args.warmup):
            op.round(10 ** 6 + i)
        dt = sum(op.round(i) for i in range(args.steps))
    finally:
        op.close()
    value = op.rows_per_round * args.steps / dt
    sample = "each step = " + op.sample(1).split(" of ", 1)[1]
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "B": w.B, "K": w.K, "V": w.V, "logits_dtype": w.dtype, "theta_nats": w.theta,
                   "W": w.W, "boundary": w.boundary, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": op.workers, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------------------

EXTRA_WORKLOADS = ("tiny_verify", "llama3_vocab_batch", "long_draft_batch", "high_batch_serving",
                   "paper_default_70b", "paper_default_405b", "fused_lm_head")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--workload", default="llama3_vocab_batch")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--launch", default="graph", choices=["stream", "graph"],
                    help="logits path: launch the timed steps from CUDA graphs (default) or one by one from the host")
    ap.add_argument("--shard", default="batch", choices=["batch", "vocab"])
    ap.add_argument("--no-extra", action="store_true", help="time only --workload (no `workloads` object)")
    ap.add_argument("--splits", type=int, default=0, help="logits path: cut every row into exactly this many pieces "
                    "(FLY_OPT_SPLITS; 0 = the library's own choice); recorded in config")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--vocab", type=int, default=None, help="run the workload's recipe at another vocabulary size "
                    "(smaller cases for profiler captures); recorded in config")
    ap.add_argument("--batch", type=int, default=None, help="run the workload's recipe at another batch size")
    args = ap.parse_args()

    from paper_2511_22972_b200 import synthetic as S
    w = S.WORKLOADS[args.workload]
    if args.vocab or args.batch:
        w = S.shrink(w, V=args.vocab or w.V, B=args.batch or w.B)
    if args.impl == "reference":
        args.steps = args.steps or 5
        args.warmup = 1 if args.warmup is None else args.warmup
        (run_reference_fused if w.hidden else run_reference)(args, w)
        return
    if w.hidden:
        run_fused(args, w)
        return
    if args.shard == "vocab":
        run_vocab_parallel(args, w)
        return
    warmup = 20 if args.warmup is None else max(args.warmup, 3)

    import torch
    from paper_2511_22972_b200 import dist as D
    ranks = D.init_from_env("nccl")
    assert ranks.world == args.gpus, f"--gpus {args.gpus} but WORLD_SIZE={ranks.world}"
    torch.cuda.set_device(ranks.local_rank)
    device = torch.device("cuda", ranks.local_rank)
    peaks = measured_peaks()

    # ---- the named workload: whole steps over device-resident inputs, serial and overlapped ---------------
    r = bench_logits(w, ranks, device, args.steps, warmup, args.launch, peaks, splits=args.splits,
                     library_read=ranks.world == 1)
    assert r["launches_per_step"] == 1, r["launches_per_step"]     # the acceptance scan is the tail of the reduction
    ms_per_step = r["serial_ms"]
    rows_all = w.rows * ranks.world
    value = rows_all / (ms_per_step * 1e-3)
    achieved = r["step_bytes"] / (ms_per_step * 1e-3) / 1e9
    e2e = e2e_logits(w, r, ranks, device, r["steps"])
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": ranks.world, "steps": r["steps"],
        "warmup": warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": w.name, "B_per_gpu": w.B, "K": w.K, "V": w.V, "logits_dtype": w.dtype,
                   "theta_nats": w.theta, "W": w.W, "boundary": w.boundary, "parallelism": f"dp{ranks.world}",
                   "launch": args.launch, "splits": args.splits or "auto", "order": "plain stream order (each step waits for the previous kernel before its first read)",
                   "l2": f"inputs rotate over {r['nbuf']} distinct buffers = {r['nbuf'] * r['step_bytes'] / 1e6:.0f} MB (> 2x L2)"},
        "hbm_gbs": rows_all * w.V * w.elem_bytes / (ms_per_step * 1e-3) / 1e9,
        "hbm_pct_of_peak": 100.0 * achieved / peaks["hbm"],
        "overlapped": {"ms_per_step": r["overlapped_ms"], "value": rows_all / (r["overlapped_ms"] * 1e-3),
                       "frac": r["step_bytes"] / (r["overlapped_ms"] * 1e-3) / 1e9 / peaks["hbm"],
                       "note": "same steps with inputs_ready: a step may read its logits while the previous step drains; "
                               "valid only over inputs that are complete beforehand, not inside a decode loop"},
        "roofline": {"bound": "hbm", "kernel": "reduce_rows_flat (row reduction + acceptance scan in its tail; one launch per step)",
                     "achieved": achieved, "peak": peaks["hbm"], "peak_kind": f"of {peaks['kind']} (copy bandwidth)",
                     "unit": "GB/s", "frac": achieved / peaks["hbm"], "bytes_per_launch": r["step_bytes"],
                     "us_per_launch": ms_per_step * 1e3,
                     "note": "one launch per step in plain stream order, so the step time is the launch duration plus "
                             "the gap to the next launch",
                     "frac_overlapped": r["step_bytes"] / (r["overlapped_ms"] * 1e-3) / 1e9 / peaks["hbm"],
                     "library_read_same_bytes": r.get("library_read_same_bytes"),
                     "traffic": ncu_traffic("reduce_rows_flat", w.rows * w.V * w.elem_bytes)},
        "e2e": e2e,
        "gpu_launches": r["launches_per_step"] * r["steps"],
        "clocks": r["clocks"],
    }
    main_row = logits_row(w, r, peaks, ranks.world)
    long_enough = r["steps"] * r["serial_ms"] * 1e-3 >= MIN_TIMED_S
    r["fv"].close()
    del r

    # ---- every other workload, same protocol (one GPU only: it is a report, not part of the scaling run) ----
    if ranks.world == 1 and not args.no_extra and not (args.vocab or args.batch):
        rows = {}
        for name in EXTRA_WORKLOADS:
            wx = S.WORKLOADS[name]
            torch.cuda.empty_cache()
            if name == w.name and long_enough:
                rows[name] = main_row
            elif wx.hidden:
                rf = bench_fused(wx, ranks, device, None, 5, peaks, e2e=False)
                rows[name] = fused_row(wx, rf)
                del rf
            else:
                rx = bench_logits(wx, ranks, device, None, warmup, args.launch, peaks, near_miss=False)
                rows[name] = logits_row(wx, rx, peaks, 1)
                rx["fv"].close()
                del rx
        line["workloads"] = rows
    if ranks.is_main and ranks.world == 1 and not args.no_cpu_baseline:
        v, sample, cores = oracle_rate(w)
        line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample}
    if ranks.is_main:
        print(json.dumps(line), flush=True)
    D.finalize(ranks)


if __name__ == "__main__":
    main()
