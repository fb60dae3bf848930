#!/usr/bin/env python
"""Benchmark of the chunk-pipelined reduce / broadcast hot path on B200.

    python bench.py --gpus N --steps K --warmup W [--workload cfg4] [--impl ours|reference]

One step is one pass of the whole path over one batch of synthetic objects of the chosen workload:
directory updates on Put, arrival ordering and tree formation, the kernels, Get.  The default workload
is the policy round (broadcast a 64 MiB bf16 object to 64 receivers, then sum 64 returned bf16 objects
in fp32, chunk 2 MiB, degree 4): the largest single-GPU configuration that uses both collectives.
Inputs are resident in HBM before the timed region; every step is bracketed by CUDA events on the
library's stream and the K steps by a barrier + synchronize.  Rank 0 prints one JSON line.

With N > 1 every rank runs the same workload on its own GPU (independent rounds: the path has no
exchange step between GPUs), the time is the maximum over ranks and the value the sum over ranks.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

import workloads as wl  # noqa: E402

MiB = 1 << 20
FALLBACK_HBM_GBS = 6650.0
# the headline value is effective GB/s = algorithmic bytes / time of the default workload; the curve against object size
# and the fractions of the HBM peak are in the same line (`sweep`, `frac_of_hbm_peak`, `roofline`)
METRIC = "reduce/broadcast effective GB/s and fraction of HBM peak vs object size, 1 B200"

KERNEL_SOURCES = ("paper_2002_05814_b200/csrc/kernels.cu", "paper_2002_05814_b200/csrc/device_types.h")


def kernel_source_hash() -> str:
    """Hash of the kernel sources as they stand: an ncu figure is only quoted for the kernels it was taken on."""
    import hashlib
    h = hashlib.sha256()
    for rel in KERNEL_SOURCES:
        with open(os.path.join(ROOT, rel), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def ncu_traffic(workload: str, kernel: str):
    """dram__bytes_read.sum + dram__bytes_write.sum per full-size launch, from the record line of the ncu summary
    under profiles/ (`bench-record: workload=... kernel=... traffic_bytes=... kernel_sources=<hash>`).  None when
    there is no record or the kernels have changed since the counters were taken."""
    import glob
    import re
    cur = kernel_source_hash()
    for path in sorted(glob.glob(os.path.join(ROOT, "profiles", "*.md"))):
        with open(path) as f:
            for ln in f:
                m = re.search(r"bench-record: workload=(\S+) kernel=(\S+) traffic_bytes=(\S+) kernel_sources=(\S+)", ln)
                if m and m.group(1) == workload and m.group(2) == kernel:
                    return float(m.group(3)) if m.group(4) == cur else None
    return None


# ----------------------------------------------------------------------------------------- helpers
def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines: list[str] = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for ln in self.lines:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for nm, val in zip(names, parts[2:6]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def algorithmic_bytes(w: wl.Workload) -> dict:
    """Bytes the method must move: every selected source read once and the result written once; the
    broadcast source read once and every receiver written once."""
    S = w.object_bytes
    out = {"reduce": 0, "broadcast": 0}
    if w.kind in ("reduce", "round"):
        out["reduce"] = w.k * S + w.elems * 4
    if w.kind == "ft_reduce":
        out["reduce"] = (w.k - 1) * S + w.elems * 4          # the survivors and the result
    if w.kind in ("broadcast", "round"):
        out["broadcast"] = S + w.n_receivers * S
    if w.kind == "multi_reduce":
        out["reduce"] = w.extra["collectives"] * (w.k * S + w.elems * 4)
    if w.kind == "allreduce":
        # reduce followed by broadcast of its output: the sources read once, the result written once to the target
        # and once to every receiver (reading the target back is not part of what the method must move)
        out["reduce"] = w.k * S + w.elems * 4
        out["broadcast"] = w.n_receivers * w.elems * 4
    return out


# ----------------------------------------------------------------------------------------- our arm
class Runner:
    """Holds the device buffers of one workload and runs steps through the C ABI."""

    def __init__(self, w: wl.Workload, device, host_buffers: bool = False, plan_ahead: bool = False, ft_eager: bool = True,
                 fuse_fanout: bool = True):
        import torch
        import paper_2002_05814_b200 as hpl

        self.torch, self.hpl, self.w = torch, hpl, w
        self.dt = hpl.HPL_BF16 if w.dtype == "bf16" else hpl.HPL_F32
        S = w.object_bytes
        self.host_buffers = host_buffers
        self.ft_eager = ft_eager
        n_src = w.n_objects * w.extra.get("collectives", 1)
        arena_bytes = 64 * MiB + 2 * w.elems * 4 + (n_src + 2) * S * (1 if host_buffers else 0)
        if w.kind == "ft_reduce":
            arena_bytes += 8 * w.elems * 4       # partial results of the subtrees beside the failing worker's root path
        arena_bytes += w.extra.get("partials", 0) * w.elems * 4
        self.arena = torch.empty(arena_bytes, dtype=torch.uint8, device=device)
        self.plan_ahead = plan_ahead
        self.fuse_fanout = fuse_fanout
        self.ctx_flags = {}          # further context settings (degree sweep: fuse, the Eq. 1 model)
        self.ctx = None
        self.open_context(time_kernels=False)
        self.src = [wl.values_torch(w.dist, w.seed + i, i, 0, w.elems, w.dtype, device=device) for i in range(n_src)]
        self.policy = None
        self.recv = []
        if w.n_receivers:
            if w.kind != "allreduce":
                self.policy = wl.values_torch(w.dist, w.seed + 1000, 1000, 0, w.elems, w.dtype, device=device)
            self.recv = [torch.empty(w.elems * 4 if w.kind == "allreduce" else S, dtype=torch.uint8, device=device)
                         for _ in range(w.n_receivers)]
        self.host_src, self.host_policy, self.host_out, self.host_recv = [], None, None, None
        if host_buffers:
            n_distinct = min(n_src, 8)      # pinned host images; objects beyond the 8th reuse them (same bytes to copy)
            self.host_src = [self.src[i].cpu().pin_memory() for i in range(n_distinct)]
            if self.policy is not None:
                self.host_policy = self.policy.cpu().pin_memory()
                self.host_recv = torch.empty(S, dtype=torch.uint8).pin_memory()
            if n_src:
                self.host_out = torch.empty(w.elems, dtype=torch.float32).pin_memory()
        self.round = 0
        self.prepared = {}
        torch.cuda.synchronize()

    def open_context(self, time_kernels: bool):
        """(Re)creates the context on the same arena and buffers.  Per-launch event timing is a mode of its own: its
        two event records per launch would otherwise sit inside the step times they are compared with."""
        torch, w = self.torch, self.w
        if self.ctx is not None:
            self.ctx.shutdown()
        self.ctx = self.hpl.Context(w.chunk_bytes, w.degree, max(1, w.degree), arena=self.arena.data_ptr(), arena_bytes=self.arena.numel(),
                                    stream=torch.cuda.current_stream().cuda_stream, time_kernels=time_kernels,
                                    plan_ahead=self.plan_ahead, fuse_fanout=self.fuse_fanout, **self.ctx_flags)
        self.prepared = {}

    def close(self):
        self.ctx.shutdown()

    # ---- the timeline of one round, prepared outside the timed region (it is input data, like the objects)
    def build_round(self, r: int, marks=None):
        """Event lists of round ``r``: (first part, second part, deletes, h2d bytes, d2h bytes).  The first part
        holds the broadcast of the round (if any), the second the reduce; each is applied by ONE hpl_submit.
        ``marks``: three CUDA event handles the library records on its stream at the start of the step, between
        the two parts (when the step has two) and at the end (device timing without a foreign call of its own)."""
        H, w = self.hpl, self.w
        S = w.object_bytes
        t = (r + 1) * 2_000_000_000
        n, R = w.n_objects, w.n_receivers
        if w.kind == "multi_reduce":
            # many small collectives requested together: their tasks share waves and the Gets wait once
            m = w.extra["collectives"]
            e2, dl = H.EventList(8 + m * (2 * n + 2)), H.EventList(4 + m * (n + 1))
            if marks:
                e2.add(H.HPL_EV_MARK, 0, ptr=marks[0])
            for q in range(m):
                ids = list(range(q * n, (q + 1) * n))
                for i in ids:
                    e2.add(H.HPL_EV_CREATE, t, i, i, nbytes=w.object_bytes, dtype=self.dt)
                    e2.add(H.HPL_EV_PUT, t, i, ptr=self.src[i].data_ptr(), nbytes=w.object_bytes)
            for q in range(m):
                e2.add(H.HPL_EV_REDUCE, t, 100_000 + q, ids=list(range(q * n, (q + 1) * n)), k=w.k, op=H.HPL_SUM, dtype=self.dt)
            for q in range(m):
                e2.add(H.HPL_EV_GET, 0, 100_000 + q)
            for q in range(m):
                dl.add(H.HPL_EV_DELETE, 0, 100_000 + q)
                for i in range(q * n, (q + 1) * n):
                    dl.add(H.HPL_EV_DELETE, 0, i)
            if marks:
                e2.add(H.HPL_EV_MARK, 0, ptr=marks[2])
            return H.EventList(1), e2, dl, 0, 0
        e1, e2, dl = H.EventList(12 + 3 * R + n), H.EventList(12 + 3 * n + 3 * R), H.EventList(4 + n)
        h2d = d2h = 0
        put_kind = H.HPL_EV_PUT_HOST if self.host_buffers else H.HPL_EV_PUT
        ids = list(range(n))
        tgt = 9000
        early = w.kind == "round" and not self.host_buffers
        first = e1 if w.kind in ("broadcast", "round") else e2
        if marks:
            first.add(H.HPL_EV_MARK, 0, ptr=marks[0])
        if w.kind in ("broadcast", "round"):
            src_id = 5000
            dsts = [6000 + j for j in range(R)]
            e1.add(H.HPL_EV_CREATE, t, src_id, 900, nbytes=S, dtype=self.dt)
            if self.host_buffers:
                e1.add(put_kind, t, src_id, ptr=self.host_policy.data_ptr(), nbytes=S)
                h2d += S
            else:
                e1.add(put_kind, t, src_id, ptr=self.policy.data_ptr(), nbytes=S)
            for j in range(R):
                e1.add(H.HPL_EV_CREATE, t, dsts[j], 1000 + j, nbytes=S, dtype=self.dt)
            e1.add(H.HPL_EV_BROADCAST, t, src_id, ids=dsts)
            if w.kind == "broadcast":
                offs = wl.uniform_offsets_ns(w.seed + r, R, w.extra["join_window_ns"])
                for j in sorted(range(R), key=lambda j: (offs[j], j)):
                    e1.add(H.HPL_EV_JOIN, t + offs[j], dsts[j], ptr=self.recv[j].data_ptr())
                t += w.extra["join_window_ns"]
            else:
                for j in range(R):
                    e1.add(H.HPL_EV_JOIN, t, dsts[j], ptr=self.recv[j].data_ptr())
            if early:
                # the Reduce of the objects the workers will return is requested with futures while the
                # broadcast is still running (the pattern of the paper's Fig. 1)
                e1.add(H.HPL_EV_PROGRESS)
                for i in ids:
                    e1.add(H.HPL_EV_CREATE, t, i, i, nbytes=S, dtype=self.dt)
                e1.add(H.HPL_EV_REDUCE, t, tgt, ids=ids, k=w.k, op=H.HPL_SUM, dtype=self.dt)
            for j in range(R):
                e1.add(H.HPL_EV_GET, 0, dsts[j])          # every receiver's Get
            t += 200_000_000                             # the Gets let virtual time run until the copies had landed
            dl.add(H.HPL_EV_DELETE, 0, src_id)
        if marks and w.kind == "round":                  # (a step with one part is timed from its first mark to its last)
            first.add(H.HPL_EV_MARK, 0, ptr=marks[1])
        if w.kind in ("reduce", "round", "ft_reduce"):
            if not early:
                for i in ids:
                    e2.add(H.HPL_EV_CREATE, t, i, i, nbytes=S, dtype=self.dt)
                e2.add(H.HPL_EV_REDUCE, t, tgt, ids=ids, k=w.k, op=H.HPL_SUM, dtype=self.dt)
            if w.kind == "reduce" and "mean_arrival_ns" in w.extra:
                arr = wl.exponential_arrivals_ns(w.seed + r, n, w.extra["mean_arrival_ns"])
            else:
                arr = [0] * n
            for i in sorted(ids, key=lambda i: (arr[i], i)):
                nbytes = S
                if w.kind == "ft_reduce" and i == w.extra["fail_worker"]:
                    nbytes = int(w.extra["fail_fraction"] * wl.n_chunks(S, w.chunk_bytes)) * w.chunk_bytes
                    if nbytes == 0:
                        continue
                if self.host_buffers:
                    e2.add(put_kind, t + arr[i], i, ptr=self.host_src[i % len(self.host_src)].data_ptr(), nbytes=nbytes)
                    h2d += nbytes
                else:
                    e2.add(put_kind, t + arr[i], i, ptr=self.src[i].data_ptr(), nbytes=nbytes)
            t += max(arr)
            if w.kind == "ft_reduce":
                if self.ft_eager:
                    e2.add(H.HPL_EV_PROGRESS)            # chunks delivered by every worker are reduced before the failure
                e2.add(H.HPL_EV_FAIL, t + 1, worker=w.extra["fail_worker"])
            if not self.host_buffers:
                e2.add(H.HPL_EV_GET, 0, tgt)
            for i in [tgt] + ids:
                dl.add(H.HPL_EV_DELETE, 0, i)
        if w.kind == "allreduce":
            # the allreduce of Section 3.4.3: a Reduce whose output is broadcast to the R participants.  Puts first,
            # then the requests (equal-time order), then every receiver's Get.
            dsts = [6000 + j for j in range(R)]
            for i in ids:
                e2.add(H.HPL_EV_CREATE, t, i, i, nbytes=S, dtype=self.dt)
                e2.add(H.HPL_EV_PUT, t, i, ptr=self.src[i].data_ptr(), nbytes=S)
            for j in range(R):
                e2.add(H.HPL_EV_CREATE, t, dsts[j], 1000 + j, nbytes=w.elems * 4, dtype=H.HPL_F32)
            e2.add(H.HPL_EV_REDUCE, t, tgt, ids=ids, k=w.k, op=H.HPL_SUM, dtype=self.dt)
            e2.add(H.HPL_EV_BROADCAST, t, tgt, ids=dsts)
            for j in range(R):
                e2.add(H.HPL_EV_JOIN, t, dsts[j], ptr=self.recv[j].data_ptr())
            for j in range(R):
                e2.add(H.HPL_EV_GET, 0, dsts[j])
            e2.add(H.HPL_EV_GET, 0, tgt)
            for i in [tgt] + ids:
                dl.add(H.HPL_EV_DELETE, 0, i)
        if marks:
            (e2 if len(e2) else e1).add(H.HPL_EV_MARK, 0, ptr=marks[2])
        return e1, e2, dl, h2d, d2h

    def prepare(self, n_rounds: int, marks=None):
        for i, r in enumerate(range(self.round, self.round + n_rounds)):
            self.prepared[r] = self.build_round(r, marks[i] if marks else None)

    # one pass of the whole path; returns (h2d bytes, d2h bytes) of the step
    def step(self):
        w, ctx = self.w, self.ctx
        if self.round not in self.prepared:
            self.prepare(1)
        e1, e2, dl, h2d, d2h = self.prepared.pop(self.round)
        S = w.object_bytes
        if len(e1):
            ctx.submit(e1)
            if self.host_buffers:
                ctx.get_host(6000 + w.n_receivers - 1, self.host_recv.data_ptr(), S)
                d2h += S
        self.mid_event()
        if len(e2):
            ctx.submit(e2)
            if self.host_buffers:
                ctx.get_host(9000, self.host_out.data_ptr(), w.elems * 4)
                d2h += w.elems * 4
        self.end_event()
        ctx.submit(dl)
        self.round += 1
        return h2d, d2h

    def mid_event(self):
        pass

    def end_event(self):
        pass


def time_steps(runner: Runner, steps: int, warmup: int, dist=None):
    torch = runner.torch
    runner.prepare(warmup)              # the timelines are inputs: built before the timed region
    for _ in range(warmup):
        runner.step()
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(steps)]
    cur = {"i": 0}
    if runner.host_buffers:
        # the end-to-end step leaves the library between its parts (hpl_get_host): events recorded from here
        runner.prepare(steps)
        runner.mid_event = lambda: ev[cur["i"]][1].record()
        runner.end_event = lambda: ev[cur["i"]][2].record()
    else:
        # device-resident step: the library records the events itself, inside hpl_submit (HPL_EV_MARK)
        for tri in ev:
            for e in tri:
                e.record()              # creates the underlying CUDA event
        torch.cuda.synchronize()
        runner.prepare(steps, [[e.cuda_event for e in tri] for tri in ev])
    st0 = runner.ctx.stats()
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    h2d = d2h = 0
    for i in range(steps):
        cur["i"] = i
        if runner.host_buffers:
            ev[i][0].record()
        a, b = runner.step()
        h2d, d2h = a, b
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    wall_ms = (time.perf_counter() - t0) * 1e3
    st1 = runner.ctx.stats()
    runner.mid_event = runner.end_event = lambda: None
    tot = [e[0].elapsed_time(e[2]) for e in ev]
    if runner.w.kind == "round" or runner.host_buffers:
        bc = [e[0].elapsed_time(e[1]) for e in ev]
        rd = [e[1].elapsed_time(e[2]) for e in ev]
    elif runner.w.kind == "broadcast":
        bc, rd = tot, [0.0] * len(tot)
    else:
        bc, rd = [0.0] * len(tot), tot
    delta = {k: st1[k] - st0[k] for k in st1}
    return {"bcast_ms": bc, "reduce_ms": rd, "total_ms": tot, "wall_ms": wall_ms, "stats": delta,
            "h2d": h2d, "d2h": d2h}


def max_over_ranks(values, dist, device):
    """Element-wise maximum of a list of floats over all ranks (identity without a process group)."""
    if dist is None:
        return [float(v) for v in values]
    import torch
    t = torch.tensor(list(values), device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def whole_job_value(step_bytes, steps, world, total_ms):
    """Aggregate throughput: every rank moved ``step_bytes * steps``; the job took the slowest rank's time."""
    return gbs(step_bytes * steps * world, total_ms)


def realtime_rounds(device, rounds: int = 8):
    """The asynchrony view of the paper's Fig. 8 on the async-SGD shape (cfg3): objects are put at their real
    arrival offsets (the host waits), every event lets the library run what has become runnable, and the
    figure is the time from the k-th arrival -- the last one the Reduce needs -- until the caller holds the
    result.  Early arrivals are reduced while the later ones are still on their way."""
    import torch
    import paper_2002_05814_b200 as hpl

    w = wl.workload("cfg3")
    S = w.object_bytes
    arena = torch.empty(64 * MiB + 10 * w.elems * 4, dtype=torch.uint8, device=device)
    out = {}
    for eager in (True, False):
        ctx = hpl.Context(w.chunk_bytes, w.degree, w.degree, arena=arena.data_ptr(), arena_bytes=arena.numel(),
                          stream=torch.cuda.current_stream().cuda_stream, eager=eager)
        src = [wl.values_torch(w.dist, w.seed + i, i, 0, w.elems, "f32", device=device) for i in range(w.n_objects)] if eager else src_keep
        src_keep = src
        torch.cuda.synchronize()
        lat, tail_bytes = [], []
        t_base = 0
        for r in range(rounds + 1):
            arr = wl.exponential_arrivals_ns(w.seed + r, w.n_objects, w.extra["mean_arrival_ns"])
            order = sorted(range(w.n_objects), key=lambda i: (arr[i], i))
            t_base += 1_000_000_000
            ctx.advance(t_base)
            ids = list(range(w.n_objects))
            ctx.create_batch(ids, ids, S)
            ctx.reduce(9000, ids, w.k)
            t0 = time.perf_counter_ns()
            b0 = 0
            for n, i in enumerate(order[:w.k]):            # the spares arrive later and are not needed
                while time.perf_counter_ns() - t0 < arr[i]:
                    pass
                ctx.advance(t_base + arr[i])
                if n == w.k - 1:
                    st = ctx.stats()
                    b0 = st["bytes_read_planned"] + st["bytes_written_planned"]
                    t_last = time.perf_counter_ns()
                ctx.put(i, src[i].data_ptr(), S)
            ctx.get(9000)
            t_done = time.perf_counter_ns()
            st = ctx.stats()
            if r > 0:                                      # the first round warms up
                lat.append((t_done - t_last) / 1e3)
                tail_bytes.append(st["bytes_read_planned"] + st["bytes_written_planned"] - b0)
            for i in [9000] + ids:
                ctx.delete(i)
        ctx.shutdown()
        out["eager" if eager else "lazy"] = {"latency_after_last_needed_arrival_us": float(np.mean(lat)),
                                             "std_us": float(np.std(lat)), "bytes_moved_in_that_tail": float(np.mean(tail_bytes)),
                                             "rounds": rounds}
    # the same view for the broadcast shape (cfg2): receivers join at their real offsets; each join starts the
    # copy for that receiver (from its sender's copy once that is complete); the figure is the time from the
    # last join until every receiver holds the object
    w2 = wl.workload("cfg2")
    S2 = w2.object_bytes
    ctx = hpl.Context(w2.chunk_bytes, w2.degree, w2.degree, arena=arena.data_ptr(), arena_bytes=arena.numel(),
                      stream=torch.cuda.current_stream().cuda_stream, eager=True)
    srcb = wl.values_torch(w2.dist, w2.seed, 0, 0, w2.elems, "f32", device=device)
    recv = [torch.empty(w2.elems, dtype=torch.float32, device=device) for _ in range(w2.n_receivers)]
    torch.cuda.synchronize()
    lat = []
    t_base = 0
    for r in range(rounds + 1):
        offs = wl.uniform_offsets_ns(w2.seed + r, w2.n_receivers, w2.extra["join_window_ns"])
        order = sorted(range(w2.n_receivers), key=lambda j: (offs[j], j))
        t_base += 1_000_000_000
        ctx.advance(t_base)
        ids = [100 + j for j in range(w2.n_receivers)]
        ctx.create(0, 99, S2)
        ctx.put(0, srcb.data_ptr(), S2)
        ctx.create_batch(ids, ids, S2)
        ctx.broadcast(0, ids)
        t0 = time.perf_counter_ns()
        for j in order:
            while time.perf_counter_ns() - t0 < offs[j]:
                pass
            ctx.advance(t_base + offs[j])
            ctx.join(ids[j], recv[j].data_ptr())
        t_last = time.perf_counter_ns()
        ctx.get_batch(ids)
        if r > 0:
            lat.append((time.perf_counter_ns() - t_last) / 1e3)
        ctx.delete(0)
    ctx.shutdown()
    out["broadcast_cfg2"] = {"latency_after_last_join_us": float(np.mean(lat)), "std_us": float(np.std(lat)), "rounds": rounds,
                             "note": "joins at real offsets over 1 ms, every join starts that receiver's copy"}
    out["note"] = ("eager: every Put also runs what became runnable (arrived operands are merged into their parents' partial "
                   "results); lazy: everything is planned at the Get, one fused pass over the 8 members")
    return out


def gbs(nbytes, ms):
    return nbytes / (ms * 1e-3) / 1e9 if ms > 0 else 0.0


# ----------------------------------------------------------------------------------------- oracle arm
def oracle_sample(w: wl.Workload, budget_s: float = 12.0, window: int = 0, raw: bool = False):
    """Times the oracle, as it stands, on a bounded sample of the workload: the same objects cut to a
    window of their elements (same chunk size, same tree, same timeline).  Returns GB/s on the
    algorithmic bytes of the sample.  ``window`` picks which 1/16 of the elements (0 = the first)."""
    from oracle.store import OracleStore, DT_F32, DT_BF16

    frac = 16
    elems = max(4096, (w.elems // frac) // 8 * 8)
    dt = DT_BF16 if w.dtype == "bf16" else DT_F32
    start = (window % frac) * elems if (window % frac + 1) * elems <= w.elems else 0
    distinct = [wl.values_np(w.dist, w.seed + i, i, start, elems, w.dtype) for i in range(min(8, max(1, w.n_objects)))]
    S = distinct[0].nbytes
    sw = wl.Workload(**{**w.__dict__, "elems": elems})
    ab = algorithmic_bytes(sw)
    total_bytes = ab["reduce"] + ab["broadcast"]
    reps, t_total = 0, 0.0
    while t_total < budget_s and reps < 200:
        o = OracleStore(w.chunk_bytes, w.degree, w.degree)
        t0 = time.perf_counter()
        if w.kind in ("broadcast", "round"):
            o.create(5000, 900, S, dt)
            o.put(5000, distinct[0], S)
            dsts = [6000 + j for j in range(w.n_receivers)]
            for j, dd in enumerate(dsts):
                o.create(dd, 1000 + j, S, dt)
            o.broadcast(5000, dsts)
            offs = wl.uniform_offsets_ns(w.seed + reps, w.n_receivers, w.extra.get("join_window_ns", 1))
            for j in sorted(range(w.n_receivers), key=lambda j: (offs[j], j)):
                o.advance(max(o.now, offs[j] if w.kind == "broadcast" else 0))
                o.join(dsts[j])
            for dd in dsts:
                o.get(dd)
        if w.kind in ("reduce", "round", "ft_reduce"):
            n = w.n_objects
            for i in range(n):
                o.create(i, i, S, dt)
            arr = wl.exponential_arrivals_ns(w.seed + reps, n, w.extra["mean_arrival_ns"]) if "mean_arrival_ns" in w.extra else [0] * n
            o.reduce(9000, list(range(n)), w.k, 0, dt)
            base = o.now
            for i in sorted(range(n), key=lambda i: (arr[i], i)):
                o.advance(max(o.now, base + arr[i]))
                nbytes = S
                if w.kind == "ft_reduce" and i == w.extra["fail_worker"]:
                    nbytes = int(w.extra["fail_fraction"] * wl.n_chunks(S, w.chunk_bytes)) * w.chunk_bytes
                    if nbytes == 0:
                        continue
                o.put(i, distinct[i % len(distinct)], nbytes)
            if w.kind == "ft_reduce":
                o.fail(w.extra["fail_worker"])
            o.get(9000)
        t_total += time.perf_counter() - t0
        reps += 1
    if raw:
        return total_bytes * reps, t_total, elems
    value = total_bytes * reps / t_total / 1e9
    sample = (f"{reps} pass(es) of the oracle over the first {elems} of {w.elems} elements of every object "
              f"({total_bytes * reps / 1e9:.2f} GB algorithmic, {t_total:.1f} s, numpy single thread)")
    return value, sample, t_total / reps * 1e3


def _oracle_worker(args):
    w, budget_s, window = args
    return oracle_sample(w, budget_s, window, raw=True)


def oracle_all_cores(w: wl.Workload, budget_s: float = 8.0):
    """The same oracle passes on every core the process may use: one process per core (started with `spawn`), each
    over its own window of the elements.  Throughput = bytes of all processes / the slowest one's time."""
    import multiprocessing as mp
    cores = len(os.sched_getaffinity(0))
    with mp.get_context("spawn").Pool(cores) as pool:
        out = pool.map(_oracle_worker, [(w, budget_s, i) for i in range(cores)])
    nbytes = sum(o[0] for o in out)
    t = max(o[1] for o in out)
    sample = (f"{cores} processes, each the oracle's passes over its own window of {out[0][2]} of {w.elems} elements of every "
              f"object ({nbytes / 1e9:.2f} GB algorithmic in all, slowest process {t:.1f} s, numpy, one thread each)")
    return nbytes / t / 1e9, cores, sample


# ----------------------------------------------------------------------------------------- measured points
def measure_point(rr: "Runner", steps: int, warmup: int, peak: float, k_steps: int = 0):
    """Step throughput of the runner's workload (event timing off) and, from a pass of its own with event timing on,
    the kernels' figures."""
    ab = algorithmic_bytes(rr.w)
    b = ab["reduce"] + ab["broadcast"]
    rr.open_context(time_kernels=False)
    r = time_steps(rr, steps, warmup)
    g = gbs(b * steps, float(np.sum(r["total_ms"])))
    k_steps = k_steps or min(steps, 10)
    rr.open_context(time_kernels=True)
    s2 = time_steps(rr, k_steps, 1)["stats"]
    kns = s2["reduce_kernel_ns"] + s2["fanout_kernel_ns"]
    planned = s2["bytes_read_planned"] + s2["bytes_written_planned"]
    kern = gbs(planned, kns / 1e6)       # bytes the planned tasks move / their summed launch time
    return {"GBps": g, "frac_of_measured_copy": g / peak, "ms_per_step": float(np.mean(r["total_ms"])),
            "ms_std": float(np.std(r["total_ms"])), "steps": steps, "kernel_GBps": kern,
            "kernel_frac_of_measured_copy": kern / peak, "kernel_ms_per_step": kns / 1e6 / k_steps,
            "launches_per_step": s2["kernel_launches"] / k_steps, "planned_over_algorithmic_bytes": planned / (b * k_steps)}


def size_sweep(device, peak: float):
    """The metric's curve: effective GB/s and fraction of the HBM peak against object size, 1 KiB ... 1 GiB in powers
    of 4, for the fault-tolerant reduce of 32 objects (the compressed timeline planned at the Get, and with the chunks
    delivered before the failure reduced first) and for a broadcast to 16 receivers."""
    import torch
    rows = []
    for size in wl.workload("cfg5").extra["sizes_bytes"]:
        n = 20 if size <= (16 << 20) else (5 if size <= (256 << 20) else 3)
        row = {"object_bytes": size}
        rr = Runner(wl.cfg5_at(size), device)
        for mode in ("lazy", "eager"):
            rr.ft_eager = mode == "eager"
            m = measure_point(rr, n, 3, peak, k_steps=min(n, 5))
            row[f"reduce_{mode}"] = {k: m[k] for k in ("GBps", "frac_of_measured_copy", "ms_per_step", "kernel_ms_per_step",
                                                         "planned_over_algorithmic_bytes", "launches_per_step")}
        rr.close()
        del rr
        torch.cuda.empty_cache()
        if size <= (64 << 10):
            # small objects: 32 Reduces of 8 objects each requested together (shared waves, one wait)
            mw = wl.Workload("reduce_x32", "multi_reduce", "f32", ("uniform",), size // 4, size, 2, n_objects=8, k=8,
                             extra={"collectives": 32})
            rr = Runner(mw, device)
            m = measure_point(rr, n, 3, peak, k_steps=min(n, 5))
            row["reduce_8_objects_x32_together"] = {"GBps": m["GBps"], "ms_per_step": m["ms_per_step"],
                                                    "us_per_collective": m["ms_per_step"] * 1e3 / 32,
                                                    "launches_per_step": m["launches_per_step"]}
            rr.close()
            del rr
            torch.cuda.empty_cache()
        bw = wl.Workload("bcast16", "broadcast", "f32", ("uniform",), size // 4, min(1 << 20, size), 2, n_receivers=16,
                         extra={"join_window_ns": 1_000_000})
        rr = Runner(bw, device)
        m = measure_point(rr, n, 3, peak, k_steps=min(n, 5))
        row["broadcast16"] = {k: m[k] for k in ("GBps", "frac_of_measured_copy", "ms_per_step", "kernel_ms_per_step")}
        rr.close()
        del rr
        torch.cuda.empty_cache()
        rows.append(row)
    return rows


def worker_per_gpu_round(dist, device, rank: int, world: int, steps: int = 5, object_bytes: int = 64 * MiB):
    """The paper's own setting on N GPUs of one node: worker = rank, one 64 MiB fp32 object per GPU, a Reduce of all of
    them through a binary tree whose edges cross NVLink (every node's result materialised on its own GPU, remote
    operands pulled from peer memory; levels separated by a barrier).  Reported beside the replicas headline; every
    rank takes part in every collective step even after a local error, so a refused peer mapping ends the round with a
    message instead of a hang."""
    import torch
    import paper_2002_05814_b200 as hpl

    state = {"ok": True, "err": ""}

    def fail(e):
        state["ok"] = False
        state["err"] = state["err"] or repr(e)

    # (with the gloo backend -- ranks that share one GPU in a test -- collectives take host tensors)
    coll_device = device if dist.get_backend() == "nccl" else torch.device("cpu")

    def agree():
        """All ranks learn whether all are still fine (doubles as the barrier between levels)."""
        t = torch.tensor([1 if state["ok"] else 0], device=coll_device, dtype=torch.int32)
        dist.all_reduce(t, op=dist.ReduceOp.MIN)
        return bool(t.item())

    S = object_bytes
    arena_bytes = 64 * MiB + 4 * S
    ctx, mapped = None, []
    out = {"objects": world, "object_bytes": S, "degree": 2}
    try:
        arena = torch.empty(arena_bytes, dtype=torch.uint8, device=device)
        obj = wl.values_torch(("uniform",), wl.BASE_SEED + rank, rank, 0, S // 4, "f32", device=device)
        mine = (hpl.ipc_export(arena.data_ptr()), hpl.ipc_export(obj.data_ptr()))
    except Exception as e:      # noqa: BLE001
        fail(e)
        mine = None
    handles = [None] * world
    dist.all_gather_object(handles, mine)
    peer_arena, peer_obj = {}, {}
    if agree():
        try:
            for r in range(world):
                if r == rank:
                    peer_arena[r], peer_obj[r] = arena.data_ptr(), obj.data_ptr()
                else:
                    (ha, oa), (ho, oo) = handles[r]
                    peer_arena[r] = hpl.ipc_import(ha, oa)
                    peer_obj[r] = hpl.ipc_import(ho, oo)
                    mapped += [peer_arena[r], peer_obj[r]]
            ctx = hpl.Context(4 * MiB, 2, 2, arena=arena.data_ptr(), arena_bytes=arena_bytes,
                              stream=torch.cuda.current_stream().cuda_stream, fuse=False, rank=rank, world_size=world)
            for r in range(world):
                if r != rank:
                    ctx.set_peer_arena(r, peer_arena[r])
        except Exception as e:  # noqa: BLE001
            fail(e)
    times = []
    if agree():
        t = 0
        for step in range(steps + 2):
            dist.barrier()
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            try:
                t += 1_000_000_000
                ctx.advance(t)
                ids = list(range(world))
                ctx.create_batch(ids, ids, S)
                ctx.put_batch(ids, [peer_obj[r] for r in ids], S)
                ctx.reduce(1000, ids, world)
            except Exception as e:  # noqa: BLE001
                fail(e)
            while True:                       # Context.drive, with `agree` as the barrier and a way out after an error
                n = 0
                try:
                    if state["ok"]:
                        ctx.progress()
                        n = ctx.pending_levels()
                except Exception as e:  # noqa: BLE001
                    fail(e)
                if not agree() or n == 0:
                    break
                for _ in range(n):
                    try:
                        if state["ok"]:
                            ctx.run_level()
                            ctx.sync()
                    except Exception as e:  # noqa: BLE001
                        fail(e)
                    if not agree():
                        break
                if not state["ok"]:
                    break
            if not agree():
                break
            torch.cuda.synchronize()
            dt = (time.perf_counter() - t0) * 1e3
            if step >= 2:
                times.append(max_over_ranks([dt], dist, coll_device)[0])
            try:
                ctx.get(1000)
                for i in [1000] + ids:
                    ctx.delete(i)
            except Exception as e:  # noqa: BLE001
                fail(e)
    agree()
    try:
        if ctx is not None:
            ctx.shutdown()
        dist.barrier()
        for p in mapped:
            hpl.ipc_close(p)
    except Exception as e:      # noqa: BLE001
        fail(e)
    errs = [None] * world
    dist.all_gather_object(errs, state["err"])
    if any(errs):
        out["error"] = next(e for e in errs if e)
    if times:
        ms = float(np.mean(times))
        out.update({"ms_per_reduce": ms, "GBps_algorithmic": gbs((world + 1) * S, ms),
                    "how": "wall clock from the Puts to the last level's barrier, maximum over ranks; levels = tree height, "
                           "one NCCL all-reduce of a flag between levels"})
    return out


def degree_sweep(device, peak: float):
    """Section 3.4.2 / Appendix B on one GPU: reduce time against the tree degree d in {1, 2, k}, for k in {8, 32} objects
    of several sizes, (a) as the paper executes a tree -- every node writes its reduced object, one wave per tree level
    (fuse = 0) -- and (b) with ready subtrees fused in registers (fuse = 1, where the degree only changes the
    association order).  L and B of Eq. 1 are calibrated from the measurements themselves: L = time per tree level
    (chain against star on the smallest objects), B = bytes per second of the largest fused pass; the degree Eq. 1
    picks from them (reduce_degree = 0) is then run and compared with the best measured one."""
    import torch
    import paper_2002_05814_b200 as hpl
    sizes = [64 << 10, 1 << 20, 16 << 20, 64 << 20]
    rows, cal = [], {}
    for k in (8, 32):
        for size in sizes:
            w = wl.Workload("degree", "reduce", "f32", ("uniform",), size // 4, min(4 * MiB, size), 2, n_objects=k, k=k,
                            extra={"partials": k})
            rr = Runner(w, device)
            n = 20 if size <= (1 << 20) else 6
            cell = {"k": k, "object_bytes": size}
            for fuse in (0, 1):
                for d in (1, 2, k):
                    w.degree = d
                    rr.ctx_flags = {"fuse": bool(fuse)}
                    rr.open_context(time_kernels=False)
                    r = time_steps(rr, n, 3)
                    cell[f"fuse{fuse}_d{d}_ms"] = float(np.mean(r["total_ms"]))
            rows.append((cell, rr, w, n))
    # calibration: per-level latency from the smallest objects (k = 32: the chain has 31 levels, the star one), bandwidth
    # from the largest fused pass
    small = next(c for c, _, _, _ in rows if c["k"] == 32 and c["object_bytes"] == sizes[0])
    big = next(c for c, _, _, _ in rows if c["k"] == 32 and c["object_bytes"] == sizes[-1])
    L = max(1e-7, (small["fuse0_d1_ms"] - small["fuse0_d32_ms"]) * 1e-3 / 30.0)
    B = (33 * sizes[-1]) / (big["fuse1_d2_ms"] * 1e-3)
    out = []
    for cell, rr, w, n in rows:
        k, size = cell["k"], cell["object_bytes"]
        w.degree = 0
        rr.ctx_flags = {"fuse": False, "model_latency_ns": max(1, int(L * 1e9)), "model_bandwidth_bps": int(B)}
        rr.open_context(time_kernels=False)
        r = time_steps(rr, n, 3)
        chosen = hpl.choose_degree(k, size, L, B)
        best0 = min((1, 2, k), key=lambda d: cell[f"fuse0_d{d}_ms"])
        cell.update({"eq1_degree": chosen, "eq1_degree_ms_fuse0": float(np.mean(r["total_ms"])), "best_degree_fuse0": best0,
                     "best_ms_fuse0": cell[f"fuse0_d{best0}_ms"],
                     "fuse1_spread": max(cell[f"fuse1_d{d}_ms"] for d in (1, 2, k)) / min(cell[f"fuse1_d{d}_ms"] for d in (1, 2, k))})
        out.append(cell)
        rr.close()
    del rows
    torch.cuda.empty_cache()
    return {"L_s_per_level": L, "B_bytes_per_s": B, "cells": out,
            "note": ("Eq. 1 models nodes with links of their own: a larger d costs d S / B at one node while the others work in "
                     "parallel.  On one GPU every node shares the same HBM: a tree that writes every partial result moves "
                     "(k + 2 (I - 1) + 1) S bytes for I internal nodes, so the star (d = k) is best whenever it fits, and the "
                     "fused path makes the degree irrelevant (fuse1_spread is about 1).")}


# ----------------------------------------------------------------------------------------- main
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg4")
    ap.add_argument("--size", type=int, default=64 * MiB, help="object bytes for cfg5")
    ap.add_argument("--shrink", type=int, default=1, help="divide the object size by this (profiling captures on a smaller case)")
    ap.add_argument("--ft-mode", default="eager", choices=["eager", "lazy"],
                    help="cfg5: 'eager' runs hpl_progress before the failure (chunks delivered by every worker are reduced, "
                         "then partly redone); 'lazy' applies the compressed timeline and plans at the Get")
    ap.add_argument("--no-realtime", action="store_true", help="skip the view with puts / joins at their real offsets (cfg3, cfg2)")
    ap.add_argument("--no-sweep", action="store_true",
                    help="skip GB/s against object size: the fault-tolerant reduce (32 objects, both modes) and a "
                         "broadcast to 16 receivers, for 1 KiB ... 1 GiB in powers of 4")
    ap.add_argument("--worker-per-gpu", action="store_true",
                    help="with --gpus N > 1: also run a Reduce whose objects live one per GPU and whose tree edges cross NVLink "
                         "(peer memory through CUDA IPC); off by default: this path has never run on more than one GPU")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--also", default="cfg2,cfg3", help="extra workloads reported under 'also' (cfg3 for its 50 rounds); 'none' skips them")
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if args.workload == "allreduce":     # reduce followed by broadcast, 8 x 64 MiB fp32 to 8 receivers (Section 5.1's allreduce shape)
        w = wl.Workload("allreduce", "allreduce", "f32", ("uniform",), 16 * MiB, 4 * MiB, 2, n_objects=8, k=8, n_receivers=8)
    else:
        w = wl.cfg5_at(args.size) if args.workload == "cfg5" else wl.workload(args.workload)
    if args.shrink > 1:
        w.elems = max(8, w.elems // args.shrink // 8 * 8)
    ab = algorithmic_bytes(w)
    step_bytes = ab["reduce"] + ab["broadcast"]
    name = {"cfg1": "cfg1 reduce 8 x 1 MiB fp32", "cfg2": "cfg2 broadcast 64 MiB fp32 to 16 receivers",
            "cfg3": "cfg3 async-SGD reduce, first 8 of 16 x 97.5 MiB fp32",
            "cfg4": "cfg4 policy round: broadcast 64 MiB bf16 to 64 receivers + fp32 sum of 64 x 64 MiB bf16",
            "cfg5": f"cfg5 fault-tolerant reduce of 32 x {args.size} B fp32, worker 7 fails at 40%",
            "allreduce": "allreduce: fp32 sum of 8 x 64 MiB broadcast to 8 receivers, fused into one pass"}[w.name]
    if args.shrink > 1:
        name += f" [objects shrunk {args.shrink}x]"
    config = {"workload": name, "chunk_bytes": w.chunk_bytes, "degree": w.degree, "object_bytes": w.object_bytes,
              "algorithmic_bytes_per_step": step_bytes, "l2": "inputs larger than L2 (no flush)",
              "timed_region": "first Put of the step to the last Get, CUDA events on the library's stream; Delete outside"}

    if args.impl == "reference":
        if rank != 0:
            return
        value, sample, ms = oracle_sample(w, budget_s=min(60.0, max(5.0, 4.0 * (args.steps + args.warmup))))
        line = {"impl": "reference", "metric": METRIC, "value": value,
                "unit": "GB/s", "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms,
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                "config": config, "cpu_baseline": {"value": value, "unit": "GB/s", "cores": 1, "kind": "oracle", "sample": sample},
                "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
        print(json.dumps(line))
        return

    import torch
    from paper_2002_05814_b200 import build as hpl_build

    if rank == 0 or world == 1:
        hpl_build.build()
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        torch.cuda.set_device(local)
        dist_mod.init_process_group("nccl", device_id=torch.device("cuda", local))
        dist = dist_mod
        dist.barrier()
    else:
        torch.cuda.set_device(local)
    device = torch.device("cuda", local)

    sampler = ClockSampler(local)
    runner = Runner(w, device, ft_eager=args.ft_mode == "eager")
    sampler.start()
    res = time_steps(runner, args.steps, args.warmup, dist)
    clocks = sampler.stop()
    # per-launch device times for the roofline come from a short pass of their own, with event timing switched on
    k_steps = max(1, min(args.steps, 10))
    runner.open_context(time_kernels=True)
    res_k = time_steps(runner, k_steps, 3)
    runner.close()
    del runner
    torch.cuda.empty_cache()

    total_ms, wall_ms = max_over_ranks([float(np.sum(res["total_ms"])), res["wall_ms"]], dist, device)
    value = whole_job_value(step_bytes, args.steps, world, total_ms)
    peak, peak_kind = measured_peak()
    st = res_k["stats"]

    def roof(kind_ns, kind_launches, per_launch_bytes, traffic=None):
        if st[kind_launches] == 0:
            return None
        avg_ms = st[kind_ns] / st[kind_launches] / 1e6
        ach = gbs(per_launch_bytes, avg_ms)
        return {"bound": "hbm", "achieved": ach, "peak": peak, "unit": "GB/s", "frac": ach / peak, "traffic": traffic,
                "peak_kind": f"of {peak_kind} (copy bandwidth)", "avg_launch_ms": avg_ms, "launches": st[kind_launches],
                "algorithmic_bytes_per_launch": per_launch_bytes, "frac_of_8TBs_nominal": ach / 8000.0}

    traf = {k: ncu_traffic(w.name, k) for k in ("reduce", "fanout")} if args.shrink == 1 else {}
    r_red = roof("reduce_kernel_ns", "reduce_launches", ab["reduce"] * k_steps / max(1, st["reduce_launches"]), traf.get("reduce")) if ab["reduce"] else None
    r_fan = roof("fanout_kernel_ns", "fanout_launches", ab["broadcast"] * k_steps / max(1, st["fanout_launches"]), traf.get("fanout")) if ab["broadcast"] else None
    line = {"metric": METRIC, "value": value, "unit": "GB/s",
            "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": total_ms / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32" if w.dtype == "f32" else "f32 (bf16 inputs widened)", "data": "synthetic",
            "config": config, "clocks": clocks, "gpu_launches": int(res["stats"]["kernel_launches"]),
            "wall_ms_per_step": wall_ms / args.steps,
            "frac_of_hbm_peak": {"measured_copy": value / world / peak, "nominal_8TBs": value / world / 8000.0},
            "roofline": r_red if r_red is not None else r_fan}
    if r_red is not None and r_fan is not None:
        line["roofline_fanout"] = r_fan
    planned = (st["bytes_read_planned"] + st["bytes_written_planned"]) / k_steps
    kern_ms = (st["reduce_kernel_ns"] + st["fanout_kernel_ns"]) / 1e6 / k_steps
    line["planned_traffic"] = {"bytes_per_step": planned, "over_algorithmic": planned / step_bytes,
                               "kernel_GBps_on_planned_bytes": gbs(planned, kern_ms), "kernel_ms_per_step": kern_ms}
    if w.kind == "ft_reduce":
        line["config"]["ft_mode"] = args.ft_mode
    if ab["reduce"]:
        line["reduce"] = {"GBps": gbs(ab["reduce"] * args.steps, float(np.sum(res["reduce_ms"]))), "ms": float(np.mean(res["reduce_ms"])),
                          "ms_std": float(np.std(res["reduce_ms"]))}
    if ab["broadcast"]:
        line["broadcast"] = {"GBps": gbs(ab["broadcast"] * args.steps, float(np.sum(res["bcast_ms"]))), "ms": float(np.mean(res["bcast_ms"])),
                             "ms_std": float(np.std(res["bcast_ms"]))}

    if rank == 0 and world == 1 and args.also and args.also != "none":
        also = {}
        for nm in [x for x in args.also.split(",") if x and x != "none" and x != w.name]:
            ww = wl.workload(nm)
            rr = Runner(ww, device)
            also[nm] = measure_point(rr, ww.rounds if ww.rounds > 1 else 30, 5, peak)
            rr.close()
            del rr
            torch.cuda.empty_cache()
        # reduce followed by broadcast (the allreduce microbenchmark of Section 5.1): 8 x 64 MiB fp32 to 8 receivers, with
        # the result tile fanned out from the reduce pass and, for comparison, with the broadcast reading the target
        aw = wl.Workload("allreduce", "allreduce", "f32", ("uniform",), 16 * MiB, 4 * MiB, 2, n_objects=8, k=8, n_receivers=8)
        for label, fused in (("allreduce_8x64MiB_fused", True), ("allreduce_8x64MiB_two_waves", False)):
            rr = Runner(aw, device, fuse_fanout=fused)
            also[label] = measure_point(rr, 20, 5, peak)
            rr.close()
            del rr
            torch.cuda.empty_cache()
        line["also"] = also

    if rank == 0 and world == 1 and not args.no_sweep and args.shrink == 1:
        rows = size_sweep(device, peak)
        line["sweep"] = rows
        big = [r for r in rows if r["object_bytes"] >= (64 << 20)]
        line["sweep_summary"] = {
            "min_frac_reduce_at_64MiB_and_above": min(r["reduce_lazy"]["frac_of_measured_copy"] for r in big),
            "min_frac_broadcast_at_64MiB_and_above": min(r["broadcast16"]["frac_of_measured_copy"] for r in big),
            "max_ms_per_step_up_to_4MiB": max(max(r["reduce_lazy"]["ms_per_step"], r["broadcast16"]["ms_per_step"])
                                              for r in rows if r["object_bytes"] <= (4 << 20)),
            "of": "measured copy bandwidth; reduce = fault-tolerant reduce of 32 objects planned at the Get"}

    if rank == 0 and world == 1 and not args.no_sweep and args.shrink == 1:
        line["degree_sweep"] = degree_sweep(device, peak)

    if rank == 0 and world == 1 and not args.no_realtime and args.shrink == 1:
        line["realtime"] = realtime_rounds(device)

    if world > 1 and args.worker_per_gpu:
        try:
            line["worker_per_gpu"] = worker_per_gpu_round(dist, device, rank, world)
        except Exception as e:  # noqa: BLE001
            line["worker_per_gpu"] = {"error": repr(e)}

    if not args.no_e2e:
        e_steps = max(1, min(args.steps, 3))
        rr = Runner(w, device, host_buffers=True, plan_ahead=True)
        r3 = time_steps(rr, e_steps, 1, dist)
        rr.close()
        del rr
        torch.cuda.empty_cache()
        e_ms = max_over_ranks([float(np.sum(r3["total_ms"]))], dist, device)[0]
        line["e2e"] = {"value": whole_job_value(step_bytes, e_steps, world, e_ms), "unit": "GB/s", "h2d_bytes_per_step": int(r3["h2d"]),
                       "d2h_bytes_per_step": int(r3["d2h"]), "ms_per_step": e_ms / e_steps,
                       "how": "hpl_put_host from pinned host memory, chunks consumed by polling kernels as they land; hpl_get_host of the result"}

    if rank == 0 and world == 1 and not args.no_cpu:
        v, sample, _ = oracle_sample(w)
        va, cores, sample_all = oracle_all_cores(w)
        line["cpu_baseline"] = {"value": va, "unit": "GB/s", "cores": cores, "kind": "oracle", "sample": sample_all}
        line["cpu_baseline_one_core"] = {"value": v, "unit": "GB/s", "cores": 1, "kind": "oracle", "sample": sample}

    if rank == 0:
        print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
