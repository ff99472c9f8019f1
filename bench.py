#!/usr/bin/env python
"""Benchmark of the TopKV data plane on B200.

A "step" is one pass of the hot path over one synthetic batch: the plan (prefix sums), then
pack of every layer, then unpack of every layer, device to device. The headline workload is
the largest single-GPU configuration: the Llama-3-70B-shaped cache (8 requests of 4096
tokens, 80 layers, 10 GiB of wire). The same JSON line also carries the host-leg (PCIe) figure
as ``e2e`` (all 80 layers through pinned host memory), the live roofline of the pack kernel,
the CPU oracle timed on this machine as ``cpu_baseline``, and, at one GPU, the other benchmark
shapes (8B GQA, DeepSeek-V3 MLA), the side-stream overlap runs and the checksummed copy under
``extra``.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--extras ...]

With N > 1 (launched by torchrun) every rank runs its own batch (weak scaling, no data-path
collective); the time is the max over ranks, the value the sum of bytes over that time.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "kv_pack_unpack_GBps"
UNIT = "GB/s"
FALLBACK_HBM_GBS = 6650.0

# DRAM traffic of one pack launch relative to its algorithmic bytes comes from an ncu capture
# of this kernel at the same per-launch size, summarised under profiles/: the summary carries
# a line "traffic_ratio = <(dram__bytes_read.sum + dram__bytes_write.sum) / (2*N_layer)>" and
# the date and command of the capture, which are stamped into the bench line beside the number.
TRAFFIC_PROFILE = os.path.join("profiles", "page_copy_kernel_pack_cfg3_4layers.md")


def ncu_traffic(bytes_per_launch):
    """(traffic bytes per launch or None, where the figure comes from)."""
    import re
    path = os.path.join(ROOT, TRAFFIC_PROFILE)
    try:
        text = open(path).read()
        ratio = float(re.search(r"^traffic_ratio\s*=\s*([0-9.]+)", text, re.M).group(1))
        when = re.search(r"^captured\s*=\s*(\S+)", text, re.M)
        src = f"{TRAFFIC_PROFILE} (ncu capture of {when.group(1) if when else 'unknown date'}, " \
              f"ratio {ratio} x algorithmic bytes; not re-measured in this run)"
        return int(ratio * bytes_per_launch), src
    except Exception:
        return None, f"{TRAFFIC_PROFILE} not found or without a traffic_ratio line"


def measured_peak_gbs():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (6650 GB/s, earlier measurement on this pool)"


class ClockSampler:
    """Samples the SM clock and the throttle reasons while the timed region runs: NVML from a
    thread (a read-only query every ~2 ms), or nvidia-smi if NVML cannot be loaded."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, index: int):
        self.index, self.sm, self.reasons, self.max_mhz = index, [], set(), None
        self.proc = self.thread = self.nvml = None
        self.stop_flag = threading.Event()

    def start(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            visible = os.environ.get("CUDA_VISIBLE_DEVICES")
            idx = self.index
            if visible and all(x.strip().isdigit() for x in visible.split(",")):
                idx = int(visible.split(",")[self.index])
            self.handle = pynvml.nvmlDeviceGetHandleByIndex(idx)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self.handle, pynvml.NVML_CLOCK_SM))
            self.nvml = pynvml
            self.thread = threading.Thread(target=self._poll_nvml, daemon=True)
            self.thread.start()
            return
        except Exception:
            self.nvml = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-i", str(self.index), "-lms", "50"], stdout=subprocess.PIPE, text=True)
            self.thread = threading.Thread(target=self._read_smi, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _poll_nvml(self):
        n = self.nvml
        masks = {"hw_slowdown": n.nvmlClocksThrottleReasonHwSlowdown,
                 "hw_thermal_slowdown": n.nvmlClocksThrottleReasonHwThermalSlowdown,
                 "sw_thermal_slowdown": n.nvmlClocksThrottleReasonSwThermalSlowdown,
                 "sw_power_cap": n.nvmlClocksThrottleReasonSwPowerCap}
        while not self.stop_flag.is_set():
            try:
                self.sm.append(float(n.nvmlDeviceGetClockInfo(self.handle, n.NVML_CLOCK_SM)))
                r = n.nvmlDeviceGetCurrentClocksThrottleReasons(self.handle)
                for name, m in masks.items():
                    if r & m:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.002)

    def _read_smi(self):
        for line in self.proc.stdout:
            r = [x.strip() for x in line.split(",")]
            try:
                self.sm.append(float(r[0]))
                self.max_mhz = float(r[1])
                for name, v in zip(self.NAMES, r[2:6]):
                    if v.lower().startswith("active"):
                        self.reasons.add(name)
            except Exception:
                pass

    def stop(self):
        if self.nvml is None and self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["clock query unavailable"]}
        if self.nvml is not None:
            self.stop_flag.set()
            self.thread.join(timeout=2)
            src = "nvml"
        else:
            time.sleep(0.15)
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()
            self.thread.join(timeout=2)
            src = "nvidia-smi"
        return {"sm_mhz": statistics.median(self.sm) if self.sm else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.sm), "source": src}


def host_cores():
    return len(os.sched_getaffinity(0))


def oracle_sample(spec, batch, seconds_target=12.0, threads=None, impl="rows"):
    """Times the CPU oracle (row-memcpy form on all cores unless told otherwise) on whole layers
    of this workload until about ``seconds_target`` of wall time has passed. Returns
    (GB/s, layers timed, threads, seconds)."""
    import numpy as np
    import oracle
    from paper_2607_28633_b200 import workloads as wl
    cores = host_cores() if threads is None else threads
    cores = max(1, min(cores, spec.R))   # the rows form splits by request: the threads it really uses
    g = oracle.Geom(L=1, F=spec.F, h_kv=spec.H, d_h=spec.D, b_p=spec.E, P=spec.P,
                    num_pages=batch.num_pool_pages)
    src = wl.fill_numpy(g.pool_bytes(), batch.seeds["data"], raw_bits=True)
    dst = np.zeros_like(src)
    n_layer = g.wire_layer_bytes(batch.total_tokens)
    wire = np.zeros(n_layer, dtype=np.uint8)
    oracle.pack(g, 0, src, batch.src_block_table, batch.seq_lens, wire=wire, impl="rows",
                threads=cores)  # touch every page once (first-touch faults are not the oracle)
    oracle.unpack(g, 0, dst, batch.dst_block_table, batch.seq_lens, wire, impl="rows", threads=cores)
    t0, n = time.perf_counter(), 0
    while True:
        oracle.pack(g, 0, src, batch.src_block_table, batch.seq_lens, wire=wire, impl=impl,
                    threads=cores)
        oracle.unpack(g, 0, dst, batch.dst_block_table, batch.seq_lens, wire, impl=impl,
                      threads=cores)
        n += 1
        dt = time.perf_counter() - t0
        if dt >= seconds_target:
            break
    return 4.0 * n_layer * n / dt / 1e9, n, cores, dt


def run_reference(args):
    """The reference arm: the CPU oracle as it stands, on this machine's host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2607_28633_b200 import workloads as wl
    spec = HEADLINE(wl)
    batch = wl.make_batch(spec)
    per_step = max(1.0, min(20.0, 120.0 / max(1, args.steps + args.warmup)))
    for _ in range(args.warmup):
        oracle_sample(spec, batch, seconds_target=per_step)
    vals, times = [], []
    for _ in range(args.steps):
        v, n, cores, dt = oracle_sample(spec, batch, seconds_target=per_step)
        vals.append(v)
        times.append(dt / n * spec.L)   # a full step = all L layers at the sampled rate
    value = statistics.mean(vals)
    sample = (f"one of the {spec.L} layers of this workload, pack+unpack, repeated {n} times per step "
              f"({per_step:.0f} s), rows-memcpy oracle, {cores} threads")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": round(value, 3), "unit": UNIT,
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": round(statistics.mean(times) * 1e3, 3), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "u8", "data": "synthetic",
        "config": workload_config(spec, batch),
        "cpu_baseline": {"value": round(value, 3), "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": round(value, 3), "unit": UNIT, "h2d_bytes_per_step": 0,
                "d2h_bytes_per_step": 0},
    }))


def HEADLINE(wl):
    """The workload the N = 1 line is quoted on: the largest single-GPU configuration."""
    return wl.CFG3


_PINNED = {}


def pinned_buffer(nbytes, fallback_bytes=None):
    """One pinned host buffer for the whole run, grown on demand and handed out as views (pinning
    10 GiB takes seconds, and the host allocator rounds sizes up). Returns a uint8 tensor of
    nbytes, or of fallback_bytes when the box refuses the larger size."""
    import torch
    have = _PINNED.get("buf")
    if have is not None and have.numel() >= nbytes:
        return have[:nbytes]
    try:
        _PINNED["buf"] = None
        del have
        _PINNED["buf"] = torch.empty(nbytes, dtype=torch.uint8, pin_memory=True)
        return _PINNED["buf"][:nbytes]
    except Exception:
        if fallback_bytes is None:
            raise
        _PINNED["buf"] = torch.empty(fallback_bytes, dtype=torch.uint8, pin_memory=True)
        return _PINNED["buf"][:fallback_bytes]


def workload_config(spec, batch):
    return {"workload": spec.name, "note": spec.note, "layers": spec.L, "requests": spec.R,
            "total_tokens": batch.total_tokens, "page_tokens": spec.P,
            "wire_bytes_per_layer": batch.total_tokens * spec.tok_bytes,
            "pool_pages": batch.num_pool_pages,
            "l2": "inputs larger than L2: every layer touches distinct memory and all packs "
                  "precede all unpacks, so no slab is re-read from L2"}


def bench_d2d(w, stream, steps, warmup, barrier):
    """Times K steps of plan + pack(all layers) + unpack(all layers). Returns per-step ms
    (whole region / K), and the summed pack-phase and unpack-phase ms."""
    import torch
    from paper_2607_28633_b200 import binding as tk
    L = w.layers
    plan_batch = tk.make_batch(w.src_bt, w.seq_lens)

    def step(rec):
        tk.check(tk.topkv_build_plan(plan_batch, w.cu, stream))
        e0 = torch.cuda.Event(enable_timing=True); e0.record(stream)
        # Layers are independent of each other, so every launch after the first of a phase
        # carries TOPKV_FLAG_OVERLAP_PREVIOUS; the first one must see the plan / the wire.
        for l in range(L):
            w.pack(l, stream, overlap=l > 0)
        e1 = torch.cuda.Event(enable_timing=True); e1.record(stream)
        for l in range(L):
            w.unpack(l, stream, overlap=l > 0)
        e2 = torch.cuda.Event(enable_timing=True); e2.record(stream)
        if rec is not None:
            rec.append((e0, e1, e2))

    for _ in range(warmup):
        step(None)
    stream.synchronize()
    barrier()
    rec = []
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = tk.topkv_kernel_launch_count()
    t0.record(stream)
    for _ in range(steps):
        step(rec)
    t1.record(stream)
    stream.synchronize()
    launches = tk.topkv_kernel_launch_count() - launches0
    total_ms = t0.elapsed_time(t1)
    pack_ms = sum(a.elapsed_time(b) for a, b, _ in rec)
    unpack_ms = sum(b.elapsed_time(c) for _, b, c in rec)
    return total_ms / steps, pack_ms / steps, unpack_ms / steps, launches


def bench_host_leg(w, stream, pinned, staging, steps, warmup, barrier, slots, staging2=None):
    """pack_to_host for all layers then unpack_from_host for all layers, through pinned host
    memory (``slots`` slabs used as a ring). With ``staging2`` the layers alternate between two
    streams with a staging slab each, so that the copy engine moves layer l while the kernel of
    layer l + 1 runs. Returns ms per step and the two phase times."""
    import ctypes
    import torch
    from paper_2607_28633_b200 import binding as tk
    L, n = w.layers, w.n_layer
    lo = type(w.layout)()
    ctypes.memmove(ctypes.byref(lo), ctypes.byref(w.layout), ctypes.sizeof(lo))
    lo.wire_layer_stride = 0
    cap = 0 if staging is None else staging.numel()
    second = torch.cuda.Stream(w.src_pool.device) if staging2 is not None else None

    def phase(call):
        """All layers through `call`, on one stream or alternating between two."""
        if second is None:
            for l in range(L):
                call(l, staging, stream)
            return
        fork = torch.cuda.Event()
        fork.record(stream)
        second.wait_event(fork)
        for l in range(L):
            call(l, staging if l % 2 == 0 else staging2, stream if l % 2 == 0 else second)
        join = torch.cuda.Event()
        join.record(second)
        stream.wait_event(join)

    def to_host(l, st, q):
        slab = pinned[(l % slots) * n:(l % slots + 1) * n]
        tk.check(tk.topkv_pack_layer_to_host(l, w.src_pool, lo, w.src_batch, slab, n, st, cap, q))

    def from_host(l, st, q):
        slab = pinned[(l % slots) * n:(l % slots + 1) * n]
        tk.check(tk.topkv_unpack_layer_from_host(l, w.dst_pool, lo, w.dst_batch, slab, n, st, cap, q))

    def two_lanes(fn, pool, batch):
        """All layers through one library call that alternates between two streams and two
        staging slabs (needs one pinned slab per layer)."""
        lanes = [stream, second]
        fork = torch.cuda.Event()
        fork.record(stream)
        second.wait_event(fork)
        tk.check(fn(0, L, pool, w.layout, batch, pinned, L * n, [staging, staging2], cap, None, None,
                    lanes))
        join = torch.cuda.Event()
        join.record(second)
        stream.wait_event(join)

    def step(rec):
        e0 = torch.cuda.Event(enable_timing=True); e0.record(stream)
        if second is not None and slots >= L:
            two_lanes(tk.topkv_pack_layers_to_host_two_lanes, w.src_pool, w.src_batch)
        else:
            phase(to_host)
        e1 = torch.cuda.Event(enable_timing=True); e1.record(stream)
        if second is not None and slots >= L:
            two_lanes(tk.topkv_unpack_layers_from_host_two_lanes, w.dst_pool, w.dst_batch)
        else:
            phase(from_host)
        e2 = torch.cuda.Event(enable_timing=True); e2.record(stream)
        if rec is not None:
            rec.append((e0, e1, e2))

    for _ in range(warmup):
        step(None)
    stream.synchronize()
    barrier()
    rec = []
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record(stream)
    for _ in range(steps):
        step(rec)
    t1.record(stream)
    stream.synchronize()
    total = t0.elapsed_time(t1) / steps
    to_host = sum(a.elapsed_time(b) for a, b, _ in rec) / steps
    from_host = sum(b.elapsed_time(c) for _, b, c in rec) / steps
    return total, to_host, from_host


def bench_host_relay(w, stream, pinned, staging_tx, staging_rx, steps, warmup, barrier, slots):
    """The same layers through pinned host memory, pipelined the way a relay would run it: layer
    l is packed to the host while layers that have already arrived are unpacked from it, so both
    directions of the PCIe link are busy. The whole relay is two library calls
    (topkv_pack_layers_to_host_two_lanes, topkv_unpack_layers_from_host_two_lanes): each direction
    alternates between two streams with a staging slab each, so that the copy engine moves layer
    l while the kernel of layer l + 1 runs, and the receiver's layer_ready events are the
    sender's layer_done events. Returns ms per step (first pack enqueued to last unpack
    finished)."""
    import torch
    from paper_2607_28633_b200 import binding as tk
    L, n = w.layers, w.n_layer
    dev = w.src_pool.device
    assert slots >= L, "the relay keeps every layer's slab until it is unpacked"
    tx = [torch.cuda.Stream(dev), torch.cuda.Stream(dev)]
    rx = [torch.cuda.Stream(dev), torch.cuda.Stream(dev)]
    st_tx = [staging_tx, torch.empty_like(staging_tx)]
    st_rx = [staging_rx, torch.empty_like(staging_rx)]
    sent = [torch.cuda.Event() for _ in range(L)]

    def step():
        start = torch.cuda.Event()
        start.record(stream)
        for q in tx + rx:
            q.wait_event(start)
        tk.check(tk.topkv_pack_layers_to_host_two_lanes(
            0, L, w.src_pool, w.layout, w.src_batch, pinned, L * n, st_tx, n, None, sent, tx))
        tk.check(tk.topkv_unpack_layers_from_host_two_lanes(
            0, L, w.dst_pool, w.layout, w.dst_batch, pinned, L * n, st_rx, n, sent, None, rx))
        for q in tx + rx:                # the step ends when both directions have finished
            done = torch.cuda.Event()
            done.record(q)
            stream.wait_event(done)

    for _ in range(warmup):
        step()
    torch.cuda.synchronize()
    barrier()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record(stream)
    for _ in range(steps):
        step()
    t1.record(stream)
    torch.cuda.synchronize()
    return t0.elapsed_time(t1) / steps


def bench_repage(w, stream, steps):
    """Direct pool -> pool re-paging of every layer (topkv_repage_layer); GB/s of read + write."""
    import torch
    from paper_2607_28633_b200 import binding as tk

    def run():
        for l in range(w.layers):
            ov = l > 0
            tk.check(tk.topkv_repage_layer(l, w.src_pool, w.layout, w._flagged(w.src_batch, ov),
                                           w.dst_pool, w.layout, w._flagged(w.dst_batch, ov), stream))
    run()
    stream.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(stream)
    for _ in range(steps):
        run()
    b.record(stream)
    stream.synchronize()
    return 2.0 * w.n_layer * w.layers * steps / (a.elapsed_time(b) * 1e-3) / 1e9


def bench_crc(w, stream, steps):
    """pack and unpack with the CRC-64 of every request's K and V tensors fused in
    (topkv_pack_layer_crc / topkv_unpack_layer_crc); GB/s of read + write traffic."""
    import torch
    from paper_2607_28633_b200 import binding as tk
    spec = w.batch.spec
    nws = tk.topkv_crc_workspace_bytes(w.layout, spec.R, w.batch.max_pages_per_req)
    ws = torch.empty(nws, dtype=torch.uint8, device=w.src_pool.device)
    crc = torch.empty(spec.R * spec.F, dtype=torch.int64, device=w.src_pool.device)
    out = {}
    for name, fn, pool, batch in (("pack_crc", tk.topkv_pack_layer_crc, w.src_pool, w.src_batch),
                                  ("unpack_crc", tk.topkv_unpack_layer_crc, w.dst_pool, w.dst_batch)):
        def run():
            tk.check(tk.topkv_crc_begin(w.layout, batch, ws, nws, stream))
            for l in range(w.layers):
                tk.check(fn(l, pool, w.layout, w._flagged(batch, l > 0), w.wire, w.wire.numel(), ws,
                            nws, stream))
            tk.check(tk.topkv_crc_finish(w.layout, batch, ws, nws, crc, stream))
        run()
        stream.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(steps):
            run()
        b.record(stream)
        stream.synchronize()
        ms = a.elapsed_time(b) / steps
        out[name + "_GBps"] = round(2.0 * w.n_layer * w.layers / (ms * 1e-3) / 1e9, 1)
        out[name + "_us_per_layer"] = round(ms / w.layers * 1e3, 2)
    out["checksummed_payload_GBps"] = round(out["pack_crc_GBps"] / 2, 1)
    return out


def pinned_copy_baseline(dev, stream, nbytes, reps=5):
    """cudaMemcpyAsync of one slab between pinned host and device memory (torch copy_), GB/s."""
    import torch
    h = torch.empty(nbytes, dtype=torch.uint8, pin_memory=True)
    d = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    out = {}
    with torch.cuda.stream(stream):
        for name, (dst, src) in (("d2h", (h, d)), ("h2d", (d, h))):
            dst.copy_(src, non_blocking=True)
            stream.synchronize()
            best = 1e30
            for _ in range(reps):
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(stream)
                dst.copy_(src, non_blocking=True)
                b.record(stream)
                stream.synchronize()
                best = min(best, a.elapsed_time(b))
            out[name] = nbytes / (best * 1e-3) / 1e9
    return out


def pinned_copy_bidirectional_baseline(dev, nbytes, reps=8):
    """cudaMemcpyAsync device->host and host->device at the same time on two streams (torch
    copy_), ``reps`` slabs each way back to back: GB/s per direction with both busy."""
    import torch
    h_out = torch.empty(nbytes, dtype=torch.uint8, pin_memory=True)
    h_in = torch.empty(nbytes, dtype=torch.uint8, pin_memory=True)
    d_out = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    d_in = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    s1, s2 = torch.cuda.Stream(dev), torch.cuda.Stream(dev)
    best = 1e30
    for it in range(3):
        torch.cuda.synchronize(dev)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        c, d = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(s1):
            a.record(s1)
            for _ in range(reps):
                h_out.copy_(d_out, non_blocking=True)
            b.record(s1)
        with torch.cuda.stream(s2):
            c.record(s2)
            for _ in range(reps):
                d_in.copy_(h_in, non_blocking=True)
            d.record(s2)
        torch.cuda.synchronize(dev)
        if it:
            best = min(best, max(a.elapsed_time(b), c.elapsed_time(d)))
    return reps * nbytes / (best * 1e-3) / 1e9


def device_copy_baseline(dev, stream, nbytes, reps=10):
    """Plain device-to-device copy of nbytes (torch copy_), read+write GB/s, best of reps."""
    import torch
    a_ = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    b_ = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    best = 1e30
    with torch.cuda.stream(stream):
        for _ in range(3):
            b_.copy_(a_)
        for _ in range(reps):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            b_.copy_(a_)
            b.record(stream)
            stream.synchronize()
            best = min(best, a.elapsed_time(b))
    return 2 * nbytes / (best * 1e-3) / 1e9


def bench_chain(w, stream, steps, unpack_flags=0, slabs=1):
    """The dependent order of a relay without a host hop: pack(l), unpack(l), pack(l+1), ...
    where every unpack needs the slab that the pack just before it wrote, so an unpack can never
    be declared independent. With ``slabs`` = 1 all layers go through ONE wire slab, so pack(l+1)
    also has to wait for unpack(l) to have read it and no launch may overlap its predecessor.
    With 2 slabs the layers alternate between them: pack(l+1) then touches nothing that
    unpack(l) or pack(l) touch and carries TOPKV_FLAG_OVERLAP_PREVIOUS within the flag's
    contract, while every unpack still waits for its pack. GB/s of read + write traffic, and
    microseconds per launch."""
    import ctypes
    import torch
    from paper_2607_28633_b200 import binding as tk
    lo = type(w.layout)()
    ctypes.memmove(ctypes.byref(lo), ctypes.byref(w.layout), ctypes.sizeof(lo))
    lo.wire_layer_stride = 0
    n = w.n_layer
    slab = [w.wire[k * n:(k + 1) * n] for k in range(slabs)]
    T = w.batch.total_tokens
    ov = tk.TOPKV_FLAG_OVERLAP_PREVIOUS if slabs > 1 else 0
    bs0 = tk.make_batch(w.src_bt, w.seq_lens, T, w.cu, 0)
    bs = tk.make_batch(w.src_bt, w.seq_lens, T, w.cu, ov)
    bd = tk.make_batch(w.dst_bt, w.seq_lens, T, w.cu, unpack_flags)

    def run():
        for l in range(w.layers):
            q = slab[l % slabs]
            tk.check(tk.topkv_pack_layer(l, w.src_pool, lo, bs if l else bs0, q, n, stream))
            tk.check(tk.topkv_unpack_layer(l, w.dst_pool, lo, bd, q, n, stream))
    run()
    stream.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(stream)
    for _ in range(steps):
        run()
    b.record(stream)
    stream.synchronize()
    ms = a.elapsed_time(b) / steps
    return 4.0 * w.n_layer * w.layers / (ms * 1e-3) / 1e9, ms / (2 * w.layers) * 1e3


def bench_chain_linked(w, stream, steps, slabs=1):
    """The same dependent order with span links (topkv_pack_layer_linked /
    topkv_unpack_layer_linked): unpack(l) waits span by span for pack(l), pack(l + slabs) span by
    span for unpack(l) to have read the slab, and no launch waits for its predecessor as a whole."""
    import ctypes
    import torch
    from paper_2607_28633_b200 import binding as tk
    lo = type(w.layout)()
    ctypes.memmove(ctypes.byref(lo), ctypes.byref(w.layout), ctypes.sizeof(lo))
    lo.wire_layer_stride = 0
    n = w.n_layer
    slab = [w.wire[k * n:(k + 1) * n] for k in range(slabs)]
    T = w.batch.total_tokens
    bs = tk.make_batch(w.src_bt, w.seq_lens, T, w.cu)
    bd = tk.make_batch(w.dst_bt, w.seq_lens, T, w.cu)
    words = tk.check(tk.topkv_span_link_words(lo, bs))
    dev = w.src_pool.device
    fp = [torch.zeros(words, dtype=torch.int32, device=dev) for _ in range(slabs)]
    fu = [torch.zeros(words, dtype=torch.int32, device=dev) for _ in range(slabs)]
    uses = [0] * slabs           # how often each slab has been through a pack / unpack pair

    def run():
        for l in range(w.layers):
            q = l % slabs
            e = uses[q]
            lp = tk.make_span_link(fu[q] if e else None, e, fp[q], e + 1)
            tk.check(tk.topkv_pack_layer_linked(l, w.src_pool, lo, bs, slab[q], n, lp, stream))
            lu = tk.make_span_link(fp[q], e + 1, fu[q], e + 1)
            tk.check(tk.topkv_unpack_layer_linked(l, w.dst_pool, lo, bd, slab[q], n, lu, stream))
            uses[q] = e + 1
    run()
    stream.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(stream)
    for _ in range(steps):
        run()
    b.record(stream)
    stream.synchronize()
    assert tk.topkv_device_error_flags() == 0
    ms = a.elapsed_time(b) / steps
    return 4.0 * w.n_layer * w.layers / (ms * 1e-3) / 1e9, ms / (2 * w.layers) * 1e3


def launch_modes(w, stream, peak):
    """The pack and the unpack of every layer of the workload in the ways a caller can issue them,
    each layer into its own slab of the wire (every launch touches memory no earlier one touched,
    so L2 holds nothing for it): one call alone between two synchronisations (what the side
    stream of §5.2 issues after a layer's event; the median over the layers, CUDA events around
    each call), all layers back to back with no flag (every launch waits for the one before it),
    with TOPKV_FLAG_TABLES_SETTLED, and with TOPKV_FLAG_OVERLAP_PREVIOUS (the headline's form).
    GB/s of read + write traffic per launch."""
    import statistics
    import torch
    from paper_2607_28633_b200 import binding as tk
    L, n, T = w.layers, w.n_layer, w.batch.total_tokens
    tk.check(tk.topkv_build_plan(tk.make_batch(w.src_bt, w.seq_lens), w.cu, stream))
    stream.synchronize()
    out = {}
    for what, fn, pool, bt in (("pack", tk.topkv_pack_layer, w.src_pool, w.src_bt),
                               ("unpack", tk.topkv_unpack_layer, w.dst_pool, w.dst_bt)):
        def batch(flags):
            return tk.make_batch(bt, w.seq_lens, T, w.cu, flags)

        def call(l, b):
            tk.check(fn(l, pool, w.layout, b, w.wire, w.wire.numel(), stream))
        r = {}
        b0 = batch(0)
        for l in range(min(L, 3)):
            call(l, b0)
        stream.synchronize()
        times = []
        for l in range(L):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            call(l, b0)
            b.record(stream)
            stream.synchronize()
            times.append(a.elapsed_time(b) * 1e3)
        us = statistics.median(times)
        r["one_call_alone"] = {"us_per_launch_median": round(us, 2), "us_min": round(min(times), 2),
                               "us_max": round(max(times), 2), "calls": L,
                               "GBps": round(2.0 * n / (us * 1e-6) / 1e9, 1)}
        for label, first, rest in (("back_to_back_no_flag", 0, 0),
                                   ("back_to_back_tables_settled", 0, tk.TOPKV_FLAG_TABLES_SETTLED),
                                   ("back_to_back_overlap_previous", 0, tk.TOPKV_FLAG_OVERLAP_PREVIOUS)):
            bf, br = batch(first), batch(rest)
            best = None
            for _ in range(3):
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(stream)
                for l in range(L):
                    call(l, br if l else bf)
                b.record(stream)
                stream.synchronize()
                t = a.elapsed_time(b) * 1e3 / L
                best = t if best is None else min(best, t)
            r[label] = {"us_per_launch": round(best, 2), "GBps": round(2.0 * n / (best * 1e-6) / 1e9, 1)}
        for v in r.values():
            v["frac_of_hbm_peak"] = round(v["GBps"] / peak, 4)
            v["frac_of_8000_spec"] = round(v["GBps"] / 8000.0, 4)
        out[what] = r
    if L >= 2:
        # for scale: a plain device copy of one slab (torch copy_, N_layer read + N_layer written)
        # issued the same way, alone between two synchronisations
        times = []
        with torch.cuda.stream(stream):
            for k in range(max(20, L)):
                i, j = k % L, (k + L // 2) % L
                if i == j:
                    continue
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(stream)
                w.wire[i * n:(i + 1) * n].copy_(w.wire[j * n:(j + 1) * n])
                b.record(stream)
                stream.synchronize()
                times.append(a.elapsed_time(b) * 1e3)
        us = statistics.median(times[3:])
        out["plain_copy_one_call_alone"] = {"us_per_launch_median": round(us, 2),
                                            "GBps": round(2.0 * n / (us * 1e-6) / 1e9, 1),
                                            "frac_of_hbm_peak": round(2.0 * n / (us * 1e-6) / 1e9 / peak, 4)}
    return out


def host_leg_forms(w, dev, stream, pinned, slots, steps):
    """The host leg of the workload in its three forms against a pinned cudaMemcpyAsync of one
    slab measured in the same run."""
    import torch
    nobar = lambda: None
    staging = torch.empty(w.n_layer, dtype=torch.uint8, device=dev)
    staging2 = torch.empty(w.n_layer, dtype=torch.uint8, device=dev)
    base = pinned_copy_baseline(dev, stream, w.n_layer)
    out = {}
    for form, st, st2 in (("staged", staging, None), ("staged_two_lanes", staging, staging2),
                          ("direct", None, None)):
        _, th, fh = bench_host_leg(w, stream, pinned, st, steps, 1, nobar, slots, st2)
        d2h = w.n_layer * w.layers / (th * 1e-3) / 1e9
        h2d = w.n_layer * w.layers / (fh * 1e-3) / 1e9
        out[form] = {"to_host_GBps": round(d2h, 2), "from_host_GBps": round(h2d, 2),
                     "to_host_frac_of_pinned_copy": round(d2h / base["d2h"], 4),
                     "from_host_frac_of_pinned_copy": round(h2d / base["h2d"], 4)}
    out["pinned_copy_GBps"] = {k: round(v, 2) for k, v in base.items()}
    out["pinned_slots"] = slots
    return out


def run_extra(name, dev, stream, args, peak):
    """Other benchmark shapes at one GPU; returns a dict for the ``extra`` object."""
    import torch
    from paper_2607_28633_b200 import binding as tk
    from paper_2607_28633_b200 import harness, overlap
    from paper_2607_28633_b200 import workloads as wl
    nobar = lambda: None
    spec = wl.ALL[name] if name in wl.ALL else None
    out = {"workload": spec.name if spec else name}
    if name == "cfg1":
        # the tiny, launch-bound case: eager issue against one CUDA graph of the whole step
        w = harness.setup(wl.CFG1, dev, fill_dst=False)

        def step():
            for l in range(w.layers):
                w.pack(l, stream, overlap=l > 0)
            for l in range(w.layers):
                w.unpack(l, stream, overlap=l > 0)

        def timed(fn, reps=200):
            for _ in range(10):
                fn()
            stream.synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            for _ in range(reps):
                fn()
            b.record(stream)
            stream.synchronize()
            return a.elapsed_time(b) / reps * 1e3

        def step_one_launch():
            tk.check(tk.topkv_pack_layers(0, w.layers, w.src_pool, w.layout, w.src_batch, w.wire,
                                          w.wire.numel(), stream))
            tk.check(tk.topkv_unpack_layers(0, w.layers, w.dst_pool, w.layout, w.dst_batch, w.wire,
                                            w.wire.numel(), stream))

        with torch.cuda.stream(stream):
            eager_us = timed(step)
            one_launch_us = timed(step_one_launch)
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=stream):
                step()
            graph_us = timed(graph.replay)
        out = {"workload": wl.CFG1.name, "kernels_per_step": 2 * w.layers,
               "eager_us_per_step": round(eager_us, 2), "cuda_graph_us_per_step": round(graph_us, 2),
               "all_layers_in_one_launch_us_per_step": round(one_launch_us, 2),
               "bytes_moved_per_step": 4 * w.n_layer * w.layers,
               "note": "1.8 MB per layer: L2-resident and launch-bound, no roofline claim"}
        del w, graph
        torch.cuda.empty_cache()
        return out
    if name == "session":
        # the whole protocol through pinned host memory: checksummed host leg on both sides,
        # pipelined per layer, one header per request, receiver-side verification (§3.4, §5.2)
        from paper_2607_28633_b200 import session
        spec = wl.CFG2 if args.layers is None else wl.with_layers(wl.CFG2, args.layers)
        w = harness.setup(spec, dev, need_wire=False, fill_dst=False)
        b = w.batch
        tx = session.TransferSender(w.src_pool, w.layout, w.src_bt, w.seq_lens, b.total_tokens)
        rx = session.TransferReceiver(w.dst_pool, w.layout, w.dst_bt, w.seq_lens, b.total_tokens)
        h_wire = pinned_buffer(w.layers * w.n_layer)
        ids = list(range(spec.R))
        best, ok = 1e30, True
        for it in range(3):
            torch.cuda.synchronize(dev)
            t0 = time.perf_counter()
            _, status = session.transfer(tx, rx, h_wire, ids, 1, b.seq_lens)
            torch.cuda.synchronize(dev)
            dt = time.perf_counter() - t0
            ok = ok and all(st == tk.TOPKV_OK for st in status)
            if it:
                best = min(best, dt)
        out = {"workload": spec.name, "all_requests_verified": ok,
               "ms_per_transfer": round(best * 1e3, 3),
               "GBps_read_plus_write_equivalent": round(4.0 * w.n_layer * w.layers / best / 1e9, 1),
               "link_GBps_each_direction": round(w.n_layer * w.layers / best / 1e9, 2),
               "note": "wall clock around the whole transfer, checksum read-back and header checks included"}
        del w, tx, rx, h_wire
        torch.cuda.empty_cache()
        return out
    if name == "crc":
        # the checksummed copy on the three benchmark shapes, all layers: begin, one copy per
        # layer, finish, all inside the timed region
        out = {}
        for base, layers in ((wl.CFG2, None), (wl.CFG3, None), (wl.CFG4, None)):
            layers = args.layers if args.layers is not None else layers
            spec = base if layers is None else wl.with_layers(base, layers)
            w = harness.setup(spec, dev, fill_dst=False)
            r = {"layers": w.layers}
            r.update(bench_crc(w, stream, max(1, min(args.steps, 5))))
            r["frac_of_hbm_peak"] = round(r["pack_crc_GBps"] / peak, 4)
            r["unpack_frac_of_hbm_peak"] = round(r["unpack_crc_GBps"] / peak, 4)
            out[base.name] = r
            del w
            torch.cuda.empty_cache()
        out["workload"] = wl.CFG2.name
        out["frac_of_hbm_peak"] = out[wl.CFG2.name]["frac_of_hbm_peak"]
        return out
    if name == "chain":
        # pack(l) -> unpack(l) per layer, the order of a device-to-device relay: every unpack
        # depends on the pack before it. One shared slab (nothing may overlap) or two alternating
        # slabs (pack(l+1) is independent of unpack(l) and says so); unpack plain or with
        # TOPKV_FLAG_TABLES_SETTLED
        out = {"workload": "cfg2_llama3_8b, cfg4_dsv3_mla", "order": "pack(l), unpack(l), pack(l+1), ..."}
        for base in (wl.CFG2, wl.CFG4):
            spec = base if args.layers is None else wl.with_layers(base, args.layers)
            w = harness.setup(spec, dev, fill_dst=False)
            r = {}
            ts = tk.TOPKV_FLAG_TABLES_SETTLED
            for label, flags, slabs in (("one_slab_plain", 0, 1), ("one_slab_tables_settled", ts, 1),
                                        ("two_slabs_plain", 0, 2), ("two_slabs_tables_settled", ts, 2)):
                gbs, us = bench_chain(w, stream, max(1, min(args.steps, 5)), flags, slabs)
                r[label] = {"GBps": round(gbs, 1), "us_per_launch": round(us, 2),
                            "frac_of_hbm_peak": round(gbs / peak, 4),
                            "frac_of_8000_spec": round(gbs / 8000.0, 4)}
            for label, slabs in (("one_slab_span_linked", 1), ("two_slabs_span_linked", 2)):
                gbs, us = bench_chain_linked(w, stream, max(1, min(args.steps, 5)), slabs)
                r[label] = {"GBps": round(gbs, 1), "us_per_launch": round(us, 2),
                            "frac_of_hbm_peak": round(gbs / peak, 4),
                            "frac_of_8000_spec": round(gbs / 8000.0, 4)}
            # the same one-slab linked chain as ONE library call per pass
            words = tk.check(tk.topkv_span_link_words(w.layout, w.src_batch))
            flags = torch.zeros(2 * words, dtype=torch.int32, device=dev)
            slab = w.wire[:w.n_layer]
            done, reps = 0, max(1, min(args.steps, 5))

            def relay():
                nonlocal done
                tk.check(tk.topkv_relay_layers_linked(0, w.layers, w.src_pool, w.layout, w.src_batch,
                                                      w.dst_pool, w.layout, w.dst_batch, slab, w.n_layer,
                                                      flags, flags.numel(), done, stream))
                done += w.layers
            relay()
            stream.synchronize()
            ea, eb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            ea.record(stream)
            for _ in range(reps):
                relay()
            eb.record(stream)
            stream.synchronize()
            rms = ea.elapsed_time(eb) / reps
            gbs = 4.0 * w.n_layer * w.layers / (rms * 1e-3) / 1e9
            r["one_slab_relay_call"] = {"GBps": round(gbs, 1), "us_per_launch": round(rms / (2 * w.layers) * 1e3, 2),
                                        "frac_of_hbm_peak": round(gbs / peak, 4),
                                        "frac_of_8000_spec": round(gbs / 8000.0, 4)}
            del flags
            out[base.name] = r
            del w
            torch.cuda.empty_cache()
        return out
    if name == "hybrid":
        # models whose layers differ in kind (§2.2) through the layer-table calls, device to
        # device: a gpt-oss-shaped one (36 layers, every other one windowed at 128 tokens, 8 KV
        # heads of 64) and a Qwen3.5-shaped one (60 layers, 45 of them a constant 1 MiB state
        # per request, 15 full layers of 2 KV heads of 256), both on cfg2's 16 requests of
        # 512..4096 tokens. GB/s of read + write traffic over all slabs of the model.
        import numpy as np
        from dataclasses import replace
        out = {"workload": "cfg2 batch; gpt-oss-shaped and Qwen3.5-shaped layer tables"}
        F_, W_, S_ = tk.TOPKV_LAYER_FULL, tk.TOPKV_LAYER_WINDOW, tk.TOPKV_LAYER_STATE
        state = 1 << 20
        models = (("gpt_oss_shaped", replace(wl.CFG2, L=36, H=8, D=64),
                   [(W_, 128) if l % 2 == 0 else (F_, 0) for l in range(36)]),
                  ("qwen35_shaped", replace(wl.CFG2, L=15, H=2, D=256),
                   [(F_, 0) if l % 4 == 3 else (S_, state) for l in range(60)]))
        for label, spec, specs in models:
            w = harness.setup(spec, dev, fill_dst=False, need_wire=False)
            R = spec.R
            n_state = sum(1 for k, _ in specs if k == S_)
            slots = R + 4
            sp_s = wl.fill_torch(max(n_state * slots * state, 16), 77, dev, raw_bits=True)
            sp_d = torch.zeros_like(sp_s)
            g = np.random.Generator(np.random.PCG64(78))
            sl_s = torch.from_numpy(g.permutation(slots)[:R].astype(np.int32)).to(dev)
            sl_d = torch.from_numpy(g.permutation(slots)[:R].astype(np.int32)).to(dev)
            ts = tk.make_layer_table(specs, w.batch.seq_lens, sp_s, sl_s, slots * state, state, slots)
            td = tk.make_layer_table(specs, w.batch.seq_lens, sp_d, sl_d, slots * state, state, slots)
            st, off = tk.topkv_layer_table_offsets(w.layout, ts, R)
            tk.check(st)
            total = int(off[-1])
            wire = torch.empty(total, dtype=torch.uint8, device=dev)
            nl = len(specs)

            def run():
                tk.check(tk.topkv_pack_model_layers(0, nl, w.src_pool, w.layout, w.src_batch, ts, wire,
                                                    total, stream))
                tk.check(tk.topkv_unpack_model_layers(0, nl, w.dst_pool, w.layout, w.dst_batch, td, wire,
                                                      total, stream))
            run()
            stream.synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            steps = max(1, min(args.steps, 5))
            a.record(stream)
            for _ in range(steps):
                run()
            b.record(stream)
            stream.synchronize()
            ms = a.elapsed_time(b) / steps
            gbs = 4.0 * total / (ms * 1e-3) / 1e9
            out[label] = {"model_layers": nl, "wire_bytes_all_layers": total,
                          "largest_slab_bytes": int(np.diff(off).max()),
                          "smallest_slab_bytes": int(np.diff(off).min()),
                          "ms_pack_plus_unpack": round(ms, 4), "GBps": round(gbs, 1),
                          "frac_of_hbm_peak": round(gbs / peak, 4),
                          "device_error_flags": tk.topkv_device_error_flags()}
            del w, sp_s, sp_d, wire
            torch.cuda.empty_cache()
        return out
    if name == "overlap_curve":
        # three points on the Eq. 3 curve (§5.2) and the interference §5.5 could not validate:
        # slack (64 MiB per layer under a 2.8 ms layer), near-saturated (128 MiB per layer, about
        # 2.4 ms on the link, under the same layer) and oversubscribed (128 MiB per layer under
        # a halved stand-in, so that T_xfer > T_rem and Eq. 3 predicts hidden < 1)
        points = (("slack", wl.CFG5, wl.GEMM_FFN), ("near_saturated", wl.CFG3, wl.GEMM_FFN),
                  ("oversubscribed", wl.CFG3, wl.GEMM_FFN // 2))
        out = {"workload": "cfg5 / cfg3 batches under the GEMM stand-in"}
        for label, base, ffn in points:
            spec = base if args.layers is None else wl.with_layers(base, args.layers)
            w = harness.setup(spec, dev, need_dst=False, need_wire=False)
            slots = w.layers
            pinned = pinned_buffer(slots * w.n_layer, 8 * w.n_layer)
            slots = min(slots, pinned.numel() // w.n_layer)
            staging = torch.empty(w.n_layer, dtype=torch.uint8, device=dev)
            pre = overlap.PrefillStandIn(dev, w.batch.seeds["data"] + 50, ffn=ffn)
            pt = {"requests": spec.R, "bytes_per_layer": w.n_layer, "gemm_ffn": ffn}
            for form, st in (("staged", staging), ("direct", None)):
                r = overlap.run_overlap(w, pinned, st, pre, slots=slots)
                model = tk.topkv_model_hidden_fraction(r.layers, r.t_layer_compute_ms * 1e-3,
                                                       r.t_xfer_serial_ms * 1e-3)
                # what Eq. 3 allows at best: the last slab's transfer can never be hidden
                bound = min(model, 1.0 - 1.0 / r.layers)
                pt[form] = {"hidden": round(r.hidden, 4), "hidden_model": round(model, 4),
                            "hidden_model_minus_last_slab": round(bound, 4),
                            "slowdown": round(r.slowdown, 4),
                            "t_layer_compute_ms": round(r.t_layer_compute_ms, 4),
                            "t_xfer_serial_ms": round(r.t_xfer_serial_ms, 3),
                            "t_main_overlap_ms": round(r.t_main_overlap_ms, 3),
                            "exposed_ms": round(r.exposed_ms, 3),
                            "xfer_gbs_serial": round(r.xfer_gbs_serial, 2)}
            if label == "oversubscribed":
                # the direct form's interference against the number of CTAs that walk the spans
                # (every one of them holds an SM for the whole run once the link is always busy)
                sweep = {}
                for ctas in (4, 8, 16):
                    prev = tk.topkv_set_host_leg_ctas(ctas)
                    r = overlap.run_overlap(w, pinned, None, pre, slots=slots)
                    tk.topkv_set_host_leg_ctas(prev)
                    sweep[str(ctas)] = {"hidden": round(r.hidden, 4), "slowdown": round(r.slowdown, 4),
                                        "xfer_gbs_serial": round(r.xfer_gbs_serial, 2)}
                pt["direct_by_host_leg_ctas"] = sweep
            out[label] = pt
            del w, pinned, staging, pre
            torch.cuda.empty_cache()
        return out
    if name in ("cfg2", "cfg3", "cfg4"):
        if args.layers is not None:                      # fewer layers: profiling only
            spec = wl.with_layers(spec, args.layers)
        w = harness.setup(spec, dev, fill_dst=False)
        ms, pack_ms, unpack_ms, _ = bench_d2d(w, stream, args.steps, args.warmup, nobar)
        traffic = 2.0 * w.n_layer * w.layers
        out.update({"pack_GBps": round(traffic / (pack_ms * 1e-3) / 1e9, 1),
                    "unpack_GBps": round(traffic / (unpack_ms * 1e-3) / 1e9, 1),
                    "pack_frac_of_peak": round(traffic / (pack_ms * 1e-3) / 1e9 / peak, 4),
                    "unpack_frac_of_peak": round(traffic / (unpack_ms * 1e-3) / 1e9 / peak, 4),
                    "ms_per_step": round(ms, 4), "wire_bytes_per_layer": w.n_layer,
                    "layers": w.layers})
        if name == "cfg2":
            out["repage_GBps"] = round(bench_repage(w, stream, max(1, min(args.steps, 5))), 1)
        del w
    elif name == "cfg5":
        w = harness.setup(spec, dev, need_dst=False, need_wire=False)
        slots = w.layers
        pinned = pinned_buffer(slots * w.n_layer, 8 * w.n_layer)
        slots = min(slots, pinned.numel() // w.n_layer)
        staging = torch.empty(w.n_layer, dtype=torch.uint8, device=dev)
        pre = overlap.PrefillStandIn(dev, w.batch.seeds["data"] + 50)
        best = None
        # direct = mapped stores from a bounded grid (the library's default, 8 CTAs);
        # direct_cta_per_span = the same stores from one CTA per page span, for contrast
        for form, st, ctas in (("staged", staging, None), ("direct", None, None),
                               ("direct_cta_per_span", None, 0)):
            prev = tk.topkv_set_host_leg_ctas(ctas) if ctas is not None else None
            r = overlap.run_overlap(w, pinned, st, pre, slots=slots)
            if prev is not None:
                tk.topkv_set_host_leg_ctas(prev)
            d = r.as_dict()
            d["form"] = form
            d["hidden_model"] = round(min(1.0, (r.layers - 1) * r.t_layer_compute_ms
                                          / r.t_xfer_serial_ms), 6)
            d["prefill_tflops_alone"] = round(pre.flop_per_layer / (r.t_layer_compute_ms * 1e-3)
                                              / 1e12, 1)
            out[form] = d
            # among the forms that hide >= 95 %: the one that disturbs the prefill least, where a
            # difference below 5 % is run-to-run noise and the earlier (faster-link) form stays
            if best is None or (d["hidden"] >= 0.95 and d["slowdown"] < out[best]["slowdown"] - 0.05):
                best = form
        # the same staged transfer with the CRC-64 of every request folded in
        nws = tk.topkv_crc_workspace_bytes(w.layout, spec.R, w.batch.max_pages_per_req)
        ws = torch.empty(nws, dtype=torch.uint8, device=dev)
        tk.check(tk.topkv_crc_begin(w.layout, w.src_batch, ws, nws, stream))
        stream.synchronize()
        r = overlap.run_overlap(w, pinned, staging, pre, slots=slots, crc_workspace=ws)
        out["staged_crc"] = {"hidden": round(r.hidden, 6), "slowdown": round(r.slowdown, 6),
                             "t_xfer_serial_ms": round(r.t_xfer_serial_ms, 3),
                             "xfer_gbs_serial": round(r.xfer_gbs_serial, 2)}
        out["best_form"] = best
        out["hidden_fraction"] = out[best]["hidden"]
        out["pinned_slots"] = slots
        del w, pinned, staging, pre
    torch.cuda.empty_cache()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="topkv", choices=["topkv", "reference"])
    ap.add_argument("--no-launch-modes", action="store_true",
                    help="skip the one-call-alone / back-to-back comparison of the headline workload")
    ap.add_argument("--extras", default="cfg5,overlap_curve,cfg2,cfg4,chain,crc,hybrid,session,cfg1",
                    help="comma list of extra workloads measured at one GPU ('' for none)")
    ap.add_argument("--variant", type=int, default=None, help="kernel family (see topkv.h)")
    ap.add_argument("--layers", type=int, default=None, help="fewer layers (profiling only)")
    ap.add_argument("--workload", default=None, choices=["cfg2", "cfg3", "cfg4"],
                    help="time another benchmark shape in place of the headline one (profiling only)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 0)

    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    import __graft_entry__ as entry
    from paper_2607_28633_b200 import binding as tk
    from paper_2607_28633_b200 import harness
    from paper_2607_28633_b200 import workloads as wl

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the TopKV path has no CPU fallback")
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if rank == 0:
        entry.build()
    from paper_2607_28633_b200 import dist_util
    dev = torch.device("cuda", local)
    torch.cuda.set_device(dev)
    # Keep stdout to the one JSON line: the communicator's set-up prints a version banner there,
    # so file descriptor 1 points at stderr while the process group comes up.
    sys.stdout.flush()
    saved_stdout = os.dup(1)
    os.dup2(2, 1)
    try:
        dist = dist_util.init("nccl", dev)
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize(dev)
    finally:
        sys.stdout.flush()
        os.dup2(saved_stdout, 1)
        os.close(saved_stdout)
    tk.lib()
    if args.variant is not None:
        tk.check(tk.topkv_set_kernel_variant(args.variant))

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize(dev)

    def max_over_ranks(x: float) -> float:
        return dist_util.max_over_ranks(dist, x, dev)

    def sum_over_ranks(x: float) -> float:
        return dist_util.sum_over_ranks(dist, x, dev)

    peak, peak_src = measured_peak_gbs()
    head = HEADLINE(wl) if args.workload is None else wl.ALL[args.workload]
    spec = head if args.layers is None else wl.with_layers(head, args.layers)
    w = harness.setup(spec, dev, rank=rank, fill_dst=False)
    stream = torch.cuda.Stream(dev)
    L, n_layer = w.layers, w.n_layer

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    barrier()
    ms, pack_ms, unpack_ms, launches = bench_d2d(w, stream, args.steps, args.warmup, barrier)
    barrier()
    clocks = sampler.stop() if rank == 0 else None

    ms_max = max_over_ranks(ms)
    bytes_step_all = sum_over_ranks(4.0 * n_layer * L)        # pack r+w, unpack r+w
    value = bytes_step_all / (ms_max * 1e-3) / 1e9
    pack_launch_ms = pack_ms / L
    unpack_launch_ms = unpack_ms / L
    achieved = 2.0 * n_layer / (pack_launch_ms * 1e-3) / 1e9
    achieved_unpack = 2.0 * n_layer / (unpack_launch_ms * 1e-3) / 1e9

    e2e = None
    extra = {}
    if not args.no_e2e:
        # every layer through pinned host memory with the C-ABI host-leg calls: one slab per
        # layer (10 GiB for the 70B shape), or a ring of 4 slabs when the box refuses that much
        pinned = pinned_buffer(L * n_layer, 4 * n_layer)
        # every rank takes the same path (the barriers inside the timed legs must match): the
        # smallest number of slabs any rank obtained decides
        slots = int(round(-max_over_ranks(-float(min(L, pinned.numel() // n_layer)))))
        staging = torch.empty(n_layer, dtype=torch.uint8, device=dev)
        hs = max(1, min(args.steps, 3))
        ems, th, fh = bench_host_leg(w, stream, pinned, staging, hs, 1, barrier, slots)
        form = "staged (kernel + copy engine), pack of all layers then unpack of all layers"
        if slots < L:
            form += f"; ring of {slots} pinned slabs (the box refused one slab per layer)"
        if slots >= L:   # both link directions at once: unpack layer l while later layers pack
            staging_rx = torch.empty(n_layer, dtype=torch.uint8, device=dev)
            rms = bench_host_relay(w, stream, pinned, staging, staging_rx, hs, 1, barrier, slots)
            if rms < ems:
                ems = rms
                form = ("staged (kernel + copy engine), pipelined relay as two library calls "
                        "(topkv_pack_layers_to_host_two_lanes, topkv_unpack_layers_from_host_two_lanes): "
                        "layer l is unpacked from the host while later layers are still packed to it; "
                        "one pinned slab per layer")
            del staging_rx
        ems_max = max_over_ranks(ems)
        e2e = {"value": round(bytes_step_all / (ems_max * 1e-3) / 1e9, 3), "unit": UNIT,
               "h2d_bytes_per_step": n_layer * L, "d2h_bytes_per_step": n_layer * L,
               "form": form, "steps": hs, "ms_per_step": round(ems_max, 3),
               "pinned_slots": slots,
               "sequential_ms_per_step": round(th + fh, 3),
               "to_host_link_GBps": round(n_layer * L / (th * 1e-3) / 1e9, 2),
               "from_host_link_GBps": round(n_layer * L / (fh * 1e-3) / 1e9, 2)}
        del staging
        if rank == 0 and world == 1:
            if slots >= L:
                # what the link gives each direction while both are busy: plain pinned copies
                bidir = pinned_copy_bidirectional_baseline(dev, n_layer)
                e2e["pinned_copy_both_directions_GBps_each"] = round(bidir, 2)
                e2e["link_GBps_each_direction"] = round(n_layer * L / (ems_max * 1e-3) / 1e9, 2)
                e2e["frac_of_pinned_copy_both_directions"] = round(
                    n_layer * L / (ems_max * 1e-3) / 1e9 / bidir, 4)
            # the host leg one direction at a time, in its three forms, against a pinned copy
            hl = host_leg_forms(w, dev, stream, pinned, slots, hs)
            e2e["host_leg"] = hl
            e2e["to_host_frac_of_pinned_copy"] = hl["staged"]["to_host_frac_of_pinned_copy"]
            e2e["from_host_frac_of_pinned_copy"] = hl["staged"]["from_host_frac_of_pinned_copy"]
        del pinned

    if rank == 0:
        # the paper's own quoted link rates and the rates its orchestrator plans with (§3.3,
        # Table 2, Table 4): context for the figures above, measured on other hardware or not at
        # all, never a target of this run
        modes = (tk.TOPKV_TRANSPORT_NVLINK, tk.TOPKV_TRANSPORT_PCIE, tk.TOPKV_TRANSPORT_RDMA,
                 tk.TOPKV_TRANSPORT_TCP)
        extra["paper_context"] = {
            "published_link_GBps": {"nvlink4_h100_domain": 900, "nvlink5_per_gpu": 1800,
                                    "pcie_gen5_x16": 128, "infiniband_ndr": 50, "tcp_100gbe": 12.5},
            "planning_GBps": {tk.topkv_transport_name(m): tk.topkv_planning_rate(m) / 1e9 for m in modes},
            "eq2_ms_for_this_workload_per_request": {
                tk.topkv_transport_name(m): round(tk.topkv_model_transfer_s(
                    float(tk.topkv_kv_bytes(w.layout, 4096)) * head.L / max(1, w.layers),
                    tk.topkv_planning_rate(m), 0.0) * 1e3, 2) for m in modes},
            "note": "analytic or vendor figures quoted by the paper (H100-era hardware); no measured "
                    "number for this path exists in the paper"}
    if rank == 0 and world == 1:
        extra["device_copy_GBps_same_bytes"] = round(device_copy_baseline(dev, stream, n_layer), 1)
        if not args.no_launch_modes:
            extra["launch_modes"] = launch_modes(w, stream, peak)
    batch = w.batch
    del w
    torch.cuda.empty_cache()
    if world == 1 and args.extras:
        for name in [x for x in args.extras.split(",") if x]:
            xs = ClockSampler(local)      # every extra carries the clocks seen while it ran
            xs.start()
            try:
                extra[name] = run_extra(name, dev, stream, args, peak)
            except Exception as e:  # an extra must not take the headline line down
                extra[name] = {"error": f"{type(e).__name__}: {e}"}
                torch.cuda.empty_cache()
            c = xs.stop()
            if isinstance(extra[name], dict):
                extra[name]["clocks"] = {"sm_mhz": c.get("sm_mhz"), "reasons": c.get("reasons")}

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        v, n, cores, dt = oracle_sample(head, wl.make_batch(head), seconds_target=12.0)
        cpu = {"value": round(v, 3), "unit": UNIT, "cores": cores, "kind": "oracle",
               "sample": f"one of the {head.L} layers of this workload, pack+unpack, repeated "
                         f"{n} times, rows-memcpy oracle, {dt:.1f} s"}
        # for context: the same oracle on one thread, and the byte-by-byte definition on cfg1
        v1, n1, _, dt1 = oracle_sample(head, wl.make_batch(head), seconds_target=4.0, threads=1)
        vr, nr, _, dtr = oracle_sample(wl.CFG1, wl.make_batch(wl.CFG1), seconds_target=3.0, threads=1,
                                       impl="ref")
        cpu["one_thread_GBps"] = round(v1, 3)
        cpu["byte_loop_definition_cfg1_GBps"] = round(vr, 4)

    if rank == 0:
        traffic, traffic_src = ncu_traffic(2 * n_layer)
        line = {
            "metric": METRIC, "value": round(value, 3), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(ms_max, 4),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u8",
            "data": "synthetic", "config": workload_config(spec, batch),
            "gpu_launches": int(launches), "clocks": clocks,
            "roofline": {"bound": "hbm", "kernel": "topkv_page_copy_kernel (pack)",
                         "achieved": round(achieved, 1), "peak": peak, "unit": "GB/s",
                         "frac": round(achieved / peak, 4), "peak_source": peak_src,
                         "frac_of_8000_spec": round(achieved / 8000.0, 4),
                         "bytes_per_launch": 2 * n_layer,
                         "launch_ms": round(pack_launch_ms, 5),
                         "traffic": traffic, "traffic_source": traffic_src,
                         "unpack_achieved": round(achieved_unpack, 1),
                         "unpack_frac": round(achieved_unpack / peak, 4),
                         "unpack_launch_ms": round(unpack_launch_ms, 5)},
            "e2e": e2e, "cpu_baseline": cpu, "extra": extra,
        }
        print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
