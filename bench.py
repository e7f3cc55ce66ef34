#!/usr/bin/env python
"""Throughput of the adaptive-compression hot path on synthetic gradient buckets.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

One "step" is one pass of the whole path over one synthetic gradient set: the
host controller picks a ratio, every bucket is compressed (top-k selection,
compaction, value codec) and the W workers' payloads are decompressed and
summed into a dense buffer.  The metric is input-gradient bytes per second.
Prints ONE JSON line (rank 0).

Workloads (value distributions are described in synth.py):
  gpt2      124M fp32 parameters in GPT-2-small's shapes, 25M-element buckets,
            ratio 0.01, int8, W = 4 workers summed into one dense buffer  (default:
            the configuration with buckets of the size the bandwidth target is stated for)
  resnet50  25.6M fp32 parameters in ResNet-50's tensor shapes, 25 MB buckets,
            ratio sweep {0.5, 0.1, 0.01, 0.001} x {int8, fp16}, W = 1
  decoder   1.3B bf16 parameters, 64M-element buckets, fp16 values, ratio chosen
            every step by the controller from a synthetic 100/10/1 Gbps link trace
  agg       8 workers x int8 payloads for a 350M-element bucket (ratio 0.05),
            decompress + sum only
  alg2      the whole of Alg. 2 on 25M-element fp32 buckets: L2 norm, pruning mask
            built from synthetic weights, compress of gradient + residual (ratio
            0.01, int8), sum, W = 1

With --gpus N > 1 (started by torchrun, or by this script itself when it is run
plainly) every rank runs the workload on its own GPU and the ranks' times are
reduced with MAX; an extra leg times the data-parallel exchange: compress,
all-gather of the payloads over NCCL, sum of the N payloads.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "compress+decompress input-gradient GB/s per bucket; % of B200 HBM roofline"
UNIT = "GB/s"
SWEEP = [(r, b) for r in (0.5, 0.1, 0.01, 0.001) for b in (8, 16)]

def ncu_traffic(workload_key):
    """DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of the kernels of one workload, from
    the text summary of its ncu capture: lines 'traffic <workload> <kernel> <bytes>'.  Missing file or
    workload: no figures (the bench then reports traffic as null)."""
    out = {}
    try:
        with open(os.path.join(ROOT, "profiles", "dram_traffic_per_launch.txt")) as f:
            for line in f:
                parts = line.split()
                if len(parts) == 4 and parts[0] == "traffic" and parts[1] == workload_key:
                    out[parts[2]] = float(parts[3])
    except OSError:
        pass
    return out


def measured_peak_gbs():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


# --------------------------------------------------------------------------
# clocks during the timed region
# --------------------------------------------------------------------------
class ClockSampler:
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown",
               0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting"}

    def __init__(self, device_index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            import torch

            pynvml.nvmlInit()
            uuid = "GPU-" + str(torch.cuda.get_device_properties(device_index).uuid)
            self._h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode() if hasattr(uuid, "encode") else uuid)
            self._nv = pynvml
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._nv = None

    def _loop(self):
        nv = self._nv
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                try:
                    mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._h))
                except Exception:
                    mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))
                for bit, name in self.REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(0.02)

    def __enter__(self):
        if self._nv is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


# --------------------------------------------------------------------------
# workloads
# --------------------------------------------------------------------------
class Workload:
    """Device-resident inputs and preallocated outputs; step(i) enqueues one
    whole pass on the current stream and returns nothing."""

    name = ""
    dtype = "f32"

    job_turn = 0        # jobs enqueued so far (the lane of a job is its turn modulo the number of lanes)
    rotate_lanes = False  # keep counting turns from step to step instead of starting every step at lane 0
    use_graphs = False  # replay each job from a CUDA graph captured on its stream
    graph_period = 1    # steps after which the set of distinct jobs repeats (all graphs exist after that many)
    graphs_ok = True    # False where every step brings new jobs (nothing to replay)

    def account(self, acc, kernel, nbytes):
        acc[kernel] = acc.get(kernel, 0) + nbytes

    def before_step(self, i):
        """Host side of a step (the controller); returns nothing."""

    def after_step(self, i, sent):
        """Feeds the bytes this step would send back to the controller."""

    def step(self, i, acc=None):
        """One pass of the whole path.  Jobs (one bucket: its compress calls and the sum) are independent and
        go to the streams round-robin; with use_graphs a job is captured once per (inputs, ratio, codec, stream)
        and replayed, which takes the per-call launch cost off the host."""
        torch, nsml = self.torch, self.nsml
        self.before_step(i)
        sent = 0
        graphs = self.use_graphs and acc is None and self.lanes.active == len(self.lanes.all)
        if not self.rotate_lanes:
            self.job_turn = 0
        for key, nbytes, enqueue in self.jobs(i):
            # rotate_lanes: the turn count runs on from step to step, so with fewer jobs per step than lanes the
            # next step's first jobs start on the idle lanes while this step's last ones finish
            ordinal = self.job_turn
            self.job_turn += 1
            lane = self.lanes.all[ordinal % self.lanes.active]
            sent += nbytes
            if not graphs:
                enqueue(lane, acc)
                continue
            gkey = (key, ordinal % self.lanes.active)
            entry = self.graph_cache.get(gkey)
            if entry is None:
                before = nsml.nsml_launch_count()
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=lane.stream):
                    enqueue(lane, None)
                entry = (g, nsml.nsml_launch_count() - before)
                self.graph_cache[gkey] = entry
            torch.cuda.set_stream(lane.stream)
            entry[0].replay()
            self.replayed_launches += entry[1]
        if graphs:
            torch.cuda.set_stream(self.home_stream)
        self.after_step(i, sent)

    def init_graphs(self, use_graphs):
        self.use_graphs = use_graphs and self.graphs_ok
        self.graph_cache = {}
        self.job_turn = 0
        self.replayed_launches = 0
        self.home_stream = self.torch.cuda.current_stream()

    def compress_bytes(self, acc, n, esize, ratio, bits):
        k = self.nsml.nsml_k_of(n, ratio)
        vb = 1 if bits == 8 else 2
        s = 4 * ((k + 1023) // 1024) if bits == 8 else 0
        if self.nsml.nsml_compress_strategy(n, ratio) == 1:
            # dense strategy: the select reads the bucket itself once, survivors written and re-read
            self.account(acc, "k_clear", 256 + 4 * 4 * 4096)
            self.account(acc, "k_finalize_dense", esize * n + 8 * k + 4 * k + vb * k + s)
            return
        self.account(acc, "k_sample", 4 * 8192)
        self.account(acc, "k_compact_bucket", esize * n + 6 * k)  # candidates: 16-bit offset in the segment + value
        # gather: candidates read from the segmented list (6 bytes) and written contiguously (index + value)
        self.account(acc, "k_gather", 14 * k)
        # list stage: candidate values read once per phase (4 x 4k keys), indices once, survivors written and re-read
        self.account(acc, "k_finalize", 16 * k + 4 * k + 8 * k + 4 * k + vb * k + s)

    def merge_bytes(self, acc, n, ks_bits, zero_first=True):
        total = 4 * n if zero_first else 0
        for k, bits in ks_bits:
            total += k * (4 + (1 if bits == 8 else 2)) + (4 * ((k + 1023) // 1024) if bits == 8 else 0)
            if not zero_first:
                total += 8 * k
        self.account(acc, "k_merge", total)
        self.account(acc, "k_partition", 4 * len(ks_bits) * (n // 8192 + 2))


class Lanes:
    """Independent jobs (the compress calls of one bucket plus its decompress)
    go round-robin to a few CUDA streams, each with its own workspaces and
    payload buffers, so that the latency-bound list stage of one bucket
    overlaps the streaming pass of the next."""

    def __init__(self, torch, nsml, device, nlanes, ws_bytes, aws_bytes, payload_bytes, W, dense_elems, branches=1):
        self.torch = torch
        self.all = []
        for _ in range(nlanes):
            lane = type("Lane", (), {})()
            lane.stream = torch.cuda.Stream(device)
            lane.ws = nsml.alloc_bytes(ws_bytes, device) if ws_bytes else None
            # branches > 1: the compress calls of one job are independent of one another; each gets a stream and a
            # workspace of its own beside the lane's (the job's sum waits for all of them)
            lane.side = [torch.cuda.Stream(device) for _ in range(branches - 1)]
            lane.side_ws = [nsml.alloc_bytes(ws_bytes, device) for _ in range(branches - 1)]
            lane.aws = nsml.alloc_bytes(aws_bytes, device)
            lane.payloads = [nsml.alloc_bytes(payload_bytes, device) for _ in range(W)] if payload_bytes else []
            lane.dense = torch.empty(dense_elems, dtype=torch.float32, device=device)
            self.all.append(lane)
        self.active = nlanes
        self.turn = 0

    def next(self):
        lane = self.all[self.turn % self.active]
        self.turn += 1
        return lane

    def fork(self):
        ev = self.torch.cuda.Event()
        ev.record()
        for lane in self.all:
            lane.stream.wait_event(ev)

    def join(self):
        cur = self.torch.cuda.current_stream()
        for lane in self.all:
            ev = self.torch.cuda.Event()
            ev.record(lane.stream)
            cur.wait_event(ev)


class ResnetWorkload(Workload):
    name = "resnet50: 25.6M fp32 params, 4 buckets of 25 MB, ratio sweep {0.5,0.1,0.01,0.001} x {int8,fp16}, W=1"
    REPLICAS = 9  # 9 x 102 MB of inputs: a replica is reused only after > 400 MB of other inputs
    graph_period = 9

    def __init__(self, nsml, torch, device, rank, nlanes=2):
        import synth

        self.nsml, self.torch = nsml, torch
        self.replicas = []
        for r in range(self.REPLICAS):
            self.replicas.append([torch.from_numpy(b).to(device) for b in synth.resnet50_buckets(seed=1 + r + 100 * rank)])
        self.sizes = [b.numel() for b in self.replicas[0]]
        nmax = max(self.sizes)
        self.lanes = Lanes(torch, nsml, device, nlanes, nsml.nsml_workspace_bytes(nmax),
                           nsml.nsml_accumulate_workspace_bytes(nmax, 1), nsml.nsml_payload_bytes(nmax, 0.5, 16), 1, nmax)
        self.dense = self.lanes.all[0].dense
        self.ctrl = nsml.Controller()
        self.dense_bytes = 4.0 * sum(self.sizes)
        self.input_bytes_per_step = len(SWEEP) * self.dense_bytes
        self.last = (0.0, 0.0)
        self.config = {"workload": self.name, "buckets": len(self.sizes), "bucket_elems": self.sizes,
                       "sweep": [[r, b] for r, b in SWEEP], "W": 1, "streams": nlanes,
                       "l2": "inputs rotate over 9 replicas (920 MB > 126 MB L2)"}

    def before_step(self, i):
        # the controller runs every step (its ratio is reported, the sweep's ratios are the ones compressed with)
        self.ctrl.select_ratio(self.last[0], self.last[1], self.dense_bytes)

    def after_step(self, i, sent):
        self.last = (float(sent), 1e-3 + sent / 1.25e9)  # as if sent over a 10 Gbps link

    def jobs(self, i):
        nsml = self.nsml
        for c, (ratio, bits) in enumerate(SWEEP):
            r = (i * len(SWEEP) + c) % self.REPLICAS
            for b, g in enumerate(self.replicas[r]):
                n = g.numel()

                def enqueue(lane, acc, g=g, n=n, ratio=ratio, bits=bits):
                    p = nsml.nsml_compress(g, ratio, bits, payload=lane.payloads[0], workspace=lane.ws, stream=lane.stream)
                    nsml.nsml_decompress_accumulate([p], lane.dense[:n], zero_first=True, workspace=lane.aws, stream=lane.stream)
                    if acc is not None:
                        k = nsml.nsml_k_of(n, ratio)
                        self.compress_bytes(acc, n, 4, ratio, bits)
                        self.merge_bytes(acc, n, [(k, bits)])

                yield (r, b, ratio, bits), nsml.nsml_payload_bytes(n, ratio, bits), enqueue

    # ---- host-buffer variant for the end-to-end number ----
    def setup_host(self):
        torch, nsml = self.torch, self.nsml
        self.h_grads = [b.cpu().pin_memory() for b in self.replicas[0]]
        nmax = max(self.sizes)
        self.h_payload = torch.empty(nsml.nsml_payload_bytes(nmax, 0.5, 16), dtype=torch.uint8).pin_memory()
        self.h_dense = torch.empty(nmax, dtype=torch.float32).pin_memory()
        dev = self.dense.device
        self.h_scratch_c = nsml.alloc_bytes(nsml.lib.nsml_compress_host_scratch_bytes(nmax, 0, 0.5, 16), dev)
        self.h_scratch_a = nsml.alloc_bytes(
            nsml.lib.nsml_accumulate_host_scratch_bytes(nmax, 1, self.h_payload.numel()), dev)

    def step_host(self, i):
        nsml = self.nsml
        h2d = d2h = 0
        self.ctrl.select_ratio(self.last[0], self.last[1], self.dense_bytes)
        for ratio, bits in SWEEP:
            for g in self.h_grads:
                n = g.numel()
                pb = nsml.nsml_compress_host(g, ratio, bits, self.h_payload, self.h_scratch_c)
                nsml.nsml_decompress_accumulate_host([self.h_payload[:pb]], self.h_dense[:n], True, self.h_scratch_a)
                h2d += 4 * n + pb
                d2h += pb + 4 * n
        return h2d, d2h

    def oracle_sample(self):
        """Two gradient sets (four buckets each) through the whole sweep on the CPU oracle: about 10 s."""
        import oracle

        sets = [[g.cpu().numpy() for g in rep] for rep in self.replicas[:2]]
        t0 = time.perf_counter()
        nbytes = 0.0
        for grads in sets:
            for ratio, bits in SWEEP:
                for g in grads:
                    p = oracle.compress(g, ratio, bits)
                    oracle.decompress_sum([p], g.size)
                    nbytes += 4.0 * g.size
        dt = time.perf_counter() - t0
        return nbytes, dt, (f"{len(sets)} gradient sets ({len(sets[0])} buckets, {sum(g.size for g in sets[0])} elements each) "
                            "through the 8-point ratio x codec sweep")


class Gpt2Workload(Workload):
    name = "gpt2-small: 124M fp32 params, 25M-element buckets, ratio 0.01, int8, W=4 workers summed"
    W, RATIO, BITS = 4, 0.01, 8

    def __init__(self, nsml, torch, device, rank, buckets=None, nlanes=2, ratio=None, bits=None, workers=None):
        import synth

        self.nsml, self.torch = nsml, torch
        if ratio is not None:
            self.RATIO = ratio
        if bits is not None:
            self.BITS = bits
        if workers is not None:
            self.W = workers
        shapes = synth.gpt2_small_shapes()
        total = synth.total_elements(shapes)
        ranges = synth.bucket_ranges(total, 25_000_000)
        if buckets is not None:
            ranges = [ranges[b] for b in buckets]
        gen = torch.Generator(device=device)
        self.workers = []
        for w in range(self.W):
            gen.manual_seed(10 + w + 100 * rank)
            flat = torch.empty(total, dtype=torch.float32, device=device)
            pos = 0
            rs = np.random.default_rng([10 + w, rank])
            for name, shape in shapes:  # same structure as synth: per-tensor sigma, 90 % zero embedding rows
                cnt = synth.numel(shape)
                sigma = 10.0 ** rs.uniform(-4.0, -2.0)
                view = flat[pos:pos + cnt]
                view.normal_(0.0, sigma, generator=gen)
                if name == "wte":
                    rows = torch.rand(shape[0], device=device, generator=gen) < 0.9
                    view.view(shape[0], shape[1])[rows] = 0.0
                pos += cnt
            self.workers.append([flat[lo:hi] for lo, hi in ranges])
        self.sizes = [hi - lo for lo, hi in ranges]
        nmax = max(self.sizes)
        pb = nsml.nsml_payload_bytes(nmax, self.RATIO, self.BITS)
        self.lanes = Lanes(torch, nsml, device, nlanes, nsml.nsml_workspace_bytes(nmax),
                           nsml.nsml_accumulate_workspace_bytes(nmax, self.W), pb, self.W, nmax, branches=self.W)
        self.dense = self.lanes.all[0].dense
        self.ctrl = nsml.Controller()
        self.dense_bytes = 4.0 * sum(self.sizes)
        self.input_bytes_per_step = self.W * self.dense_bytes
        self.last = (0.0, 0.0)
        self.rotate_lanes = True
        self.graph_period = math.lcm(len(self.sizes), nlanes) // len(self.sizes)
        self.config = {"workload": self.name, "buckets": len(self.sizes), "bucket_elems": self.sizes,
                       "ratio": self.RATIO, "bits": self.BITS, "W": self.W, "streams": nlanes,
                       "streams_per_job": self.W,
                       "l2": "inputs are 2 GB per step, far larger than the 126 MB L2"}

    def before_step(self, i):
        self.ctrl.select_ratio(self.last[0], self.last[1], self.dense_bytes)

    def after_step(self, i, sent):
        self.last = (float(sent), 1e-3 + sent / 1.25e9)

    def jobs(self, i):
        nsml = self.nsml
        for b, n in enumerate(self.sizes):
            def enqueue(lane, acc, b=b, n=n):
                # The W workers' buckets are compressed independently of one another (each worker would do it on
                # its own GPU): worker 0 on the job's stream, the others on the lane's side streams, each with a
                # workspace of its own; the sum waits for all of them.  Other buckets run on the other lanes
                # meanwhile.  (The event-bracketed per-kernel pass, acc given, keeps everything on one stream.)
                torch = self.torch
                fan = acc is None and len(lane.side) >= self.W - 1 and self.W > 1
                if fan:
                    start = torch.cuda.Event()
                    start.record(lane.stream)
                ps = []
                for w in range(self.W):
                    st = lane.side[w - 1] if fan and w else lane.stream
                    ws = lane.side_ws[w - 1] if fan and w else lane.ws
                    if fan and w:
                        st.wait_event(start)
                    ps.append(nsml.nsml_compress(self.workers[w][b], self.RATIO, self.BITS, payload=lane.payloads[w],
                                                 workspace=ws, stream=st))
                    if fan and w:
                        done = torch.cuda.Event()
                        done.record(st)
                        lane.stream.wait_event(done)
                nsml.nsml_decompress_accumulate(ps, lane.dense[:n], zero_first=True, workspace=lane.aws, stream=lane.stream)
                if acc is not None:
                    k = nsml.nsml_k_of(n, self.RATIO)
                    for w in range(self.W):
                        self.compress_bytes(acc, n, 4, self.RATIO, self.BITS)
                    self.merge_bytes(acc, n, [(k, self.BITS)] * self.W)

            yield (b,), self.W * nsml.nsml_payload_bytes(n, self.RATIO, self.BITS), enqueue

    HOST_LANES = 3  # streams (each with its own device scratch) the workers' host-buffer calls alternate between

    def setup_host(self):
        torch, nsml = self.torch, self.nsml
        n = self.sizes[0]
        self.h_grads = [self.workers[w][0].cpu().pin_memory() for w in range(self.W)]
        pb = nsml.nsml_payload_bytes(n, self.RATIO, self.BITS)
        self.h_payloads = [torch.empty(pb, dtype=torch.uint8).pin_memory() for _ in range(self.W)]
        self.h_dense = torch.empty(n, dtype=torch.float32).pin_memory()
        dev = self.dense.device
        # The calls are asynchronous on their stream, so a caller overlaps them by giving independent calls
        # their own streams and scratch: while one worker's kernels run, the next worker's gradient is on
        # its way to the device and the previous worker's payload on its way back.
        self.h_lanes = [(torch.cuda.Stream(dev),
                         nsml.alloc_bytes(nsml.lib.nsml_compress_host_scratch_bytes(n, 0, self.RATIO, self.BITS), dev))
                        for _ in range(self.HOST_LANES)]
        self.h_scratch_a = nsml.alloc_bytes(nsml.lib.nsml_accumulate_host_scratch_bytes(n, self.W, self.W * pb), dev)
        self.host_input_bytes = self.W * 4.0 * n  # one bucket per host step
        self.config["e2e_streams"] = self.HOST_LANES

    def step_host(self, i):
        torch, nsml = self.torch, self.nsml
        n = self.sizes[0]
        pb = 0
        cur = torch.cuda.current_stream()
        start = torch.cuda.Event()
        start.record(cur)
        for stream, _ in self.h_lanes:
            stream.wait_event(start)
        for w in range(self.W):
            stream, scratch = self.h_lanes[w % len(self.h_lanes)]
            pb = nsml.nsml_compress_host(self.h_grads[w], self.RATIO, self.BITS, self.h_payloads[w], scratch, stream=stream)
        for stream, _ in self.h_lanes:  # the sum needs every worker's payload back in host memory
            done = torch.cuda.Event()
            done.record(stream)
            cur.wait_event(done)
        nsml.nsml_decompress_accumulate_host(self.h_payloads, self.h_dense, True, self.h_scratch_a)
        return self.W * (4 * n + pb), self.W * pb + 4 * n

    def oracle_sample(self):
        return self.oracle_sample_static()

    @staticmethod
    def oracle_sample_static():
        """The oracle on a bounded sample of this workload: about 10-20 s of one host core."""
        import oracle
        import synth

        n, W = 8_000_000, Gpt2Workload.W
        gs = [synth.gpt2_bucket(2, seed=10 + w)[:n] for w in range(W)]
        t0 = time.perf_counter()
        ps = [oracle.compress(g, Gpt2Workload.RATIO, Gpt2Workload.BITS) for g in gs]
        oracle.decompress_sum(ps, n)
        dt = time.perf_counter() - t0
        return W * 4.0 * n, dt, f"first {n} elements of bucket 2, {W} workers compressed (ratio 0.01, int8) and summed"


class DecoderWorkload(Workload):
    name = "decoder-1.3B: bf16 grads, 64M-element buckets, fp16 values, ratio from the controller on a 100/10/1 Gbps trace"
    dtype = "bf16"
    graphs_ok = False  # the controller emits a new ratio every step

    def __init__(self, nsml, torch, device, rank, nlanes=2):
        import synth

        self.nsml, self.torch = nsml, torch
        shapes = synth.decoder_1p3b_shapes()
        total = synth.total_elements(shapes)
        gen = torch.Generator(device=device)
        gen.manual_seed(20 + 100 * rank)
        flat = torch.empty(total, dtype=torch.bfloat16, device=device)
        rs = np.random.default_rng([20, rank])
        pos = 0
        for name, shape in shapes:
            cnt = synth.numel(shape)
            sigma = 10.0 ** rs.uniform(-6.0, -2.0)
            flat[pos:pos + cnt].normal_(0.0, sigma, generator=gen)
            pos += cnt
        self.buckets = [flat[lo:hi] for lo, hi in synth.bucket_ranges(total, 1 << 26)]
        self.sizes = [b.numel() for b in self.buckets]
        nmax = max(self.sizes)
        self.lanes = Lanes(torch, nsml, device, nlanes, nsml.nsml_workspace_bytes(nmax, nsml.NSML_BF16),
                           nsml.nsml_accumulate_workspace_bytes(nmax, 1), nsml.nsml_payload_bytes(nmax, 0.1, 16), 1, nmax)
        self.dense = self.lanes.all[0].dense
        # the configuration asks for ratios from 0.1 down to 0.001: the floor is lowered from the paper's 0.005
        self.ctrl = nsml.Controller(ratio_init=0.1, ratio_min=0.001, ratio_max=0.1, startup_max_steps=0)
        self.dense_bytes = 2.0 * total
        self.input_bytes_per_step = self.dense_bytes
        self.last = (0.0, 0.0)
        self.ratios = []
        self.config = {"workload": self.name, "buckets": len(self.sizes), "bucket_elems": self.sizes[0], "W": 1,
                       "controller": {"ratio_init": 0.1, "ratio_min": 0.001, "ratio_max": 0.1}, "streams": nlanes,
                       "l2": "inputs are 2.6 GB per step"}

    def before_step(self, i):
        self.ratio = self.ctrl.select_ratio(self.last[0], self.last[1], self.dense_bytes)
        self.ratios.append(self.ratio)

    def after_step(self, i, sent):
        bw = (100e9, 10e9, 1e9)[min(2, i // 30)] / 8.0  # bytes/s of the synthetic link
        self.last = (float(sent), 1e-3 + sent / bw)

    def jobs(self, i):
        nsml = self.nsml
        ratio = self.ratio
        for b, g in enumerate(self.buckets):
            n = g.numel()

            def enqueue(lane, acc, g=g, n=n, ratio=ratio):
                p = nsml.nsml_compress(g, ratio, 16, payload=lane.payloads[0], workspace=lane.ws, stream=lane.stream)
                nsml.nsml_decompress_accumulate([p], lane.dense[:n], zero_first=True, workspace=lane.aws, stream=lane.stream)
                if acc is not None:
                    k = nsml.nsml_k_of(n, ratio)
                    self.compress_bytes(acc, n, 2, ratio, 16)
                    self.merge_bytes(acc, n, [(k, 16)])

            yield (b, ratio), nsml.nsml_payload_bytes(n, ratio, 16), enqueue

    def setup_host(self):
        torch, nsml = self.torch, self.nsml
        n = self.sizes[0]
        self.h_grad = self.buckets[0].cpu().pin_memory()
        self.h_payload = torch.empty(nsml.nsml_payload_bytes(n, 0.1, 16), dtype=torch.uint8).pin_memory()
        self.h_dense = torch.empty(n, dtype=torch.float32).pin_memory()
        dev = self.dense.device
        self.h_scratch_c = nsml.alloc_bytes(nsml.lib.nsml_compress_host_scratch_bytes(n, 1, 0.1, 16), dev)
        self.h_scratch_a = nsml.alloc_bytes(nsml.lib.nsml_accumulate_host_scratch_bytes(n, 1, self.h_payload.numel()), dev)
        self.host_input_bytes = 2.0 * n

    def step_host(self, i):
        nsml = self.nsml
        n = self.sizes[0]
        pb = nsml.nsml_compress_host(self.h_grad, 0.01, 16, self.h_payload, self.h_scratch_c)
        nsml.nsml_decompress_accumulate_host([self.h_payload[:pb]], self.h_dense, True, self.h_scratch_a)
        return 2 * n + pb, pb + 4 * n

    def oracle_sample(self):
        import oracle

        n = 8_000_000
        bits16 = self.buckets[5][:n].view(self.torch.int16).cpu().numpy().view(np.uint16)
        t0 = time.perf_counter()
        p = oracle.compress(oracle.widen_bf16(bits16), 0.01, 16)
        oracle.decompress_sum([p], n)
        dt = time.perf_counter() - t0
        return 2.0 * n, dt, f"first {n} bf16 elements of bucket 5 at ratio 0.01, fp16 values"


class Bf16BucketWorkload(Workload):
    """Buckets of the largest configuration's size and type, at one fixed ratio: where a pass over a bucket is
    long enough for the memory system to reach its steady state."""

    name = "decoder-1.3B shapes: three 64M-element bf16 buckets, ratio 0.01, fp16 values, W=1"
    dtype = "bf16"
    RATIO, BITS, N, BUCKETS = 0.01, 16, 1 << 26, 3
    has_host = False

    def __init__(self, nsml, torch, device, rank, nlanes=2):
        self.nsml, self.torch = nsml, torch
        gen = torch.Generator(device=device)
        gen.manual_seed(700 + rank)
        rs = np.random.default_rng([700, rank])
        self.buckets = []
        for _ in range(self.BUCKETS):  # four tensors of 16M elements each, per-tensor sigma log-uniform [1e-6, 1e-2]
            g = torch.empty(self.N, dtype=torch.bfloat16, device=device)
            for t in range(4):
                g[t * (self.N // 4):(t + 1) * (self.N // 4)].normal_(0.0, 10.0 ** rs.uniform(-6.0, -2.0), generator=gen)
            self.buckets.append(g)
        n = self.N
        self.lanes = Lanes(torch, nsml, device, nlanes, nsml.nsml_workspace_bytes(n, nsml.NSML_BF16),
                           nsml.nsml_accumulate_workspace_bytes(n, 1), nsml.nsml_payload_bytes(n, self.RATIO, self.BITS), 1, n)
        self.dense = self.lanes.all[0].dense
        self.sizes = [n] * self.BUCKETS
        self.input_bytes_per_step = 2.0 * n * self.BUCKETS
        self.rotate_lanes = True  # three independent jobs per step: the next step's start on the idle lanes
        self.graph_period = math.lcm(self.BUCKETS, nlanes) // self.BUCKETS
        self.config = {"workload": self.name, "buckets": self.BUCKETS, "bucket_elems": n, "ratio": self.RATIO,
                       "bits": self.BITS, "W": 1, "streams": nlanes, "l2": "inputs are 384 MB per step"}

    def jobs(self, i):
        nsml, n = self.nsml, self.N
        for b, g in enumerate(self.buckets):
            def enqueue(lane, acc, g=g):
                p = nsml.nsml_compress(g, self.RATIO, self.BITS, payload=lane.payloads[0], workspace=lane.ws, stream=lane.stream)
                nsml.nsml_decompress_accumulate([p], lane.dense, zero_first=True, workspace=lane.aws, stream=lane.stream)
                if acc is not None:
                    self.compress_bytes(acc, n, 2, self.RATIO, self.BITS)
                    self.merge_bytes(acc, n, [(nsml.nsml_k_of(n, self.RATIO), self.BITS)])

            yield (b,), nsml.nsml_payload_bytes(n, self.RATIO, self.BITS), enqueue


class AggWorkload(Workload):
    name = "aggregation stress: W=8 int8 payloads (ratio 0.05) for one dense bucket (350M elements unless --agg-elements), decompress + sum only"
    W, N, RATIO = 8, 350_000_000, 0.05

    def __init__(self, nsml, torch, device, rank, nlanes=1):
        import synth

        self.nsml, self.torch = nsml, torch
        self.k = nsml.nsml_k_of(self.N, self.RATIO)
        self.payloads = []
        for w in range(self.W):
            idx, codes, scales = synth.stress_payload_parts(self.N, self.k, 30 + w + 100 * rank, shared_seed=99)
            self.payloads.append(torch.from_numpy(nsml.pack_payload(self.N, 8, idx, codes=codes, scales=scales)).to(device))
        self.lanes = Lanes(torch, nsml, device, 1, 0, nsml.nsml_accumulate_workspace_bytes(self.N, self.W), 0, 0, self.N)
        self.aws, self.dense = self.lanes.all[0].aws, self.lanes.all[0].dense
        self.input_bytes_per_step = 4.0 * self.N  # the dense gradient this step reconstructs
        self.config = {"workload": self.name, "n": self.N, "k": self.k, "W": self.W,
                       "l2": "payloads 700 MB + dense 1.4 GB per step"}

    def jobs(self, i):
        def enqueue(lane, acc):
            self.nsml.nsml_decompress_accumulate(self.payloads, lane.dense, zero_first=True, workspace=lane.aws, stream=lane.stream)
            if acc is not None:
                self.merge_bytes(acc, self.N, [(self.k, 8)] * self.W)

        yield (0,), sum(p.numel() for p in self.payloads), enqueue

    def setup_host(self):
        torch, nsml = self.torch, self.nsml
        self.h_payloads = [p.cpu().pin_memory() for p in self.payloads]
        self.h_dense = torch.empty(self.N, dtype=torch.float32).pin_memory()
        total = sum(p.numel() for p in self.h_payloads)
        self.h_scratch_a = nsml.alloc_bytes(nsml.lib.nsml_accumulate_host_scratch_bytes(self.N, self.W, total), self.dense.device)
        self.host_input_bytes = 4.0 * self.N

    def step_host(self, i):
        self.nsml.nsml_decompress_accumulate_host(self.h_payloads, self.h_dense, True, self.h_scratch_a)
        return sum(p.numel() for p in self.h_payloads), 4 * self.N

    def oracle_sample(self):
        import oracle
        import synth

        n, k = 35_000_000, 1_750_000
        ps = []
        for w in range(self.W):
            idx, codes, scales = synth.stress_payload_parts(n, k, 30 + w, shared_seed=99)
            ps.append(oracle.Payload(n=n, k=k, bits=8, idx=idx, raw=np.zeros(0, np.float32), codes=codes, scales=scales))
        t0 = time.perf_counter()
        oracle.decompress_sum(ps, n)
        dt = time.perf_counter() - t0
        return 4.0 * n, dt, f"the same payload recipe at one tenth of the size (n={n}, k={k}, W=8)"


class Alg2Workload(Workload):
    """The whole of Alg. 2 per bucket, with the local accumulation of Section 4.2 Step 3: L2 norm of the gradient
    (Step 1; enqueued, not waited for), pruning mask from the weights at the step's ratio (Step 2), compress of
    gradient + residual under that mask (Step 3), and the receiver's decompress + sum (W = 1)."""

    name = "alg2: 25M-element fp32 buckets, L2 norm + pruning mask from weights + compress with local accumulation (ratio 0.01, int8) + sum, W=1"
    RATIO, BITS, N = 0.01, 8, 25_000_000
    GRADS, STATE = 8, 4  # gradient buckets and weight / residual buffers the steps rotate over (100 MB each)
    has_host = False     # no host-buffer entry points for these steps
    graph_period = 8

    def __init__(self, nsml, torch, device, rank, nlanes=2):
        self.nsml, self.torch = nsml, torch
        n = self.N
        gen = torch.Generator(device=device)
        gen.manual_seed(500 + rank)
        rs = np.random.default_rng([500, rank])
        self.grads = []
        for _ in range(self.GRADS):  # a bucket = 50 equal "tensors", per-tensor sigma log-uniform [1e-4, 1e-2]
            g = torch.empty(n, dtype=torch.float32, device=device)
            for t in range(50):
                g[t * (n // 50):(t + 1) * (n // 50)].normal_(0.0, 10.0 ** rs.uniform(-4.0, -2.0), generator=gen)
            self.grads.append(g)
        self.weights = [torch.empty(n, dtype=torch.float32, device=device).normal_(0.0, 0.02, generator=gen)
                        for _ in range(self.STATE)]
        self.residual = [torch.zeros(n, dtype=torch.float32, device=device) for _ in range(self.STATE)]
        self.lanes = Lanes(torch, nsml, device, nlanes, nsml.nsml_workspace_bytes(n), nsml.nsml_accumulate_workspace_bytes(n, 1),
                           nsml.nsml_payload_bytes(n, self.RATIO, self.BITS), 1, n)
        for lane in self.lanes.all:
            lane.side = [torch.cuda.Stream(device)]  # the norm runs beside the mask build
            lane.l2ws = nsml.alloc_bytes(nsml.lib.nsml_l2_workspace_bytes(), device)
            lane.pws = nsml.alloc_bytes(nsml.nsml_prune_workspace_bytes(n), device)
            lane.mask = torch.empty((n + 31) // 32, dtype=torch.int32, device=device)
        self.dense = self.lanes.all[0].dense
        self.sizes = [n] * self.STATE
        self.input_bytes_per_step = 4.0 * n * self.STATE
        self.config = {"workload": self.name, "buckets": self.STATE, "bucket_elems": self.sizes, "ratio": self.RATIO,
                       "bits": self.BITS, "W": 1, "streams": nlanes,
                       "l2": "gradients rotate over 8 buckets (800 MB), weights and residuals over 4 each"}

    def jobs(self, i):
        nsml, n = self.nsml, self.N
        k = nsml.nsml_k_of(n, self.RATIO)
        for b in range(self.STATE):
            def enqueue(lane, acc, b=b, g=self.grads[(i * self.STATE + b) % self.GRADS]):
                # Step 1 reads the gradient, Step 2 the weights: they run side by side (the norm on the lane's side
                # stream), Step 3 waits for both.  (The event-bracketed per-kernel pass keeps one stream.)
                torch = self.torch
                fan = acc is None and len(lane.side) >= 1
                if fan:
                    start = torch.cuda.Event()
                    start.record(lane.stream)
                    lane.side[0].wait_event(start)
                nsml.nsml_grad_l2(g, workspace=lane.l2ws, stream=lane.side[0] if fan else lane.stream, sync=False)
                nsml.nsml_prune_mask_build(self.weights[b], self.RATIO, prune_mask=lane.mask, workspace=lane.pws,
                                           stream=lane.stream)
                if fan:
                    done = torch.cuda.Event()
                    done.record(lane.side[0])
                    lane.stream.wait_event(done)
                p = nsml.nsml_compress_feedback(g, self.residual[b], self.RATIO, self.BITS, prune_mask=lane.mask,
                                                payload=lane.payloads[0], workspace=lane.ws, stream=lane.stream)
                nsml.nsml_decompress_accumulate([p], lane.dense, zero_first=True, workspace=lane.aws, stream=lane.stream)
                if acc is not None:
                    self.account(acc, "k_sumsq", 4 * n)
                    # mask build in two passes (sampled window); the four-pass kernels behind them leave at once
                    self.account(acc, "k_prune_sample", 4 * 8192)
                    self.account(acc, "k_prune_count", 4 * n)
                    self.account(acc, "k_prune_settle", 4 * 4096)
                    self.account(acc, "k_prune_mark", 4 * n + n // 8)
                    self.account(acc, "k_prune_fix", 8 * 1024)
                    self.account(acc, "k_feedback_subtract", 13 * k)
                    self.compress_bytes(acc, n, 4, self.RATIO, self.BITS)
                    # the bucket pass also reads the mask and the residual and writes gradient + residual back
                    self.account(acc, "k_compact_bucket", n // 8 + 8 * n)
                    self.merge_bytes(acc, n, [(k, self.BITS)])

            yield ((i * self.STATE + b) % self.GRADS, b), nsml.nsml_payload_bytes(n, self.RATIO, self.BITS), enqueue

    def oracle_sample(self):
        import oracle

        n = 4_000_000
        g = self.grads[0][:n].cpu().numpy()
        w = self.weights[0][:n].cpu().numpy()
        r = np.zeros(n, dtype=np.float32)
        t0 = time.perf_counter()
        oracle.l2_norm(g)
        mask = oracle.prune_mask(w, self.RATIO)
        p, r = oracle.error_feedback_step(g, r, self.RATIO, self.BITS, mask)
        oracle.decompress_sum([p], n)
        dt = time.perf_counter() - t0
        return 4.0 * n, dt, f"first {n} elements of one bucket: L2 norm, mask, compress with residual, sum"


WORKLOADS = {"resnet50": ResnetWorkload, "gpt2": Gpt2Workload, "decoder": DecoderWorkload, "agg": AggWorkload,
             "alg2": Alg2Workload}


# --------------------------------------------------------------------------
# measurement helpers
# --------------------------------------------------------------------------
def per_kernel_table(nsml, torch, wl, peak, steps, first_step=0, traffic=None):
    """Per-kernel device time of `steps` steps with every launch bracketed by CUDA events on its stream
    (one stream, eager), beside the algorithmic bytes the workload's accounting gives each kernel.  Event
    brackets add a few microseconds to a launch, so the fractions are lower bounds."""
    acc = {}
    nsml.nsml_prof_reset()
    nsml.nsml_prof_enable(True)
    active = wl.lanes.active
    wl.lanes.active = 1  # one stream: a kernel's events then bracket that kernel alone
    for i in range(steps):
        wl.step(first_step + i, acc)
    torch.cuda.synchronize()
    wl.lanes.active = active
    prof = nsml.nsml_prof_read()
    nsml.nsml_prof_enable(False)
    table = {}
    for name, (ms, cnt) in prof.items():
        if cnt:
            nbytes = acc.get(name, 0) / cnt
            gbs = nbytes / (1e-3 * ms / cnt) / 1e9 if ms > 0 else 0.0
            table[name] = {"launches_per_step": cnt / steps, "us_per_launch": 1e3 * ms / cnt, "ms_per_step": ms / steps,
                           "algorithmic_bytes_per_launch": nbytes, "algorithmic_GBps": gbs, "frac_of_measured": gbs / peak,
                           "frac_of_nominal_8TBps": gbs / 8000.0, "traffic": (traffic or {}).get(name)}
    return table


def timed_steps(torch, wl, steps, first_step):
    """Device time in ms of `steps` steps (all streams forked from and joined to the current one)."""
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    wl.lanes.fork()
    for i in range(steps):
        wl.step(first_step + i)
    wl.lanes.join()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1)


def whole_step(table, ms_per_step, peak):
    """The step as one unit: the algorithmic bytes of all its launches (per-kernel table) over the device time
    of the step as it is timed (all streams)."""
    nbytes = sum(k["algorithmic_bytes_per_launch"] * k["launches_per_step"] for k in table.values())
    gbs = nbytes / (ms_per_step * 1e-3) / 1e9
    return {"algorithmic_bytes_per_step": nbytes, "ms_per_step": ms_per_step, "algorithmic_GBps": gbs,
            "frac_of_measured": gbs / peak, "frac_of_nominal_8TBps": gbs / 8000.0}


def run_leg(nsml, torch, wl, peak, use_graphs, traffic=None, steps=10):
    """A further workload measured inside the default run: device time of `steps` steps, then the per-kernel table."""
    wl.init_graphs(use_graphs)
    warm = max(3, wl.graph_period if wl.use_graphs else 3)
    wl.lanes.fork()
    for i in range(warm):
        wl.step(i)
    wl.lanes.join()
    torch.cuda.synchronize()
    ms = timed_steps(torch, wl, steps, warm) / steps
    table = per_kernel_table(nsml, torch, wl, peak, 5, traffic=traffic)
    return {"workload": wl.name, "value": wl.input_bytes_per_step / (ms * 1e-3) / 1e9, "unit": UNIT, "ms_per_step": ms,
            "whole_step": whole_step(table, ms, peak), "per_kernel": table}


def serial_compress(nsml, torch, grad, ratio, bits, ws, payload, esize, peak, reps=30, restore_candidates=4096):
    """One nsml_compress at a time on one stream, back to back: what a caller that compresses a single bucket (the
    last bucket of a backward pass, say) gets.  The algorithmic bytes of the call are one read of the bucket plus
    the payload written."""
    n = grad.numel()
    nsml.nsml_set_list_block_candidates(2048)  # the setting for a call that has the GPU to itself (default 4096: 3 us more)
    for _ in range(5):
        nsml.nsml_compress(grad, ratio, bits, payload=payload, workspace=ws)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        nsml.nsml_compress(grad, ratio, bits, payload=payload, workspace=ws)
    e1.record()
    torch.cuda.synchronize()
    nsml.nsml_set_list_block_candidates(restore_candidates)
    us = 1e3 * e0.elapsed_time(e1) / reps
    nbytes = esize * n + nsml.nsml_payload_bytes(n, ratio, bits)
    gbs = nbytes / (us * 1e-6) / 1e9
    return {"us_per_call": us, "algorithmic_bytes": nbytes, "algorithmic_GBps": gbs, "frac_of_measured": gbs / peak,
            "frac_of_nominal_8TBps": gbs / 8000.0, "n": n, "ratio": ratio, "bits": bits,
            "list_block_candidates": 2048,
            "note": "one call at a time on one stream, eager launches; the same bucket every time, so a bucket that "
                    "fits the 126 MB L2 is partly served from it"}


def exchange_leg(nsml, torch, dist, device, rank, world, steps, warm=3):
    """The data-parallel exchange of one 25M-element bucket per rank (Section 5.3: top-k payloads travel by
    AllGather; Alg. 1 is fed the measured transfer): every rank compresses its bucket at the ratio rank 0's
    controller picked, the payloads are all-gathered (NCCL copies the peers' payloads into local memory; no
    kernel of this library reads a peer's memory), every rank sums the `world` payloads.  Times are device
    times per phase, MAX over ranks."""
    from paper_2506_16235_b200 import dp

    n, bits = 25_000_000, 8
    gen = torch.Generator(device=device)
    gen.manual_seed(900 + rank)
    grads = []
    for r in range(3):  # three buckets rotate: 300 MB > L2
        g = torch.empty(n, dtype=torch.float32, device=device)
        rs = np.random.default_rng([900, rank, r])
        for t in range(50):
            g[t * (n // 50):(t + 1) * (n // 50)].normal_(0.0, 10.0 ** rs.uniform(-4.0, -2.0), generator=gen)
        grads.append(g)
    # a fixed ratio keeps every step's payload the same size; the controller still runs and is fed the measured
    # all-gather, and its ratio is reported
    ratio = 0.01
    ctrl = nsml.Controller()
    ws = nsml.alloc_bytes(nsml.nsml_workspace_bytes(n), device)
    aws = nsml.alloc_bytes(nsml.nsml_accumulate_workspace_bytes(n, world), device)
    payload = nsml.alloc_bytes(nsml.nsml_payload_bytes(n, ratio, bits), device)
    dense = torch.empty(n, dtype=torch.float32, device=device)
    sums = [0.0, 0.0, 0.0]
    last = (0.0, 0.0)
    ctrl_ratio = None
    for i in range(warm + steps):
        ctrl_ratio, phases, last = dp.exchange_round(
            ctrl, last, 4.0 * n * world,
            lambda _r, i=i: nsml.nsml_compress(grads[i % 3], ratio, bits, payload=payload, workspace=ws),
            lambda views: nsml.nsml_decompress_accumulate(views, dense, zero_first=True, workspace=aws, sized=True),
            on_cuda=True)
        if i >= warm:
            for j in range(3):
                sums[j] += phases[j]
    status = nsml.nsml_last_status(aws)
    ms = [x / steps for x in sums]
    total = sum(ms)
    return {"workload": f"exchange: one 25M-element fp32 bucket per rank, ratio {ratio}, int8, all-gather of {world} payloads, sum",
            "value": world * 4.0 * n / (total * 1e-3) / 1e9, "unit": UNIT, "ms_per_step": total,
            "ms_compress": ms[0], "ms_all_gather": ms[1], "ms_sum": ms[2], "payload_bytes": int(nsml.nsml_payload_bytes(n, ratio, bits)),
            "all_gather_GBps_per_rank": (world - 1) * nsml.nsml_payload_bytes(n, ratio, bits) / (ms[1] * 1e-3) / 1e9 if world > 1 else None,
            "controller_ratio_after": ctrl_ratio, "status": status}


# --------------------------------------------------------------------------
# reference arm: the CPU oracle, timed as it stands
# --------------------------------------------------------------------------
def run_reference(args, rank):
    """The oracle as it stands on the host cores, on a bounded sample of the default workload per step: the
    first `--reference-elements` elements of one 25M-element bucket of the GPT-2-shaped gradient set, compressed
    for each of the 4 workers (ratio 0.01, int8) and summed."""
    if rank != 0:
        return
    import oracle
    import synth

    n = int(args.reference_elements or 2_000_000)
    W, ratio, bits = Gpt2Workload.W, Gpt2Workload.RATIO, Gpt2Workload.BITS
    gs = [synth.gpt2_bucket(2, seed=10 + w)[:n] for w in range(W)]

    def one(i):
        ps = [oracle.compress(g, ratio, bits) for g in gs]
        oracle.decompress_sum(ps, n)

    for i in range(args.warmup):
        one(i)
    t0 = time.perf_counter()
    for i in range(args.steps):
        one(i)
    dt = time.perf_counter() - t0
    value = args.steps * W * 4.0 * n / dt / 1e9
    sample = f"first {n} elements of bucket 2, {W} workers compressed (ratio {ratio}, int8) and summed, per step"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": Gpt2Workload.name, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


# --------------------------------------------------------------------------
# main arm
# --------------------------------------------------------------------------
def spawn_ranks(args):
    """`python bench.py --gpus N` with N > 1, not started by torchrun: start the N ranks here."""
    import socket
    import subprocess

    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    raise SystemExit(subprocess.call(cmd))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--workload", default="gpt2", choices=sorted(WORKLOADS))
    ap.add_argument("--impl", default="nsml", choices=["nsml", "reference"])
    ap.add_argument("--streams", type=int, default=8, help="CUDA streams that independent buckets alternate between")
    ap.add_argument("--list-block-candidates", type=int, default=None,
                    help="nsml_set_list_block_candidates (library default: 4096); default here: 8192 for the workloads "
                         "with many calls in flight (gpt2, decoder), 4096 for the others")
    ap.add_argument("--no-graphs", action="store_true", help="launch every call eagerly instead of replaying CUDA graphs")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-legs", action="store_true", help="skip the further workloads measured inside the default run")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (e2e is then null)")
    ap.add_argument("--no-kernel-times", action="store_true", help="skip the event-bracketed per-kernel pass")
    ap.add_argument("--reference-elements", type=int, default=None,
                    help="--impl reference only: elements of the bucket the oracle is timed on per step (default 2M)")
    ap.add_argument("--agg-elements", type=int, default=None,
                    help="agg workload only: dense elements (default 350M; smaller sizes are for profiler captures)")
    ap.add_argument("--exchange", action="store_true",
                    help="time the exchange leg on one GPU as well (one payload: the same code path as with N ranks)")
    ap.add_argument("--buckets", type=int, default=None,
                    help="gpt2 workload only: use the first this many buckets (smaller sets are for profiler captures)")
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    if args.impl == "reference":
        args.steps = args.steps or 8
        args.warmup = 1 if args.warmup is None else args.warmup
        run_reference(args, rank)
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        spawn_ranks(args)
    if world != args.gpus:
        raise SystemExit(f"bench.py: --gpus {args.gpus} but {world} rank(s) were started")

    import torch

    import paper_2506_16235_b200 as nsml

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    if torch.cuda.device_count() <= local_rank:
        raise SystemExit(f"bench.py: rank {rank} needs GPU {local_rank} but only {torch.cuda.device_count()} are visible")
    defaults = {"resnet50": (100, 5), "gpt2": (50, 5), "decoder": (90, 3), "agg": (50, 3), "alg2": (20, 8)}[args.workload]
    steps = args.steps or defaults[0]
    warmup_requested = defaults[1] if args.warmup is None else args.warmup
    warmup = max(3, warmup_requested)

    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod

        dist = dist_mod
        dist.init_process_group("nccl", device_id=device)

    if args.workload == "agg" and args.agg_elements:
        AggWorkload.N = int(args.agg_elements)
    kwargs = {}
    if args.workload == "gpt2" and args.buckets:
        kwargs["buckets"] = list(range(args.buckets))
    # several buckets in flight: the list stage takes more candidates per block (fewer SMs held while it waits
    # for memory); the one-call-at-a-time measurement below goes back to the library's default
    if args.list_block_candidates is None:
        args.list_block_candidates = 8192 if args.workload in ("gpt2", "decoder") else 4096
    nsml.nsml_set_list_block_candidates(args.list_block_candidates)
    wl = WORKLOADS[args.workload](nsml, torch, device, rank, nlanes=max(1, args.streams), **kwargs)
    wl.config["list_block_candidates"] = args.list_block_candidates
    wl.init_graphs(not args.no_graphs)
    if wl.use_graphs:
        warmup = max(warmup, wl.graph_period)  # every job has been captured before the timed region starts
    wl.config["cuda_graphs"] = bool(wl.use_graphs)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing ----
    wl.lanes.fork()
    for i in range(warmup):
        wl.step(i)
    wl.lanes.join()
    barrier()
    launches0, replayed0 = nsml.nsml_launch_count(), wl.replayed_launches
    with ClockSampler(local_rank) as clocks:
        elapsed_ms = timed_steps(torch, wl, steps, warmup)
    launches = nsml.nsml_launch_count() - launches0 + wl.replayed_launches - replayed0
    barrier()
    if dist is not None:
        t = torch.tensor([elapsed_ms], device=device, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        elapsed_ms = float(t.item())
    value = world * steps * wl.input_bytes_per_step / (elapsed_ms * 1e-3) / 1e9

    # ---- per-kernel device time (further steps, every launch bracketed by CUDA events) ----
    peak, peak_kind = measured_peak_gbs()
    kernels, roofline = {}, None
    traffic_key = {"gpt2": "gpt2_25M", "agg": "agg_350M"}.get(args.workload)
    if not args.no_kernel_times:
        kernels = per_kernel_table(nsml, torch, wl, peak, max(1, min(steps, 10)), warmup + steps,
                                   traffic=ncu_traffic(traffic_key) if traffic_key else None)
        dominant = max(kernels, key=lambda k: kernels[k]["ms_per_step"])
        d = kernels[dominant]
        roofline = {"bound": "hbm", "kernel": dominant, "achieved": d["algorithmic_GBps"], "peak": peak,
                    "peak_kind": f"of {peak_kind}", "unit": "GB/s", "frac": d["algorithmic_GBps"] / peak,
                    "frac_of_nominal_8TBps": d["algorithmic_GBps"] / 8000.0, "traffic": d["traffic"],
                    "us_per_launch": d["us_per_launch"], "algorithmic_bytes_per_launch": d["algorithmic_bytes_per_launch"],
                    "how": "achieved = algorithmic_bytes_per_launch / us_per_launch (CUDA events around every launch, one "
                           "stream); the dominant kernel is the one with the most device time per step",
                    "whole_step": whole_step(kernels, elapsed_ms / steps, peak),
                    "per_kernel": kernels}
        if rank == 0 and args.workload == "gpt2":
            g = wl.workers[0][-2] if len(wl.workers[0]) > 1 else wl.workers[0][0]
            roofline["one_compress_call"] = serial_compress(nsml, torch, g, wl.RATIO, wl.BITS, wl.lanes.all[0].ws,
                                                            wl.lanes.all[0].payloads[0], 4, peak,
                                                            restore_candidates=args.list_block_candidates)

    # ---- end to end through the host-buffer entry points ----
    e2e = None
    if not args.no_e2e and getattr(wl, "has_host", True):
        wl.setup_host()
        host_steps = max(1, min(steps, 5))
        for i in range(2):
            wl.step_host(i)
        torch.cuda.synchronize()
        hv0, hv1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        hv0.record()
        h2d = d2h = 0
        for i in range(host_steps):
            h2d, d2h = wl.step_host(i)
        hv1.record()
        torch.cuda.synchronize()
        host_ms = hv0.elapsed_time(hv1)
        if dist is not None:
            t = torch.tensor([host_ms], device=device, dtype=torch.float64)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            host_ms = float(t.item())
        host_bytes = getattr(wl, "host_input_bytes", wl.input_bytes_per_step)
        e2e = {"value": world * host_steps * host_bytes / (host_ms * 1e-3) / 1e9, "unit": UNIT,
               "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h), "steps": host_steps,
               "ms_per_step": host_ms / host_steps}

    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": warmup,
        "warmup_requested": warmup_requested, "ms_per_step": elapsed_ms / steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": wl.dtype, "data": "synthetic", "config": wl.config,
        "clocks": clocks.summary(), "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline,
    }

    # ---- the exchange between ranks (N > 1; at N = 1 the same code path with one payload) ----
    if world > 1 or args.exchange:
        out["exchange"] = exchange_leg(nsml, torch, dist, device, rank, world, steps=10)

    # ---- further workloads (one GPU, default workload only) ----
    if rank == 0 and world == 1 and args.workload == "gpt2" and not args.no_legs:
        legs = {}
        nl, graphs = max(1, args.streams), not args.no_graphs
        del wl
        torch.cuda.empty_cache()
        # (key, workload, candidates per list-stage block: the legs with few calls in flight keep the library's default)
        for key, make, candidates in (
            ("ratio_0.1_25M", lambda: Gpt2Workload(nsml, torch, device, rank, buckets=[2, 3], nlanes=nl, ratio=0.1, workers=2),
             args.list_block_candidates),
            ("ratio_0.001_25M", lambda: Gpt2Workload(nsml, torch, device, rank, buckets=[2, 3], nlanes=nl, ratio=0.001, workers=2),
             args.list_block_candidates),
            ("bf16_64M", lambda: Bf16BucketWorkload(nsml, torch, device, rank, nlanes=nl), args.list_block_candidates),
            ("alg2_25M", lambda: Alg2Workload(nsml, torch, device, rank, nlanes=nl), 4096),
            ("resnet50_sweep", lambda: ResnetWorkload(nsml, torch, device, rank, nlanes=nl), 4096),
        ):
            nsml.nsml_set_list_block_candidates(candidates)
            leg_wl = make()
            if key.startswith("ratio_"):
                leg_wl.name = f"two 25M-element fp32 buckets, ratio {leg_wl.RATIO}, int8, W=2 workers each"
            legs[key] = run_leg(nsml, torch, leg_wl, peak, graphs)
            legs[key]["list_block_candidates"] = candidates
            del leg_wl
            torch.cuda.empty_cache()
        out["legs"] = legs
        wl = None

    if rank == 0 and not args.no_cpu_baseline:
        nbytes, dt, sample = Gpt2Workload.oracle_sample_static() if wl is None else wl.oracle_sample()
        out["cpu_baseline"] = {"value": nbytes / dt / 1e9, "unit": UNIT, "cores": 1, "kind": "oracle",
                               "sample": sample, "seconds": dt, "host_cores": os.cpu_count()}
    if rank == 0:
        print(json.dumps(out))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
