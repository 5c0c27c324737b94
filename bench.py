#!/usr/bin/env python
"""Throughput of the boundary-tensor codec on one or more B200s (one process per GPU).

A step is one pass of the whole hot path over one boundary tensor: accept_compress (range,
quantize, pack) followed by accept_decompress (unpack, dequantize) of the stream just written.
The metric is GB/s of fp32 input through that round trip; compress and decompress are also
reported on their own, each with its achieved fraction of the measured HBM copy bandwidth.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--sweep]
    python bench.py --impl reference ...      # the CPU oracle on the host cores

The headline (`value`) is the round trip on --workload (cfg4_hidden by default): the median over --repeats
blocks of exactly K back-to-back steps each.  On one GPU the line also carries, under "workloads", one
row per tensor of 100 MB or more in its headline modes (cfg3 forward and backward, cfg4, the 256 MB and
1 GB points of the size sweep) with both kernels timed inside the step and in loops of their own, and under
"small" the tensors of 16 MB and less replayed from CUDA graphs next to an empty kernel launched the same way.

With N > 1 (launched under torch.distributed.run) every rank codes its own replica of the tensor;
the codec has no exchange step, so there is no data-path collective (weak scaling).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

import workloads

METRIC = "compress+decompress round-trip throughput of fp32 boundary tensor"
UNIT = "GB/s of fp32 input"
DEFAULT_WORKLOAD = "cfg4_hidden"
L2_BYTES = 126 << 20
FALLBACK_HBM_GBS = 6650.0


def mode_name(m) -> str:
    return "k%d-%s-%s-%s" % (m.k, "absmax" if m.range == 0 else "minmax", "nearest" if m.round == 0 else "stochastic",
                             "interleaved" if m.layout == 0 else "bitplane")


def algorithmic_bytes(n: int, chunk: int, k: int) -> float:
    """Bytes the method must move per call, either direction: 4 + k/8 + 8/C per element."""
    return n * (4.0 + k / 8.0 + 8.0 / chunk)


def kernel_sources_digest(files=None) -> str:
    """Digest of CUDA sources (all of csrc/, or the named files of it) and of the build recipe: ncu counters stored
    under profiles/ are quoted only for the kernels they were taken from."""
    import hashlib
    h = hashlib.sha256()
    pkg = os.path.join(ROOT, "paper_2311_05827_b200")
    csrc = os.path.join(pkg, "csrc")
    names = sorted(files) if files else sorted(n for n in os.listdir(csrc) if n.endswith((".cu", ".cuh")))
    for name in names:
        with open(os.path.join(csrc, name), "rb") as f:
            h.update(name.encode() + b"\0" + f.read())
    with open(os.path.join(pkg, "build.py"), "rb") as f:
        h.update(b"build.py\0" + f.read())
    return h.hexdigest()[:16]


def recorded_traffic(workload: str, entry_point: str):
    """DRAM bytes per launch (ncu dram__bytes_read.sum + dram__bytes_write.sum) from profiles/traffic.json, or
    None when there is no capture of this kernel on this workload or one of the sources the row names (the files
    the captured kernel is compiled from) has changed since."""
    try:
        with open(os.path.join(ROOT, "profiles", "traffic.json")) as f:
            table = json.load(f)
        row = table["captures"][workload][entry_point]
        if row["sources_digest"] != kernel_sources_digest(row["sources"]):
            return None
        return float(row["dram_bytes_per_launch"])
    except Exception:
        return None


def recorded_instructions(workload: str, kernel: str):
    """Executed thread-instructions per element of an instruction-bound kernel (ncu smsp__inst_executed.sum x 32 / n)
    from profiles/traffic.json, under the same rule as recorded_traffic; None if not captured or changed since."""
    try:
        with open(os.path.join(ROOT, "profiles", "traffic.json")) as f:
            row = json.load(f)["instructions"][workload][kernel]
        if row["sources_digest"] != kernel_sources_digest(row["sources"]):
            return None
        return float(row["thread_instructions_per_element"])
    except Exception:
        return None


# Issue rate of a B200: 148 SMs x 4 schedulers x one warp instruction of 32 lanes per cycle, at the SM clock.
def issue_peak_per_second(sm_mhz: float) -> float:
    return 148 * 4 * 32 * sm_mhz * 1e6


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# --------------------------------------------------------------------------------------------- clocks

class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.out = None

    def start(self):
        try:
            self.out = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS, "--format=csv,noheader,nounits",
                 "-lms", "20"], stdout=self.out, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.out.flush()
        self.out.seek(0)
        sm, smax, reasons = [], [], set()
        for line in self.out.read().splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                smax.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        self.out.close()
        os.unlink(self.out.name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(smax)), "reasons": sorted(reasons),
                "samples": len(sm)}


# --------------------------------------------------------------------------------------------- GPU arm

class Codec:
    """Device buffers for one (tensor, mode): enough rotating copies that a step never finds its
    inputs in L2."""

    def __init__(self, A, torch, x_host: np.ndarray, chunk: int, mode, seed: int, min_footprint: int = 3 * L2_BYTES):
        self.A, self.torch = A, torch
        n = x_host.size
        self.n, self.chunk, self.mode = n, chunk, mode
        self.p = A.Params(n, chunk, mode.k, mode.range, mode.round, mode.layout, seed, 0)
        self.stream_bytes = A.accept_compressed_size(self.p)
        per_set = 8 * n + self.stream_bytes
        self.copies = int(max(2, min(4096, -(-min_footprint // per_set))))
        x0 = torch.from_numpy(x_host).cuda()
        self.x = [x0] + [x0.clone() for _ in range(self.copies - 1)]
        self.stream = [torch.empty(self.stream_bytes, dtype=torch.uint8, device="cuda") for _ in range(self.copies)]
        self.xhat = [torch.empty(n, dtype=torch.float32, device="cuda") for _ in range(self.copies)]
        self.ws = A.new_workspace(self.p)
        self.calls = 0

    def step(self, i: int):
        A, j = self.A, i % self.copies
        A.accept_compress(self.p, self.x[j], self.stream[j], self.ws)
        A.accept_decompress(self.p, self.stream[j], self.xhat[j], self.ws)
        self.calls += 2

    def run(self, steps: int, warmup: int):
        """-> (ms per step, ms per compress, ms per decompress), device-timed.  The step time comes from
        one pair of events around `steps` back-to-back steps; the per-kernel times inside a step from a
        second pass with an event between the kernels (each recorded event costs the stream a microsecond
        or two, which is why the two are not taken in the same pass)."""
        torch = self.torch
        for i in range(warmup):
            self.step(i)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(steps):
            self.step(warmup + i)
        e1.record()
        torch.cuda.synchronize()
        total = e0.elapsed_time(e1)
        # one event before the first kernel and one after every kernel: the end of a step is the start of the next
        edge = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
        mid = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
        A = self.A
        edge[0].record()
        for i in range(steps):
            j = (warmup + steps + i) % self.copies
            A.accept_compress(self.p, self.x[j], self.stream[j], self.ws)
            mid[i].record()
            A.accept_decompress(self.p, self.stream[j], self.xhat[j], self.ws)
            edge[i + 1].record()
        self.calls += 2 * steps
        torch.cuda.synchronize()
        tc = sum(edge[i].elapsed_time(mid[i]) for i in range(steps)) / steps
        td = sum(mid[i].elapsed_time(edge[i + 1]) for i in range(steps)) / steps
        return total / steps, tc, td

    def run_blocks(self, steps: int, repeats: int):
        """`repeats` blocks of exactly `steps` back-to-back steps, one pair of events round each block:
        -> ms per step of every block."""
        torch = self.torch
        out = []
        for r in range(repeats):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for i in range(steps):
                self.step(r * steps + i)
            e1.record()
            torch.cuda.synchronize()
            out.append(e0.elapsed_time(e1) / steps)
        return out

    def run_isolated_blocks(self, steps: int, repeats: int, warmup: int = 3):
        """Each kernel in loops of its own: -> (ms per compress of every block, ms per decompress of every block)."""
        torch, A = self.torch, self.A
        out = []
        for fn in (lambda j: A.accept_compress(self.p, self.x[j], self.stream[j], self.ws),
                   lambda j: A.accept_decompress(self.p, self.stream[j], self.xhat[j], self.ws)):
            for i in range(warmup):
                fn(i % self.copies)
            torch.cuda.synchronize()
            blocks = []
            for r in range(repeats):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                for i in range(steps):
                    fn((r * steps + i) % self.copies)
                e1.record()
                torch.cuda.synchronize()
                blocks.append(e0.elapsed_time(e1) / steps)
            self.calls += warmup + steps * repeats
            out.append(blocks)
        return out[0], out[1]

    def run_isolated(self, steps: int, warmup: int = 3):
        """Each kernel in a loop of its own (rotating buffers): -> (ms per compress, ms per decompress).
        Inside a step the compress kernel also pays for the write-back of the dirty output lines the
        previous decompress left in L2; these loops charge every kernel with its own traffic only."""
        torch, A = self.torch, self.A
        out = []
        for fn in (lambda j: A.accept_compress(self.p, self.x[j], self.stream[j], self.ws),
                   lambda j: A.accept_decompress(self.p, self.stream[j], self.xhat[j], self.ws)):
            for i in range(warmup):
                fn(i % self.copies)
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for i in range(steps):
                fn((warmup + i) % self.copies)
            e1.record()
            torch.cuda.synchronize()
            out.append(e0.elapsed_time(e1) / steps)
            self.calls += steps + warmup
        return out[0], out[1]

    def run_graphed(self, launches: int = 64, replays: int = 10, warm: bool = False):
        """Small tensors are bound by the host's launch rate when timed call by call.  Here `launches`
        calls of each kernel are captured into a CUDA graph and the graph is replayed:
        -> (ms per compress, ms per decompress) as the device sees them, launch gaps included.
        Cold (default): the calls rotate over enough buffer sets that none finds its data in L2;
        warm: every call works on the same buffers, which then stay in L2."""
        torch, A = self.torch, self.A
        out = []
        side = torch.cuda.Stream()
        pick = (lambda j: 0) if warm else (lambda j: j)
        for fn in (lambda j: A.accept_compress(self.p, self.x[pick(j)], self.stream[pick(j)], self.ws, side),
                   lambda j: A.accept_decompress(self.p, self.stream[pick(j)], self.xhat[pick(j)], self.ws, side)):
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                fn(0)  # first call outside the capture
                side.synchronize()
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph, stream=side):
                    for i in range(launches):
                        fn(i % self.copies)
                graph.replay()
                side.synchronize()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(side)
                for _ in range(replays):
                    graph.replay()
                e1.record(side)
                side.synchronize()
            out.append(e0.elapsed_time(e1) / (replays * launches))
            self.calls += launches * (replays + 1) + 1
        torch.cuda.current_stream().wait_stream(side)
        return out[0], out[1]

    def copy_graphed(self, launches: int = 64, replays: int = 10) -> float:
        """ms per plain device copy of the fp32 tensor (4n bytes read, 4n written; a copy node of the graph),
        captured and replayed like run_graphed over the same rotating buffers: what the GPU itself needs to
        move a tensor of this size once, for the small tensors whose calls are not bound by bytes."""
        torch = self.torch
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            self.xhat[0].copy_(self.x[0])
            side.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=side):
                for i in range(launches):
                    self.xhat[i % self.copies].copy_(self.x[i % self.copies])
            graph.replay()
            side.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(side)
            for _ in range(replays):
                graph.replay()
            e1.record(side)
            side.synchronize()
        torch.cuda.current_stream().wait_stream(side)
        return e0.elapsed_time(e1) / (replays * launches)

    def status(self) -> int:
        return self.A.accept_last_device_status(self.ws)


E2E_LANES = 4  # streams the host-buffer leg alternates between


def e2e_run(A, torch, x_host, chunk, mode, seed, steps, warmup, lanes=E2E_LANES):
    """Round trip through the host-buffer entry points: pinned host tensor in, stream to the host,
    stream back to the device, reconstructed tensor to the host; all copies inside the timed region.
    Consecutive steps alternate between `lanes` CUDA streams, each with its own staging buffers, so
    that one step's device-to-host copies overlap the next step's host-to-device copies (PCIe is
    full duplex); every step still moves all of its bytes."""
    n = x_host.size
    p = A.Params(n, chunk, mode.k, mode.range, mode.round, mode.layout, seed, 0)
    sb = A.accept_compressed_size(p)
    h_x = torch.from_numpy(x_host).pin_memory()

    class Lane:
        def __init__(self):
            self.stream = torch.cuda.Stream()
            self.h_stream = torch.empty(sb, dtype=torch.uint8).pin_memory()
            self.h_xhat = torch.empty(n, dtype=torch.float32).pin_memory()
            self.d_x = torch.empty(n, dtype=torch.float32, device="cuda")
            self.d_xhat = torch.empty(n, dtype=torch.float32, device="cuda")
            self.d_stream, self.d_ws = A.new_stream_buffer(p), A.new_workspace(p)

    lane = [Lane() for _ in range(lanes)]
    torch.cuda.synchronize()

    def one(i):
        L = lane[i % lanes]
        A.accept_compress_host(p, h_x, L.h_stream, L.d_x, L.d_stream, L.d_ws, L.stream)
        A.accept_decompress_host(p, L.h_stream, L.h_xhat, L.d_stream, L.d_xhat, L.d_ws, L.stream)

    for i in range(warmup * lanes):
        one(i)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    main = torch.cuda.current_stream()
    e0.record(main)
    for L in lane:
        L.stream.wait_event(e0)
    for i in range(steps):
        one(i)
    for L in lane:
        main.wait_stream(L.stream)
    e1.record(main)
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    for L in lane:
        assert A.accept_last_device_status(L.d_ws) == 0
    return ms, 4 * n + sb, sb + 4 * n


def time_oracle(x_host, chunk, mode, seed, budget_s=10.0, max_reps=50):
    """The CPU oracle, as it stands, single-threaded, on x_host: seconds per round trip."""
    import oracle
    reps, t0 = 0, time.perf_counter()
    tc = td = 0.0
    while True:
        a = time.perf_counter()
        stream, _ = oracle.compress(x_host, chunk, mode.k, mode.range, mode.round, mode.layout, seed, 0)
        b = time.perf_counter()
        oracle.decompress(stream, x_host.size)
        c = time.perf_counter()
        tc += b - a
        td += c - b
        reps += 1
        if time.perf_counter() - t0 >= budget_s or reps >= max_reps:
            break
    return tc / reps, td / reps, reps


def time_oracle_all_cores(x_host, chunk, mode, seed, reps=3):
    """The same oracle over disjoint chunk ranges, one thread per host core (ctypes calls drop the GIL):
    (seconds per round trip, threads).  Each slice becomes a stream of its own; counters continue across slices."""
    import oracle
    from concurrent.futures import ThreadPoolExecutor
    cores = len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else (os.cpu_count() or 1)
    n_chunks = -(-x_host.size // chunk)
    per = -(-n_chunks // cores) * chunk
    slices = [(lo, min(lo + per, x_host.size)) for lo in range(0, x_host.size, per)]

    def one(bounds):
        lo, hi = bounds
        stream, _ = oracle.compress(x_host[lo:hi], chunk, mode.k, mode.range, mode.round, mode.layout, seed, lo)
        oracle.decompress(stream, hi - lo)

    with ThreadPoolExecutor(max_workers=len(slices)) as pool:
        list(pool.map(one, slices))          # untimed: loads the library, touches the pages
        t0 = time.perf_counter()
        for _ in range(reps):
            list(pool.map(one, slices))
        dt = (time.perf_counter() - t0) / reps
    return dt, len(slices)


def max_over_ranks(values, dist, device):
    """Element-wise maximum of per-rank timings (the slowest rank defines the job's time)."""
    import torch
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.tolist()]


def job_throughput(n_elems_per_rank: int, world: int, ms: float) -> float:
    """GB/s of fp32 input over all ranks: every rank codes its own replica in the same (max) time."""
    return world * 4.0 * n_elems_per_rank / (ms * 1e-3) / 1e9


def spread(values) -> dict:
    v = sorted(float(t) for t in values)
    return {"median": float(np.median(v)), "min": v[0], "max": v[-1], "blocks": len(v)}


def generate_on_all_cores(name: str) -> np.ndarray:
    """The whole tensor, its blocks drawn on one thread per host core (numpy's generators drop the interpreter lock)."""
    from concurrent.futures import ThreadPoolExecutor
    n, step = workloads.TENSORS[name].n, 1 << 22
    cores = len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else (os.cpu_count() or 1)
    with ThreadPoolExecutor(max_workers=max(1, cores)) as pool:
        parts = list(pool.map(lambda s0: workloads.generate(name, s0, min(step, n - s0)), range(0, n, step)))
    return np.concatenate(parts) if len(parts) > 1 else parts[0]


def kernel_figures(n: int, alg: float, us_in_step: float, us_alone: dict, peak: float) -> dict:
    """One kernel of a row: microseconds inside the step and in a loop of its own, GB/s of fp32, and the
    algorithmic bytes over the time as a fraction of the measured copy bandwidth and of 8 TB/s."""
    gbs = lambda nbytes, us: nbytes / (us * 1e-6) / 1e9
    return {"us_in_step": us_in_step, "us_alone": us_alone,
            "gbs_fp32_in_step": gbs(4 * n, us_in_step), "gbs_fp32_alone": gbs(4 * n, us_alone["median"]),
            "frac_of_measured_in_step": gbs(alg, us_in_step) / peak, "frac_of_measured_alone": gbs(alg, us_alone["median"]) / peak,
            "frac_of_8TBs_in_step": gbs(alg, us_in_step) / 8000.0, "frac_of_8TBs_alone": gbs(alg, us_alone["median"]) / 8000.0}


def measure_row(A, torch, name: str, mode, x_host, steps: int, repeats: int, warmup: int, peak: float):
    """compress + decompress of one tensor in one mode: `repeats` blocks of `steps` steps, then each kernel
    between events inside the step, then each kernel in loops of its own.  -> (row, codec)."""
    spec = workloads.TENSORS[name]
    codec = Codec(A, torch, x_host, spec.chunk, mode, spec.seed)
    for i in range(warmup):
        codec.step(i)
    torch.cuda.synchronize()
    before = A.accept_launch_count()
    step_ms = codec.run_blocks(steps, repeats)
    launches = (A.accept_launch_count() - before) // repeats
    _, ms_c, ms_d = codec.run(steps, 0)
    iso_c, iso_d = codec.run_isolated_blocks(steps, repeats)
    assert codec.status() == 0
    alg = algorithmic_bytes(spec.n, spec.chunk, mode.k)
    step_us = spread(1e3 * t for t in step_ms)
    row = {"workload": name, "mode": mode_name(mode), "mbytes": spec.n * 4 / 2 ** 20, "buffer_sets": codec.copies,
           "algorithmic_bytes_per_launch": alg, "step_us": step_us,
           "step_gbs_fp32": 4 * spec.n / (step_us["median"] * 1e-6) / 1e9,
           "step_frac_of_measured": 2 * alg / (step_us["median"] * 1e-6) / 1e9 / peak,
           "step_frac_of_8TBs": 2 * alg / (step_us["median"] * 1e-6) / 1e9 / 8000.0,
           "compress": kernel_figures(spec.n, alg, 1e3 * ms_c, spread(1e3 * t for t in iso_c), peak),
           "decompress": kernel_figures(spec.n, alg, 1e3 * ms_d, spread(1e3 * t for t in iso_d), peak),
           "launches_per_block": launches}
    return row, codec


def small_rows(A, torch, peak: float):
    """Tensors of 16 MB and less: the time of a call is set by launching, not by bytes.  Each kernel is
    replayed from a CUDA graph of 64 calls over rotating buffers (cold) next to an EMPTY kernel of the same
    grid launched the same way (same launch attribute, same graph): the floor.  What is left above the
    floor is set against the time the algorithmic bytes take at the measured copy bandwidth.  Beside them the
    time of a plain device copy of the same fp32 tensor (a copy node in the same kind of graph), which moves
    8n bytes where a codec call moves about 4n + kn/8: what a transfer of this size costs without any codec."""
    rows = []
    for name in ("cfg1_act", "cfg2_grad", "cfg5_64KB", "cfg5_1MB", "cfg5_16MB"):
        spec = workloads.TENSORS[name]
        x_host = workloads.generate(name)
        for mode in spec.headline:
            codec = Codec(A, torch, x_host, spec.chunk, mode, spec.seed)
            g_c, g_d = codec.run_graphed()
            g_copy = codec.copy_graphed()
            blocks = -(-spec.n // 4096)
            floor_c, floor_d = null_graph_ms(A, torch, blocks, 128), null_graph_ms(A, torch, blocks, 256)
            alg = algorithmic_bytes(spec.n, spec.chunk, mode.k)
            bytes_us = alg / peak / 1e3  # microseconds the bytes take at the measured copy bandwidth
            rows.append({"workload": name, "mode": mode_name(mode), "kbytes": spec.n * 4 / 1024,
                         "bytes_us_at_measured_copy": bytes_us,
                         "compress_us_graph": 1e3 * g_c, "decompress_us_graph": 1e3 * g_d,
                         "plain_copy_us_graph": 1e3 * g_copy,
                         "empty_kernel_us_graph": {"blocks": blocks, "threads_128": 1e3 * floor_c, "threads_256": 1e3 * floor_d},
                         "compress_us_above_floor": 1e3 * (g_c - floor_c), "decompress_us_above_floor": 1e3 * (g_d - floor_d),
                         "compress_frac_of_measured": bytes_us / (1e3 * g_c), "decompress_frac_of_measured": bytes_us / (1e3 * g_d)})
            assert codec.status() == 0
            del codec
            torch.cuda.empty_cache()
    return rows


def null_graph_ms(A, torch, blocks: int, threads: int, launches: int = 64, replays: int = 10) -> float:
    """ms per launch of the library's empty kernel, captured and replayed like Codec.run_graphed."""
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        A.accept_launch_null(blocks, threads, side)
        side.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            for _ in range(launches):
                A.accept_launch_null(blocks, threads, side)
        graph.replay()
        side.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(side)
        for _ in range(replays):
            graph.replay()
        e1.record(side)
        side.synchronize()
    torch.cuda.current_stream().wait_stream(side)
    return e0.elapsed_time(e1) / (replays * launches)


# tensors of 100 MB or more besides the headline workload, each in its headline modes
LARGE_ROWS = ("cfg3_act", "cfg3_grad", "cfg5_256MB", "cfg5_1GB")


def run_gpu(args):
    import torch
    import paper_2311_05827_b200 as A
    from paper_2311_05827_b200 import build as lib_build
    lib_build.build()

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the codec has no CPU path")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    spec = workloads.TENSORS[args.workload]
    mode = (spec.headline + spec.also)[args.mode_index]
    x_host = generate_on_all_cores(args.workload)
    n = spec.n
    peak, peak_src = measured_peak()

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local_rank)
    barrier()
    sampler.start()
    head, codec = measure_row(A, torch, args.workload, mode, x_host, args.steps, args.repeats, args.warmup, peak)
    barrier()
    # the slowest rank defines the job: per block, then the median over blocks
    ms_step = max_over_ranks([head["step_us"]["median"] * 1e-3], dist, "cuda")[0]
    ms_c, ms_d = max_over_ranks([head["compress"]["us_in_step"] * 1e-3, head["decompress"]["us_in_step"] * 1e-3], dist, "cuda")
    iso_c, iso_d = max_over_ranks([head["compress"]["us_alone"]["median"] * 1e-3,
                                   head["decompress"]["us_alone"]["median"] * 1e-3], dist, "cuda")
    launches_timed = head["launches_per_block"]

    rows, small = [head], []
    if world == 1 and not args.kernels_only and not args.headline_only:
        for name in LARGE_ROWS:
            if name == args.workload:
                continue
            xr = generate_on_all_cores(name)
            for m in workloads.TENSORS[name].headline:
                row, c = measure_row(A, torch, name, m, xr, args.steps, args.repeats, args.warmup, peak)
                rows.append(row)
                del c
                torch.cuda.empty_cache()
            del xr
        small = small_rows(A, torch, peak)
    clocks = sampler.stop()
    if clocks.get("sm_mhz"):
        for row in rows:
            row["step_mcycles"] = row["step_us"]["median"] * clocks["sm_mhz"] * 1e-6  # time x median SM clock

    # end to end through host buffers
    e2e_steps = max(4, min(args.steps, 12))
    if args.kernels_only:
        ms_e2e, h2d, d2h = float("nan"), 0, 0
    else:
        ms_e2e, h2d, d2h = e2e_run(A, torch, x_host, spec.chunk, mode, spec.seed, e2e_steps, 1)
    ms_e2e = max_over_ranks([ms_e2e], dist, "cuda")[0]

    alg = algorithmic_bytes(n, spec.chunk, mode.k)
    gbs = lambda nbytes, ms: nbytes / (ms * 1e-3) / 1e9
    dominant = "accept_compress" if ms_c >= ms_d else "accept_decompress"
    ms_dom = max(ms_c, ms_d)
    out = {
        "metric": METRIC, "value": job_throughput(n, world, ms_step), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": args.workload, "shape": list(spec.shape), "n_elems": n, "chunk": spec.chunk,
                   "mode": mode_name(mode), "l2": "inputs larger than L2 and %d rotating buffer sets" % codec.copies,
                   "parallelism": "replicas only" if world > 1 else "single GPU",
                   "timing": "median of %d blocks of exactly %d back-to-back steps, CUDA events round each block" % (args.repeats, args.steps)},
        "ms_per_step_blocks": {k: (v * 1e-3 if k != "blocks" else v) for k, v in head["step_us"].items()},
        "step_hbm": {"algorithmic_bytes": 2 * alg, "gbs": gbs(2 * alg, ms_step), "frac_of_measured_copy": gbs(2 * alg, ms_step) / peak,
                     "frac_of_8TBs": gbs(2 * alg, ms_step) / 8000.0},
        "roofline": {"bound": "hbm", "kernel": dominant, "achieved": gbs(alg, ms_dom), "peak": peak, "peak_source": peak_src,
                     "unit": "GB/s", "frac": gbs(alg, ms_dom) / peak, "traffic": recorded_traffic(args.workload, dominant),
                     # the same kernel in a loop of its own: inside a step it also pays for the write-back of the dirty
                     # lines its predecessor left in L2 (the step as a whole is in step_hbm)
                     "achieved_alone": gbs(alg, iso_c if dominant == "accept_compress" else iso_d),
                     "frac_alone": gbs(alg, iso_c if dominant == "accept_compress" else iso_d) / peak},
        "e2e": {"value": job_throughput(n, world, ms_e2e), "unit": UNIT, "ms_per_step": ms_e2e, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "streams": E2E_LANES, "steps": e2e_steps},
        "gpu_launches": launches_timed,
        "clocks": clocks,
        "workloads": rows,
    }
    if small:
        out["small"] = small

    if args.sweep and rank == 0:
        out["sweep"] = sweep(A, torch, peak, args)
    if args.all_modes and rank == 0:
        out["all_modes"] = sweep_all_modes(A, torch, peak)

    if rank == 0 and world == 1 and not (args.no_cpu_baseline or args.kernels_only):
        tc, td, reps = time_oracle(x_host, spec.chunk, mode, spec.seed, budget_s=args.cpu_budget)
        out["cpu_baseline"] = {"value": 4 * n / (tc + td) / 1e9, "unit": UNIT, "cores": 1, "kind": "oracle",
                               "sample": "whole %s tensor (%d elements), %d round trips; compress %.3f s, decompress %.3f s each"
                                         % (args.workload, n, reps, tc, td),
                               "host_cores_available": os.cpu_count()}
        t_all, threads = time_oracle_all_cores(x_host, spec.chunk, mode, spec.seed)
        out["cpu_baseline"]["all_cores"] = {"value": 4 * n / t_all / 1e9, "unit": UNIT, "cores": threads,
                                            "sample": "the same tensor split into %d contiguous chunk ranges, one thread each, "
                                                      "3 round trips" % threads}
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(out))


def sweep(A, torch, peak, args):
    """All five workloads, headline modes: per-kernel time and HBM fraction."""
    rows = []
    for name, spec in workloads.TENSORS.items():
        if spec.n * 4 > args.sweep_max_bytes or (args.sweep_only and name != args.sweep_only):
            continue
        x_host = workloads.generate(name)
        for mode in spec.headline:
            codec = Codec(A, torch, x_host, spec.chunk, mode, spec.seed)
            steps = 20 if spec.n * 4 >= (64 << 20) else 200
            ms_c, ms_d = codec.run_isolated(steps)
            assert codec.status() == 0
            alg = algorithmic_bytes(spec.n, spec.chunk, mode.k)
            rows.append({"workload": name, "mode": mode_name(mode), "mbytes": spec.n * 4 / 2 ** 20, "copies": codec.copies,
                         "compress_ms": ms_c, "decompress_ms": ms_d,
                         "compress_gbs_fp32": 4 * spec.n / ms_c / 1e6, "decompress_gbs_fp32": 4 * spec.n / ms_d / 1e6,
                         "compress_frac_measured": alg / ms_c / 1e6 / peak, "decompress_frac_measured": alg / ms_d / 1e6 / peak,
                         "compress_frac_8TBs": alg / ms_c / 1e6 / 8000.0, "decompress_frac_8TBs": alg / ms_d / 1e6 / 8000.0})
            note = ""
            if spec.n * 4 < (64 << 20):
                g_c, g_d = codec.run_graphed()
                rows[-1].update({"compress_ms_graph": g_c, "decompress_ms_graph": g_d,
                                 "compress_frac_measured_graph": alg / g_c / 1e6 / peak,
                                 "decompress_frac_measured_graph": alg / g_d / 1e6 / peak})
                w_c, w_d = codec.run_graphed(warm=True)
                rows[-1].update({"compress_ms_graph_warm": w_c, "decompress_ms_graph_warm": w_d})
                note = "   in a CUDA graph: c %.4f ms %5.1f%%  d %.4f ms %5.1f%%; warm (same buffers, L2 resident): c %.4f ms  d %.4f ms" % (
                    g_c, 100 * alg / g_c / 1e6 / peak, g_d, 100 * alg / g_d / 1e6 / peak, w_c, w_d)
            print("# %-12s %-34s c %8.4f ms %6.1f%%  d %8.4f ms %6.1f%% (of measured copy bw)%s" %
                  (name, mode_name(mode), ms_c, 100 * rows[-1]["compress_frac_measured"], ms_d,
                   100 * rows[-1]["decompress_frac_measured"], note), file=sys.stderr)
            del codec
            torch.cuda.empty_cache()
        if name in ("cfg3_grad", "cfg4_hidden"):
            rows.append(sweep_per_tensor(A, torch, peak, name, spec, x_host))
        if name == "cfg3_grad":  # the paper's backward encoder: stochastic codes packed along the batch dimension
            rows.append(sweep_batch_groups(A, torch, peak, name, spec, x_host))
        if name == "cfg3_act":
            rows.extend(sweep_mbq(A, torch, peak, name, spec, x_host))
            rows.append(sweep_batch_groups(A, torch, peak, name, spec, x_host))
            # eight bit planes, and values per sample that are not a multiple of eight (the feature-per-thread kernels)
            rows.append(sweep_batch_groups(A, torch, peak, name, spec, x_host, mode=workloads.Mode(8, 0, 0, 1)))
            rows.append(sweep_batch_groups(A, torch, peak, name, spec, x_host, stride=spec.n // spec.shape[0] - 4))
    return rows


def sweep_all_modes(A, torch, peak, name="cfg5_256MB"):
    """Every layout / k / range statistic / rounding combination the consecutive layouts have (28), at chunk sizes
    4096 (four warps share a chunk) and 1024 (one warp per chunk), on the 256 MB tensor: isolated loops."""
    spec = workloads.TENSORS[name]
    x_host = workloads.generate(name)
    rows = []
    for layout in (0, 1):
        for k in ((2, 4, 8) if layout == 0 else (2, 3, 4, 8)):
            for range_ in (0, 1):
                for round_ in (0, 1):
                    for chunk in (4096, 1024):
                        mode = workloads.Mode(k, range_, round_, layout)
                        codec = Codec(A, torch, x_host, chunk, mode, spec.seed)
                        ms_c, ms_d = codec.run_isolated(20)
                        assert codec.status() == 0
                        alg = algorithmic_bytes(spec.n, chunk, k)
                        rows.append({"workload": name, "mode": mode_name(mode), "chunk": chunk, "compress_ms": ms_c,
                                     "decompress_ms": ms_d, "compress_frac_measured": alg / ms_c / 1e6 / peak,
                                     "decompress_frac_measured": alg / ms_d / 1e6 / peak})
                        print("# %-12s %-34s C=%-5d c %8.4f ms %6.1f%%  d %8.4f ms %6.1f%% (of measured copy bw)" %
                              (name, mode_name(mode), chunk, ms_c, 100 * rows[-1]["compress_frac_measured"], ms_d,
                               100 * rows[-1]["decompress_frac_measured"]), file=sys.stderr)
                        del codec
                        torch.cuda.empty_cache()
    return rows


def sweep_batch_groups(A, torch, peak, name, spec, x_host, mode=None, stride=None):
    """Pack groups along the batch dimension (the paper's grouping): the tensor as batch x (values per sample).
    stride: values per sample if not the tensor's own (the first batch x stride values are coded then)."""
    mode = mode or spec.headline[0]
    stride = stride or spec.n // spec.shape[0]
    n = spec.shape[0] * stride
    x_host = x_host[:n]
    p = A.Params(n, spec.chunk, mode.k, mode.range, mode.round, mode.layout, spec.seed, 0, group_stride=stride)
    copies = 2
    x = [torch.from_numpy(x_host).cuda() for _ in range(copies)]
    st = [A.new_stream_buffer(p) for _ in range(copies)]
    xh = [torch.empty(n, dtype=torch.float32, device="cuda") for _ in range(copies)]
    ws = A.new_workspace(p)
    times = []
    for fn in (lambda j: A.accept_compress(p, x[j], st[j], ws), lambda j: A.accept_decompress(p, st[j], xh[j], ws)):
        for i in range(3):
            fn(i % copies)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(20):
            fn(i % copies)
        e1.record()
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1) / 20)
    assert A.accept_last_device_status(ws) == 0
    ms_c, ms_d = times
    alg_c, alg_d = n * (8.0 + mode.k / 8.0), n * (4.0 + mode.k / 8.0)
    row = {"workload": name, "mode": mode_name(mode) + "-batch-groups", "mbytes": n * 4 / 2 ** 20, "copies": copies,
           "group_stride": stride, "compress_ms": ms_c, "decompress_ms": ms_d, "compress_bytes_per_element": 8.0 + mode.k / 8.0,
           "compress_frac_measured": alg_c / ms_c / 1e6 / peak, "decompress_frac_measured": alg_d / ms_d / 1e6 / peak}
    print("# %-12s %-34s c %8.4f ms %6.1f%%  d %8.4f ms %6.1f%% (of measured copy bw)" %
          (name, ("k%d%s-batch-groups-%dx%d" % (mode.k, "bp" if mode.layout else "il", spec.shape[0], stride))[:34], ms_c, 100 * row["compress_frac_measured"],
           ms_d, 100 * row["decompress_frac_measured"]), file=sys.stderr)
    return row


def sweep_per_tensor(A, torch, peak, name, spec, x_host):
    """The paper's granularity: one range for the whole tensor (two passes over the input, 8 + k/8 B/element)."""
    mode = spec.headline[0]
    chunk = (spec.n + 31) // 32 * 32
    codec = Codec(A, torch, x_host, chunk, mode, spec.seed)
    ms_c, ms_d = codec.run_isolated(20)
    assert codec.status() == 0
    alg_c, alg_d = spec.n * (8.0 + mode.k / 8.0), spec.n * (4.0 + mode.k / 8.0)
    row = {"workload": name, "mode": mode_name(mode) + "-one-range", "mbytes": spec.n * 4 / 2 ** 20, "copies": codec.copies,
           "compress_ms": ms_c, "decompress_ms": ms_d, "compress_frac_measured": alg_c / ms_c / 1e6 / peak,
           "decompress_frac_measured": alg_d / ms_d / 1e6 / peak, "compress_bytes_per_element": 8.0 + mode.k / 8.0}
    print("# %-12s %-34s c %8.4f ms %6.1f%%  d %8.4f ms %6.1f%% (of measured copy bw)" %
          (name, row["mode"][:34], ms_c, 100 * row["compress_frac_measured"], ms_d, 100 * row["decompress_frac_measured"]),
          file=sys.stderr)
    return row


def sweep_mbq(A, torch, peak, name, spec, x_host):
    """The forward quantizer (multi-bit quantization): residue initialisation, encode + coefficient update, decode."""
    rows = []
    n = spec.n
    for k in (2, 3, 4):
        p0, p1 = A.MbqParams(n, k, 0, True), A.MbqParams(n, k, 1, False)
        copies = 2
        x = [torch.from_numpy(x_host).cuda() for _ in range(copies)]
        st = [A.new_stream_buffer(p0) for _ in range(copies)]
        xh = [torch.empty(n, dtype=torch.float32, device="cuda") for _ in range(copies)]
        ws, alpha = A.new_workspace(p0), torch.zeros(k, dtype=torch.float32, device="cuda")

        def timed(fn, steps=20, warm=3):
            for i in range(warm):
                fn(i % copies)
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for i in range(steps):
                fn(i % copies)
            e1.record()
            torch.cuda.synchronize()
            return e0.elapsed_time(e1) / steps

        ms_i = timed(lambda j: A.accept_mbq_compress(p0, x[j], None, alpha, st[j], ws), steps=5, warm=1)
        ms_c = timed(lambda j: A.accept_mbq_compress(p1, x[j], alpha, alpha, st[j], ws))
        ms_d = timed(lambda j: A.accept_mbq_decompress(p1, st[j], xh[j], ws))
        assert A.accept_last_device_status(ws) == 0
        alg = n * (4.0 + k / 8.0)
        rows.append({"workload": name, "mode": "mbq-k%d" % k, "mbytes": n * 4 / 2 ** 20, "copies": copies,
                     "init_ms": ms_i, "compress_ms": ms_c, "decompress_ms": ms_d,
                     "compress_frac_measured": alg / ms_c / 1e6 / peak, "decompress_frac_measured": alg / ms_d / 1e6 / peak})
        # the encode pass is bound by instruction issue, not by HBM: its second roofline is the issue rate of the
        # SMs at the nominal maximum clock, with the instruction count of the ncu capture
        ipe = recorded_instructions(name, "mbq_encode_kernel<%d>" % k)
        if ipe is not None:
            achieved = ipe * n / (ms_c * 1e-3)
            rows[-1]["compress_roofline_alu"] = {"bound": "alu", "unit": "thread-instructions/s", "achieved": achieved,
                                                 "peak": issue_peak_per_second(1965.0), "frac": achieved / issue_peak_per_second(1965.0),
                                                 "thread_instructions_per_element": ipe}
        print("# %-12s %-34s c %8.4f ms %6.1f%%  d %8.4f ms %6.1f%% (of measured copy bw); residue init %.4f ms" %
              (name, "mbq-k%d" % k, ms_c, 100 * rows[-1]["compress_frac_measured"], ms_d,
               100 * rows[-1]["decompress_frac_measured"], ms_i), file=sys.stderr)
        del x, st, xh
        torch.cuda.empty_cache()
    return rows


# --------------------------------------------------------------------------------------------- reference arm

def run_reference(args):
    """The CPU oracle on the host cores, same metric and workload; rank 0 only."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import oracle
    oracle.build()
    spec = workloads.TENSORS[args.workload]
    mode = spec.headline[0]
    # bounded sample: the leading elements of the tensor, whole chunks, sized so that the run ends in minutes
    sample = min(spec.n, args.reference_sample // spec.chunk * spec.chunk)
    x_host = workloads.generate(args.workload, 0, sample)
    for _ in range(args.warmup):
        oracle.decompress(oracle.compress(x_host, spec.chunk, mode.k, mode.range, mode.round, mode.layout, spec.seed, 0)[0], sample)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        stream, _ = oracle.compress(x_host, spec.chunk, mode.k, mode.range, mode.round, mode.layout, spec.seed, 0)
        oracle.decompress(stream, sample)
    dt = (time.perf_counter() - t0) / args.steps
    value = 4 * sample / dt / 1e9
    desc = "first %d elements of %s per step" % (sample, args.workload)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": args.workload, "shape": list(spec.shape), "n_elems": spec.n, "chunk": spec.chunk,
                   "mode": mode_name(mode), "sample": desc},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--repeats", type=int, default=10, help="blocks of --steps steps; the headline is their median")
    ap.add_argument("--headline-only", action="store_true", help="skip the rows of the other workloads")
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(workloads.TENSORS))
    ap.add_argument("--sweep", action="store_true", help="also time every workload's headline modes")
    ap.add_argument("--all-modes", action="store_true",
                    help="also time all 28 modes of the consecutive layouts on the 256 MB tensor, chunks of 4096 and 1024")
    ap.add_argument("--sweep-max-bytes", type=int, default=1 << 30)
    ap.add_argument("--sweep-only", default=None, choices=sorted(workloads.TENSORS), help="restrict the sweep to one tensor")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--kernels-only", action="store_true",
                    help="profiling runs: skip the host-buffer and CPU-oracle legs (the line is then not a bench result)")
    ap.add_argument("--mode-index", type=int, default=0, help="which of the workload's headline modes to run")
    ap.add_argument("--cpu-budget", type=float, default=10.0)
    ap.add_argument("--reference-sample", type=int, default=1 << 24)
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        args.warmup = max(args.warmup, 3)
        run_gpu(args)


if __name__ == "__main__":
    main()
