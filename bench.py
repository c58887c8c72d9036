#!/usr/bin/env python
"""Benchmark of the BlockFFN chunk-verify FFN forward on B200.

One step = one pass of the whole hot path (chunk union + expert FFN over the union
experts, scores-in) over one batch of CHUNKS successive L-token chunks, each chunk
reading a different copy of the layer's weights so that no weight byte is served
from L2. The batch is captured once in a CUDA graph and replayed per step.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 1|2|3|4] [--L 8]
    python bench.py --impl reference      # the CPU oracle on the host cores

Prints one JSON line (rank 0). `value` is active-expert-weight bytes per second.
"""
import argparse
import json
import math
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2507_08771_b200 import inputs as I  # noqa: E402

METRIC = "chunk-verify FFN active-weight HBM GB/s (latency us per chunk alongside)"
L2_BYTES = 126e6
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0


def parse():
    p = argparse.ArgumentParser()
    p.add_argument("--gpus", type=int, default=1)
    p.add_argument("--steps", type=int, default=20)
    p.add_argument("--warmup", type=int, default=5)
    p.add_argument("--impl", default="ours", choices=["ours", "reference"])
    p.add_argument("--config", type=int, default=1, choices=[1, 2, 3, 4])
    p.add_argument("--L", type=int, default=None, help="chunk length (default: the config's)")
    p.add_argument("--chunks", type=int, default=1024, help="chunks per step")
    p.add_argument("--variant", type=int, default=0, help="0 auto, 1 CUDA-core, 2 tensor-core")
    p.add_argument("--flags", type=lambda v: int(v, 0), default=0,
                   help="blockffn_config.flags (ring depths, BLOCKFFN_CFG_* bits)")
    p.add_argument("--no-cpu-baseline", action="store_true")
    p.add_argument("--no-extras", action="store_true",
                   help="skip the other configurations (L sweep, router-on layer and union sweep, "
                        "24-layer stack), which add about two minutes to a single-GPU run")
    return p.parse_args()


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def measured_traffic(config, L, kernel):
    """dram__bytes_read + dram__bytes_write per call from the ncu capture summarised in
    profiles/dram_traffic.md (rows `| config | L | kernel | bytes |`), or None if that
    configuration was not captured."""
    try:
        for line in open(os.path.join(ROOT, "profiles", "dram_traffic.md")):
            f = [v.strip() for v in line.strip().strip("|").split("|")]
            if len(f) >= 4 and f[0] == str(config) and f[1] == str(L) and f[2] == kernel:
                return int(f[3])
    except (OSError, ValueError):
        pass
    return None


def copies_needed(active_bytes):
    """Enough weight copies that twice the L2 is streamed between two uses of one copy."""
    return max(8, int(math.ceil(2 * L2_BYTES / active_bytes)) + 1)


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu), f"--query-gpu={self.Q}",
                 "--format=csv,noheader,nounits", "-lms", "20"],
                stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def mark(self):
        """Samples taken so far are from before the load started: leave them out."""
        try:
            self.skip = sum(1 for _ in open(self.path))
        except Exception:
            self.skip = 0

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        try:
            for k, line in enumerate(open(self.path)):
                if k < getattr(self, "skip", 0):
                    continue
                f = [v.strip() for v in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1])); mx.append(float(f[2]))
                except ValueError:
                    continue
                for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown",
                                    "sw_power_cap"), f[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(mx)), samples=len(sm),
                       reasons=sorted(reasons))
        return out


# ----------------------------------------------------------------------------
# workload
# ----------------------------------------------------------------------------
class Workload:
    """Device-resident synthetic inputs for one benchmark configuration."""

    def __init__(self, cfg_index, L, chunks, variant, device, flags=0, u=None, stack_layers=0):
        import torch
        from paper_2507_08771_b200 import binding as B
        self.torch, self.B = torch, B
        self.idx, self.chunks, self.device = cfg_index, chunks, device
        self.stack = cfg_index == 4 or stack_layers > 0
        self.sh = sh = I.SHAPES[cfg_index]
        self.L = L or sh.L
        seed = I.config_seed(cfg_index)
        self.u = sh.u if u is None else u
        self.active_bytes = sh.active_bytes(self.u)
        # successive chunks of configs 1-3 are independent inputs; the stack (4) feeds each layer
        # the previous layer's output, so only its routing inputs and weights are stable
        self.call_flags = B.CALL_INDEPENDENT if self.stack else B.CALL_INDEPENDENT_X
        self.layer = B.Layer(sh.d, sh.E, sh.d_e, L_max=max(self.L, 8), variant=variant, device=device,
                             flags=flags)
        if cfg_index == 4:
            self.n_copies = I.STACK_LAYERS          # 24 distinct layers, 1.6 GB >> L2
            host = [I.make_experts(sh.d, sh.E, sh.d_e, seed, layer=l) for l in range(self.n_copies)]
        elif stack_layers:
            self.n_copies = stack_layers             # same values, distinct device addresses
            one = I.make_experts(sh.d, sh.E, sh.d_e, seed)
            host = [one] * self.n_copies
        else:
            self.n_copies = copies_needed(self.active_bytes)
            one = I.make_experts(sh.d, sh.E, sh.d_e, seed)
            host = [one] * self.n_copies             # same values, distinct device addresses
        self.dws = []
        for U, D in host:
            tU, tD = B.to_device_bf16(U, device), B.to_device_bf16(D, device)
            self.dws.append(B.DeviceWeights(B.make_weights(U=tU, D=tD), {"U": tU, "D": tD}))
        self.host_weights = host
        # per-chunk inputs, on the host (pinned) and on the device
        n = chunks
        if self.stack:
            # chunk c runs through all layers; scores differ per (layer, chunk)
            self.calls_per_chunk = self.n_copies
            sc = np.stack([np.stack([I.make_scores(sh.E, self.L, self.u, seed, layer=l, chunk=c)
                                     for l in range(self.n_copies)]) for c in range(n)])
        else:
            self.calls_per_chunk = 1
            sc = np.stack([I.make_scores(sh.E, self.L, self.u, seed, chunk=c) for c in range(n)])[:, None]
        xs = np.stack([I.make_x(sh.d, self.L, seed, chunk=c) for c in range(n)])
        self.scores_host = torch.from_numpy(sc).pin_memory()
        self.x_host = torch.from_numpy(xs.view(np.int16)).pin_memory()
        self.scores = self.scores_host.to(device)
        self.x = self.x_host.to(device).view(torch.bfloat16)
        self.out = torch.zeros(n, self.L, sh.d, dtype=torch.float32, device=device)
        self.out_host = torch.empty(n, self.L, sh.d, dtype=torch.float32).pin_memory()
        self.x_pp = torch.zeros(2, self.L, sh.d, dtype=torch.bfloat16, device=device)
        self.ids = torch.zeros(n, self.calls_per_chunk, sh.E, dtype=torch.int32, device=device)
        self.nu = torch.zeros(n, self.calls_per_chunk, dtype=torch.int32, device=device)
        self.calls_per_step = n * self.calls_per_chunk
        self.h2d_bytes = self.x_host.numel() * 2 + self.scores_host.numel() * 4
        self.d2h_bytes = self.out_host.numel() * 4

    # -- the hot path: union + expert FFN per chunk (and per layer for the stack) --
    def enqueue_step(self, stream, lo=0, hi=None):
        """Chunks [lo, hi) of the step."""
        B, lay = self.B, self.layer
        hi = self.chunks if hi is None else hi
        if self.stack:
            for c in range(lo, hi):
                # residual stream: out[c] starts as h0 = f32(x[c]); x ping-pongs in bf16
                self.out[c].copy_(self.x[c])
                self.x_pp[0].copy_(self.x[c])
                for l in range(self.n_copies):
                    B.blockffn_layer_forward_scores(
                        lay.h, self.dws[l].struct, self.x_pp[l % 2], self.scores[c, l], self.L,
                        self.out[c], self.x_pp[(l + 1) % 2], lay.stats,
                        B.CALL_ACCUMULATE | B.CALL_INDEPENDENT, stream)
        else:
            for c in range(lo, hi):
                B.blockffn_layer_forward_scores(
                    lay.h, self.dws[c % self.n_copies].struct, self.x[c], self.scores[c, 0], self.L,
                    self.out[c], None, lay.stats, self.call_flags, stream)

    # -- expert stage alone (the dominant kernels), unions precomputed --
    def enqueue_unions(self, stream):
        B, lay = self.B, self.layer
        for c in range(self.chunks):
            for l in range(self.calls_per_chunk):
                B.blockffn_chunk_union(lay.h, self.scores[c, l], self.L, None, self.ids[c, l],
                                       self.nu[c, l:l + 1], None, stream)

    def enqueue_expert_only(self, stream):
        B, lay = self.B, self.layer
        for c in range(self.chunks):
            for l in range(self.calls_per_chunk):
                k = l if self.stack else c % self.n_copies
                B.blockffn_expert_ffn(lay.h, self.dws[k].struct, self.x[c], self.scores[c, l], self.L,
                                      self.ids[c, l], self.nu[c, l:l + 1], self.out[c], None,
                                      B.CALL_INDEPENDENT if self.stack else self.call_flags, stream)


def max_over_ranks(values, world, device=None):
    """Element-wise maximum of a list of floats over all ranks (the slowest rank sets the time).
    world == 1: the values themselves. Uses the default process group (NCCL on GPUs, gloo on CPU)."""
    if world <= 1:
        return [float(v) for v in values]
    import torch
    import torch.distributed as dist
    t = torch.tensor(values, dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]


def job_throughput(world, bytes_per_rank_step, ms_step):
    """Whole-job GB/s: every rank streams bytes_per_rank_step in ms_step (replicas, no collective)."""
    return world * bytes_per_rank_step / (ms_step * 1e-3) / 1e9


def time_end_to_end(torch, wl, device, steps, warmup, segments=4):
    """One step = every chunk's x and scores copied in from pinned host memory, the chunks run
    through the library, every chunk's output copied back to pinned host memory. The step is cut
    into segments that flow through three streams (copy in, compute, copy out), so the copies of
    one segment run under the compute of another; events keep a segment's buffers from being
    overwritten before they have been consumed. Returns ms per step (device time)."""
    n = wl.chunks
    segments = max(1, min(segments, n))
    bounds = [(i * n // segments, (i + 1) * n // segments) for i in range(segments)]
    s_in, s_run, s_out = (torch.cuda.Stream(device) for _ in range(3))
    graphs = [capture(torch, s_run, lambda st, lo=lo, hi=hi: wl.enqueue_step(st, lo, hi))
              for lo, hi in bounds]
    x16 = wl.x.view(torch.int16)
    ev_in = [torch.cuda.Event() for _ in bounds]
    ev_run = [torch.cuda.Event() for _ in bounds]
    ev_out = [torch.cuda.Event() for _ in bounds]
    first = [True]

    def step():
        for j, (lo, hi) in enumerate(bounds):
            with torch.cuda.stream(s_in):
                if not first[0]:
                    s_in.wait_event(ev_run[j])          # last step's compute has read x, scores
                x16[lo:hi].copy_(wl.x_host[lo:hi], non_blocking=True)
                wl.scores[lo:hi].copy_(wl.scores_host[lo:hi], non_blocking=True)
                ev_in[j].record(s_in)
            with torch.cuda.stream(s_run):
                s_run.wait_event(ev_in[j])
                if not first[0]:
                    s_run.wait_event(ev_out[j])         # last step's out has been copied back
                graphs[j].replay()
                ev_run[j].record(s_run)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_run[j])
                wl.out_host[lo:hi].copy_(wl.out[lo:hi], non_blocking=True)
                ev_out[j].record(s_out)
        first[0] = False

    for _ in range(warmup):
        step()
    torch.cuda.synchronize(device)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(s_in)
    s_run.wait_event(e0)
    s_out.wait_event(e0)
    for _ in range(steps):
        step()
    s_in.wait_stream(s_run)
    s_in.wait_stream(s_out)
    e1.record(s_in)
    torch.cuda.synchronize(device)
    return e0.elapsed_time(e1) / steps


def capture(torch, stream, fn):
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        fn(stream)                      # eager once: warms up, surfaces errors
        stream.synchronize()
        with torch.cuda.graph(g, stream=stream):
            fn(stream)
    return g


def time_replays(torch, stream, graph, steps, warmup, pre=None, post=None, per_replay=None):
    """ms per step over `steps` back-to-back replays (events around the whole run, on the stream
    the graph is launched on). per_replay (a list) also receives each replay's own time: an
    event between consecutive replays costs nothing measurable next to a step of milliseconds."""
    with torch.cuda.stream(stream):
        for _ in range(warmup):
            if pre:
                pre()
            graph.replay()
            if post:
                post()
        stream.synchronize()
        marks = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
        marks[0].record(stream)
        for k in range(steps):
            if pre:
                pre()
            graph.replay()
            if post:
                post()
            marks[k + 1].record(stream)
        stream.synchronize()
    if per_replay is not None:
        per_replay.extend(marks[k].elapsed_time(marks[k + 1]) for k in range(steps))
    return marks[0].elapsed_time(marks[steps]) / steps      # ms per step


# ----------------------------------------------------------------------------
# CPU oracle legs
# ----------------------------------------------------------------------------
def oracle_sample(cfg_index, L, budget_s, max_chunks, union_only=True):
    """Times the CPU oracle (as it stands, one thread) on successive chunks of the
    workload until the time budget is used. Returns (GB/s of active weights, us/chunk, n)."""
    import oracle
    sh = I.SHAPES[cfg_index]
    L = L or sh.L
    seed = I.config_seed(cfg_index)
    U, D = I.make_experts(sh.d, sh.E, sh.d_e, seed)
    oracle.build()
    t_total, n = 0.0, 0
    while n < max_chunks and (t_total < budget_s or n == 0):
        x = I.make_x(sh.d, L, seed, chunk=n)
        s = I.make_scores(sh.E, L, sh.u, seed, chunk=n)
        t0 = time.perf_counter()
        oracle.layer_forward_scores(x, s, U, D, union_only=union_only)
        t_total += time.perf_counter() - t0
        n += 1
    per = t_total / n
    return sh.active_bytes() / per / 1e9, per * 1e6, n


def oracle_all_cores(cfg_index, L, chunks_per_thread):
    """The same oracle, union-restricted, one chunk per call, on every core this process may use
    (one host thread per core, each working through its own chunks; the C routine runs outside
    the interpreter lock). Returns (GB/s of active weights, us per chunk of wall time, threads)."""
    import concurrent.futures
    import oracle
    sh = I.SHAPES[cfg_index]
    L = L or sh.L
    seed = I.config_seed(cfg_index)
    U, D = I.make_experts(sh.d, sh.E, sh.d_e, seed)
    oracle.build()
    try:
        threads = len(os.sched_getaffinity(0))
    except AttributeError:
        threads = os.cpu_count() or 1
    n = threads * chunks_per_thread
    xs = [I.make_x(sh.d, L, seed, chunk=c) for c in range(n)]
    ss = [I.make_scores(sh.E, L, sh.u, seed, chunk=c) for c in range(n)]

    def work(k):
        for c in range(k, n, threads):
            oracle.layer_forward_scores(xs[c], ss[c], U, D, union_only=True)

    with concurrent.futures.ThreadPoolExecutor(threads) as pool:
        t0 = time.perf_counter()
        list(pool.map(work, range(threads)))
        wall = time.perf_counter() - t0
    per = wall / n
    return sh.active_bytes() / per / 1e9, per * 1e6, threads, n


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    sh = I.SHAPES[args.config]
    L = args.L or sh.L
    per_step_chunks = 2
    import oracle
    oracle.build()
    seed = I.config_seed(args.config)
    U, D = I.make_experts(sh.d, sh.E, sh.d_e, seed)

    def step(k):
        for c in range(per_step_chunks):
            x = I.make_x(sh.d, L, seed, chunk=k * per_step_chunks + c)
            s = I.make_scores(sh.E, L, sh.u, seed, chunk=k * per_step_chunks + c)
            oracle.layer_forward_scores(x, s, U, D, union_only=True)

    for k in range(args.warmup):
        step(k)
    t0 = time.perf_counter()
    for k in range(args.steps):
        step(k)
    dt = (time.perf_counter() - t0) / args.steps
    gbs = per_step_chunks * sh.active_bytes() / dt / 1e9
    sample = (f"{per_step_chunks} chunks per step of config {args.config} "
              f"(d={sh.d}, E={sh.E}, d_e={sh.d_e}, L={L}, union {sh.u}), union-restricted sum, float64")
    line = {
        "impl": "reference", "metric": METRIC, "value": gbs, "unit": "GB/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "latency_us_per_chunk": dt / per_step_chunks * 1e6,
        "config": {"workload": f"config {args.config}: {sh.name}", "d": sh.d, "E": sh.E,
                   "d_e": sh.d_e, "L": L, "union": sh.u, "chunks_per_step": per_step_chunks},
        "cpu_baseline": {"value": gbs, "unit": "GB/s", "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": gbs, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ----------------------------------------------------------------------------
# main
# ----------------------------------------------------------------------------
def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2507_08771_b200 import binding as B

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback); "
                         "use --impl reference for the CPU oracle")
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)
    B.load()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    wl = Workload(args.config, args.L, args.chunks, args.variant, device, args.flags)
    sh = wl.sh
    stream = torch.cuda.Stream(device)
    lay = wl.layer

    n0 = lay.launch_count()
    g_step = capture(torch, stream, wl.enqueue_step)
    launches_per_step = (lay.launch_count() - n0) // 2       # fn ran twice (eager + capture)
    with torch.cuda.stream(stream):
        wl.enqueue_unions(stream)
        stream.synchronize()
    n0 = lay.launch_count()
    g_expert = capture(torch, stream, wl.enqueue_expert_only)
    expert_launches = (lay.launch_count() - n0) // 2

    # clocks and throttle reasons are sampled (every 20 ms) from before the warm-up replays until
    # the last timed leg is over: the timed legs run the same kernels back to back
    sampler = ClockSampler(local)
    barrier()
    if rank == 0:
        sampler.start()
        time.sleep(0.3)          # nvidia-smi needs a moment before its first sample
        sampler.mark()
    per_step = []
    ms_step = time_replays(torch, stream, g_step, args.steps, args.warmup, per_replay=per_step)
    barrier()

    # end to end: host buffers in, host buffers out, copies inside the timed region
    barrier()
    ms_e2e = time_end_to_end(torch, wl, device, max(3, args.steps // 2), 3)
    # One call on its own: enqueued on an idle device, events right around it (launch latency,
    # cold routing inputs and weights, no overlap with a neighbour). The same call is also timed
    # on the host alone (time spent in the Python binding and the library's launch code, no
    # synchronisation inside), which is what the device sits idle for between the two events when
    # nothing is queued ahead of it.
    iso, host_us = [], []
    with torch.cuda.stream(stream):
        for c in range(min(32, wl.chunks)):
            stream.synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            t0 = time.perf_counter()
            wl.enqueue_step(stream, c, c + 1)
            host_us.append((time.perf_counter() - t0) * 1e6)
            b.record(stream)
            stream.synchronize()
            iso.append(a.elapsed_time(b) * 1e3)
    isolated_us = float(np.median(iso[4:])) if len(iso) > 4 else float(np.median(iso))
    host_call_us = float(np.median(host_us[4:])) if len(host_us) > 4 else float(np.median(host_us))
    # the same single call as a one-node graph (no Python, no launch code between the events)
    g_one = capture(torch, stream, lambda st: wl.enqueue_step(st, 0, 1))
    one = []
    with torch.cuda.stream(stream):
        for _ in range(12):
            stream.synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            g_one.replay()
            b.record(stream)
            stream.synchronize()
            one.append(a.elapsed_time(b) * 1e3)
    isolated_graph_us = float(np.median(one[2:]))
    barrier()
    per_expert = []
    ms_expert = time_replays(torch, stream, g_expert, args.steps, args.warmup, per_replay=per_expert)
    barrier()
    # stage level: the union entry point alone (one launch per chunk), from its own graph
    g_union = capture(torch, stream, wl.enqueue_unions)
    per_union = []
    time_replays(torch, stream, g_union, max(3, args.steps // 2), 2, per_replay=per_union)
    clocks = sampler.stop() if rank == 0 else {}
    status = lay.last_status()
    assert status == 0, f"device status word {status}"
    launches_per_call = expert_launches // max(wl.calls_per_step, 1)
    assert torch.isfinite(wl.out).all()
    ms_step_median, ms_expert_median = float(np.median(per_step)), float(np.median(per_expert))

    ms_step, ms_e2e, ms_expert = max_over_ranks([ms_step, ms_e2e, ms_expert], world, device)

    calls = wl.calls_per_step
    bytes_step = calls * wl.active_bytes
    value = job_throughput(world, bytes_step, ms_step)
    e2e = job_throughput(world, bytes_step, ms_e2e)
    peak, peak_kind = measured_peak()
    # algorithmic bytes of one expert-stage call: weights + x + out + scores
    alg_bytes = wl.active_bytes + 2 * wl.L * sh.d + 4 * wl.L * sh.d + 4 * wl.L * sh.E
    us_expert = ms_expert * 1e3 / calls
    achieved = alg_bytes / (us_expert * 1e-6) / 1e9

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    line = {
        "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "latency_us_per_chunk": ms_step * 1e3 / wl.chunks,
        "latency_us_per_layer_call": ms_step * 1e3 / calls,
        "latency_us_per_layer_call_median_replay": ms_step_median * 1e3 / calls,
        "latency_us_isolated_call": isolated_us,
        "latency_isolated_call": {
            "us_events_around_python_call": isolated_us, "us_host_time_in_binding_and_launch": host_call_us,
            "us_events_around_one_node_graph": isolated_graph_us,
            "note": "on an idle device the events bracket the host's own launch work; the graph leg "
                    "has no host work between the events: launch latency plus one cold call"},
        "stage_us_per_call": {"chunk_union_entry_point": float(np.median(per_union)) * 1e3 / calls,
                              "expert_ffn_entry_point": ms_expert_median * 1e3 / calls,
                              "layer_forward_scores": ms_step_median * 1e3 / calls},
        "pct_of_nominal_8TBs": 100.0 * value / world / NOMINAL_HBM_GBS,
        "config": {
            "workload": f"config {args.config}: {sh.name} (scores-in: chunk union + expert FFN)",
            "d": sh.d, "E": sh.E, "d_e": sh.d_e, "L": wl.L, "union": wl.u,
            "chunks_per_step": wl.chunks, "layer_calls_per_step": calls,
            "active_bytes_per_call": wl.active_bytes, "weight_copies": wl.n_copies,
            "l2": f"inputs larger than L2: {wl.n_copies} weight copies rotated, "
                  f"{wl.n_copies * wl.active_bytes / 1e6:.0f} MB streamed between reuses",
            "replicas": "independent replicas per GPU, no collective" if world > 1 else "single GPU",
            "variant": args.variant, "flags": args.flags,
        },
        "clocks": clocks,
        "e2e": {"value": e2e, "unit": "GB/s", "h2d_bytes_per_step": wl.h2d_bytes,
                "d2h_bytes_per_step": wl.d2h_bytes, "ms_per_step": ms_e2e},
        "gpu_launches": launches_per_step * args.steps,
        "gpu_launches_per_step": launches_per_step,
        "roofline": {
            "bound": "hbm",
            "kernel": (("expert_lean_kernel" if wl.L <= 8 else "expert_wide_kernel") +
                       " (one launch per call: up projection, hand-over, down projection)"
                       if launches_per_call == 1 else
                       "expert_up_mma + expert_down_mma (the chained pair of one call)"
                       if launches_per_call == 2 and args.variant != 1 else "expert_up_simt + expert_down_simt"),
            "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
            "peak_kind": f"of {peak_kind}", "us_per_launch": us_expert / max(launches_per_call, 1),
            "us_per_call": us_expert, "us_per_call_median_replay": ms_expert_median * 1e3 / calls,
            "algorithmic_bytes_per_launch": alg_bytes, "launches_per_call": launches_per_call,
            # dram__bytes_read + write of one call's launches (ncu, see profiles/dram_traffic.md)
            "traffic": measured_traffic(args.config, wl.L, "lean" if launches_per_call == 1 else "pair"),
        },
    }
    if not args.no_cpu_baseline and world == 1:
        gbs, us, n = oracle_sample(args.config, wl.L, budget_s=8.0, max_chunks=64)
        gbs_all, us_all, n_all = oracle_sample(args.config, wl.L, budget_s=4.0, max_chunks=8, union_only=False)
        gbs_mt, us_mt, threads, n_mt = oracle_all_cores(args.config, wl.L, chunks_per_thread=12)
        line["cpu_baseline"] = {
            "value": gbs, "unit": "GB/s", "cores": 1, "kind": "oracle", "us_per_chunk": us,
            "sample": f"{n} chunks of the same workload (one layer call each), union-restricted "
                      f"sum, float64, single thread",
            "legs": {
                "single_thread_all_experts": {
                    "value": gbs_all, "unit": "GB/s", "us_per_chunk": us_all, "cores": 1,
                    "sample": f"{n_all} chunks, the definition's sum over all {sh.E} experts"},
                "single_thread_union_only": {"value": gbs, "unit": "GB/s", "us_per_chunk": us,
                                             "cores": 1, "sample": f"{n} chunks"},
                "all_cores_union_only": {
                    "value": gbs_mt, "unit": "GB/s", "us_per_chunk": us_mt, "cores": threads,
                    "sample": f"{n_mt} chunks over {threads} host threads (the affinity mask of "
                              f"this process), one chunk per oracle call"}}}
    if not args.no_extras and world == 1:
        del wl, g_step, g_expert
        torch.cuda.empty_cache()
        line["extras"] = extras(args, torch, device, peak)
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


class RouterWorkload:
    """Config 3 with the router on: blockffn_layer_forward over correlated or iid chunks."""

    def __init__(self, chunks, device, rho, n_copies, L=None):
        import torch
        from paper_2507_08771_b200 import binding as B
        self.torch, self.B, self.chunks = torch, B, chunks
        sh = I.SHAPES[3]
        if L is not None:
            sh = I.Shape(sh.name, d=sh.d, E=sh.E, d_e=sh.d_e, L=L, union_frac=sh.union_frac)
        self.sh = sh
        seed = I.config_seed(3)
        self.layer = B.Layer(sh.d, sh.E, sh.d_e, L_max=sh.L, device=device)
        w = I.make_layer(sh, seed, bias_shift=I.ROUTER_BIAS_SHIFT)
        first = self.layer.upload_weights(w)
        self.dws = [first]
        for _ in range(n_copies - 1):          # distinct addresses for the expert weights only
            tU, tD = B.to_device_bf16(w["U"], device), B.to_device_bf16(w["D"], device)
            t = dict(first.tensors, U=tU, D=tD)
            self.dws.append(B.DeviceWeights(B.make_weights(t["W_r"], t["gain"], t["bias"], tU, tD), t))
        if rho is None:
            xs = np.stack([I.make_x(sh.d, sh.L, seed, chunk=c) for c in range(chunks)])
        else:
            xs = np.stack([I.make_correlated_x(sh.d, sh.L, rho, seed, chunk=c) for c in range(chunks)])
        self.x = torch.from_numpy(xs.view(np.int16)).to(device).view(torch.bfloat16)
        self.out = torch.zeros(chunks, sh.L, sh.d, dtype=torch.float32, device=device)
        # the chunks are independent of one another: x never comes from the call before
        self.call_flags = B.CALL_INDEPENDENT_X

    def enqueue_step(self, stream):
        B, lay = self.B, self.layer
        for c in range(self.chunks):
            B.blockffn_layer_forward(lay.h, self.dws[c % len(self.dws)].struct, self.x[c], self.sh.L,
                                     self.out[c], None, lay.stats, self.call_flags, stream)

    def enqueue_router_only(self, stream):
        """The router entry point alone (Eq. 3 + per-token masks), one launch per chunk."""
        B, lay = self.B, self.layer
        if not hasattr(self, "scores_out"):
            self.scores_out = self.torch.zeros(self.chunks, self.sh.L, self.sh.E, device=self.out.device)
        for c in range(self.chunks):
            B.blockffn_router(lay.h, self.dws[0].struct, self.x[c], self.sh.L, self.scores_out[c], None, stream)

    def sparsity(self):
        hs = self.layer.stats_host()
        return (self.B.blockffn_tls(hs, self.sh.E), 1.0 - self.B.blockffn_cls(hs, self.sh.E))


_probe_lib = None


def probe_read(src, nbytes, chained, stream):
    """bench_probe.cu's benchprobe_read (a library of its own, built by __graft_entry__.build())."""
    global _probe_lib
    import ctypes
    if _probe_lib is None:
        path = os.path.join(ROOT, "libbenchprobe.so")
        if not os.path.exists(path):
            raise ImportError(f"{path} not found: build it with `python __graft_entry__.py`")
        _probe_lib = ctypes.CDLL(path)
        _probe_lib.benchprobe_read.argtypes = [ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int,
                                               ctypes.c_void_p]
    ptr = src if isinstance(src, int) else src.data_ptr()
    rc = _probe_lib.benchprobe_read(ptr, int(nbytes), 1 if chained else 0, stream.cuda_stream)
    if rc != 0:
        raise RuntimeError(f"benchprobe_read returned {rc}")


def read_ceilings(args, torch, device, B):
    """What a plain read reaches on this device (bench_probe.cu: 128-bit loads, four CTAs per
    SM, data discarded): streaming over 2 GiB, and single launches the size of one call's active
    weights, back to back over memory that is not in L2, launched plainly and chained like the
    library's own kernels."""
    nbytes = 2 << 30
    buf = torch.empty(nbytes, dtype=torch.uint8, device=device)
    buf.fill_(1)
    stream = torch.cuda.Stream(device)
    steps = max(3, args.steps // 2)

    def enqueue_stream(st):
        for _ in range(4):
            probe_read(buf, nbytes, False, st)

    g = capture(torch, stream, enqueue_stream)
    ms = time_replays(torch, stream, g, steps, 2)
    out = {"streaming_read_GBps": 4 * nbytes / ms / 1e6, "streaming_bytes": nbytes}
    rows = []
    for cfg_index in (1, 2):
        sh = I.SHAPES[cfg_index]
        size = sh.u * 2 * sh.d_e * sh.d * 2            # the active weights of one call
        n = min(128, nbytes // size)
        base = buf.data_ptr()
        row = {"config": cfg_index, "bytes_per_launch": size, "launches": n}
        for name, chained in (("plain", False), ("chained", True)):
            def enqueue(st, chained=chained):
                for i in range(n):
                    probe_read(base + i * size, size, chained, st)
            g = capture(torch, stream, enqueue)
            us = time_replays(torch, stream, g, steps, 2) * 1e3 / n
            row[name] = {"us_per_launch": us, "GBps": size / us / 1e3}
        rows.append(row)
    out["size_matched"] = rows
    del buf
    torch.cuda.empty_cache()
    return out


def stack_router_on(args, torch, device, peak, layers=None, chunks=16):
    from paper_2507_08771_b200 import binding as B
    sh = I.SHAPES[4]
    layers = layers or I.STACK_LAYERS
    seed = I.config_seed(4)
    lay = B.Layer(sh.d, sh.E, sh.d_e, L_max=sh.L, device=device, flags=args.flags)
    w = I.make_layer(sh, seed, bias_shift=I.ROUTER_BIAS_SHIFT)
    # residual-branch scale 1/32 (exact in bf16): the running hidden state then stays near unit
    # scale over the stack, and with it the sparsity the fixed router bias gives
    w["D"] = I.f32_to_bf16_bits(I.bf16_bits_to_f32(w["D"]) * np.float32(1.0 / 32.0))
    first = lay.upload_weights(w)
    dws = [first]
    for _ in range(layers - 1):
        t = {k: v.clone() for k, v in first.tensors.items()}
        dws.append(B.DeviceWeights(B.make_weights(t["W_r"], t["gain"], t["bias"], t["U"], t["D"]), t))
    # no normalisation of the hidden state sits between the layers (it is not part of this path):
    # the router sees x ~ N(0,1) at the first layer and the running residual after it
    xs = np.stack([I.make_correlated_x(sh.d, sh.L, 0.96, seed, chunk=c) for c in range(chunks)])
    x0 = torch.from_numpy(xs.view(np.int16)).to(device).view(torch.bfloat16)
    res = torch.zeros(chunks, sh.L, sh.d, dtype=torch.float32, device=device)
    xpp = torch.zeros(2, sh.L, sh.d, dtype=torch.bfloat16, device=device)

    def enqueue(stream):
        for c in range(chunks):
            res[c].copy_(x0[c])
            xpp[0].copy_(x0[c])
            for l in range(layers):
                B.blockffn_layer_forward(lay.h, dws[l].struct, xpp[l % 2], sh.L, res[c], xpp[(l + 1) % 2],
                                         lay.stats, B.CALL_ACCUMULATE, stream)

    stream = torch.cuda.Stream(device)
    n0 = lay.launch_count()
    g = capture(torch, stream, enqueue)
    launches_per_layer = (lay.launch_count() - n0) / (2 * chunks * layers)   # capture() enqueues twice
    ms = time_replays(torch, stream, g, max(3, args.steps // 2), 2)
    assert lay.last_status() == 0
    hs = lay.stats_host()
    mean_u = (1.0 - B.blockffn_cls(hs, sh.E)) * sh.E
    us_layer = ms * 1e3 / (chunks * layers)
    return {"layers": layers, "chunks": chunks, "us_per_layer": us_layer, "mean_union": mean_u,
            "tls": B.blockffn_tls(hs, sh.E), "GBps": mean_u * sh.expert_bytes / us_layer / 1e3,
            "launches_per_layer": launches_per_layer,
            "note": "router on every layer (one kernel per layer with the router inside, or router, up, down where "
                    "the shape does not take that form); no normalisation between "
                    "layers, down projections scaled by 1/32 so that the hidden state keeps its scale; the union "
                    "is whatever the router derives (mean reported)"}


def extras(args, torch, device, peak):
    """The other configurations, each as us per call and GB/s of active expert bytes."""
    from paper_2507_08771_b200 import binding as B
    out = {"read_ceilings": read_ceilings(args, torch, device, B)}
    chunks = min(args.chunks, 64)

    def timed(wl):
        stream = torch.cuda.Stream(device)
        g = capture(torch, stream, wl.enqueue_step)
        ms = time_replays(torch, stream, g, max(3, args.steps // 2), 3)
        assert wl.layer.last_status() == 0
        return ms

    # config 2: L sweep, tensor-core path against CUDA-core path
    rows = []
    for L in I.L_SWEEP:
        row = {"L": L}
        for name, variant, form in (("tensor_core", 0, 0), ("tensor_core_pair", 0, B.CFG_TWO_KERNELS),
                                    ("cuda_core", 1, 0)):
            wl = Workload(2, L, chunks, variant, device, args.flags | form)
            us = timed(wl) * 1e3 / wl.calls_per_step
            hs = wl.layer.stats_host()
            row[name] = {"us_per_call": us, "GBps": wl.active_bytes / us / 1e3,
                         "frac_of_measured": wl.active_bytes / us / 1e3 / peak}
            row["tls"] = wl.B.blockffn_tls(hs, wl.sh.E)
            del wl
            torch.cuda.empty_cache()
        rows.append(row)
    out["config2_L_sweep"] = rows

    # config 3: router on (iid tokens, and correlated tokens whose union is about 30 %), then the
    # scores-in union sweep against the dense all-experts layer
    sh = I.SHAPES[3]
    full = {}
    n_copies = copies_needed(sh.active_bytes(sh.E))          # sized for the dense union
    lo, hi, rho = 0.0, 1.0, 0.9
    for _ in range(7):                                        # bisect rho on the library's own router
        rho = 0.5 * (lo + hi)
        probe = RouterWorkload(16, device, rho, 1)
        probe.enqueue_step(torch.cuda.current_stream())
        torch.cuda.synchronize()
        frac = probe.sparsity()[1]
        lo, hi = (rho, hi) if frac > 0.30 else (lo, rho)
        del probe
    for name, r in (("iid_tokens", None), ("correlated_tokens", rho)):
        wl = RouterWorkload(chunks, device, r, n_copies)
        n0 = wl.layer.launch_count()
        ms = timed(wl)
        launches = (wl.layer.launch_count() - n0) / (2 * chunks)     # capture() enqueues the step twice
        hs = wl.layer.stats_host()
        tls, ufrac = wl.sparsity()
        us = ms * 1e3 / chunks
        mean_u = ufrac * sh.E
        # reuse ratio between successive tokens of a chunk (Sec. 4.1.2), from the scores each of
        # the first 16 layer calls leaves in the handle; untimed
        reuse = torch.zeros(2, dtype=torch.float64, device=device)
        for c in range(min(16, chunks)):
            B.blockffn_layer_forward(wl.layer.h, wl.dws[0].struct, wl.x[c], sh.L, wl.out[c], None, None, 0)
            B.blockffn_reuse_ratio(wl.layer.h, None, sh.L, reuse)
        rr = reuse.cpu().numpy()
        full[name] = {"rho": r, "us_per_call": us, "tls": tls, "mean_union": mean_u,
                      "GBps": mean_u * sh.expert_bytes / us / 1e3,
                      "launches_per_call": launches,
                      "reuse_ratio": float(rr[0] / rr[1]) if rr[1] > 0 else None}
        if r is not None:               # longer chunks of the same correlated tokens, router on
            for Ll in (16, 32):
                wll = RouterWorkload(chunks, device, r, n_copies, L=Ll)
                msl = timed(wll)
                tl, ul = wll.sparsity()
                usl = msl * 1e3 / chunks
                full[f"{name}_L{Ll}"] = {"rho": r, "L": Ll, "us_per_call": usl, "tls": tl,
                                         "mean_union": ul * sh.E,
                                         "GBps": ul * sh.E * sh.expert_bytes / usl / 1e3}
                del wll
                torch.cuda.empty_cache()
        if r is None:                   # stage level: the router entry point from its own graph
            st2 = torch.cuda.Stream(device)
            g2 = capture(torch, st2, wl.enqueue_router_only)
            per = []
            time_replays(torch, st2, g2, max(3, args.steps // 2), 2, per_replay=per)
            full["router_entry_point_us_per_call"] = float(np.median(per)) * 1e3 / chunks
        del wl
        torch.cuda.empty_cache()
    sweep_rows, dense_us = [], None
    for frac in (1.0, 0.9, 0.8, 0.7, 0.6, 0.5, 0.4, 0.3, 0.2, 0.1):
        u = int(round(frac * sh.E))
        # each point is timed twice: with the library's default assumption about the union
        # (30 % of the experts) and with the point's own union size given as the handle's hint
        row = {"union_frac": frac, "u": u}
        for key, hint in (("default", 0), ("hinted", B.cfg_expected_union(u))):
            wl = Workload(3, sh.L, chunks, 0, device, args.flags | hint, u=u)
            row[key] = {"us_per_call": timed(wl) * 1e3 / wl.calls_per_step}
            row[key]["GBps"] = wl.active_bytes / row[key]["us_per_call"] / 1e3
            del wl
            torch.cuda.empty_cache()
        us = min(row["default"]["us_per_call"], row["hinted"]["us_per_call"])
        dense_us = us if dense_us is None else dense_us
        row.update({"us_per_call": us, "GBps": u * sh.expert_bytes / us / 1e3,
                    "time_vs_dense": us / dense_us})
        sweep_rows.append(row)
    full["union_sweep"] = sweep_rows
    out["config3_full_layer"] = full

    # beyond the benchmark's list: the paper's largest FFN shape at its kernel table's operating
    # points (32 tree tokens over a 30.86 % union, one token with 12.45 % active), against the
    # dense layer of the same shape
    sh5 = I.SHAPES[5]
    u1 = int(round(I.PAPER_ONE_TOKEN_ACTIVE * sh5.E))
    rows = {}
    for name, L, u in (("tree_32_tokens", 32, sh5.u), ("dense_32_tokens", 32, sh5.E),
                       ("one_token", 1, u1), ("dense_one_token", 1, sh5.E)):
        wl = Workload(5, L, min(chunks, 64), 0, device, args.flags | B.cfg_expected_union(u), u=u)
        us = timed(wl) * 1e3 / wl.calls_per_step
        rows[name] = {"L": L, "u": u, "E": sh5.E, "us_per_call": us,
                      "GBps": wl.active_bytes / us / 1e3}
        del wl
        torch.cuda.empty_cache()
    rows["tree_time_vs_dense"] = rows["tree_32_tokens"]["us_per_call"] / rows["dense_32_tokens"]["us_per_call"]
    rows["one_token_time_vs_dense"] = rows["one_token"]["us_per_call"] / rows["dense_one_token"]["us_per_call"]
    # the whole FFN stack of that model: 36 layers, residual between layers, scores-in, one 32-token
    # tree per pass (4.8 GB of expert weights at distinct addresses; the layers share their values)
    for name, L, u in (("stack_36_layers_tree_32_tokens", 32, sh5.u), ("stack_36_layers_one_token", 1, u1)):
        wl = Workload(5, L, 8, 0, device, args.flags | B.cfg_expected_union(u), u=u, stack_layers=36)
        ms = timed(wl)
        us_pass = ms * 1e3 / wl.chunks
        rows[name] = {"L": L, "u": u, "layers": 36, "us_per_pass": us_pass, "us_per_layer": us_pass / 36,
                      "GBps": 36 * wl.active_bytes / us_pass / 1e3}
        del wl
        torch.cuda.empty_cache()
    out["paper_2p8b_shape"] = rows

    # config 4 with the router on: every layer computes its own scores from the running hidden
    # state (blockffn_layer_forward, Eq. 3 -> Union -> Eq. 1/2), residual and bf16 hand-over as
    # in the scores-in stack. One layer's weights (router included) at 24 distinct addresses.
    out["config4_stack_router_on"] = stack_router_on(args, torch, device, peak)

    # config 4: 24-layer stack, residual between layers
    wl = Workload(4, None, min(args.chunks, I.STACK_CHUNKS), 0, device, args.flags)
    ms = timed(wl)
    us_chunk = ms * 1e3 / wl.chunks
    out["config4_stack"] = {"layers": wl.n_copies, "chunks": wl.chunks, "us_per_chunk": us_chunk,
                            "us_per_layer": us_chunk / wl.n_copies,
                            "GBps": wl.n_copies * wl.active_bytes / us_chunk / 1e3,
                            "frac_of_measured": wl.n_copies * wl.active_bytes / us_chunk / 1e3 / peak}
    return out


if __name__ == "__main__":
    a = parse()
    if a.impl == "reference":
        run_reference(a)
    else:
        run_ours(a)
