#!/usr/bin/env python
"""Benchmark of the hierarchical, load-weighted gradient synchronisation step.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload resnet18] [--impl ours|reference]
    python bench.py --sweep            # bucket-size sweep of the fused reduce, one JSON line per point

One step = one pass of the whole path over one batch of synthetic gradients that already
sit in device memory: per bucket the fused pack+widen+weighted intra-group reduce, the relay
of the fp32 group partials through pinned host memory (when the workload says so), then the
inter-group combine + scale + unpack into per-parameter gradients.  Prints ONE JSON line.

The default workload is ResNet-18 (10-class head), fp32, K = 4 ranks in 2 groups, shares
from kt_schedule(1, 1, 1.6, 1.6; 256), 25 MiB buckets, partials staged through pinned host
memory.  With N > 1 every GPU runs an independent replica of the same problem (the path
has no exchange between GPUs); the value is the sum over replicas divided by the slowest.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2505_10183_b200 import workloads as W  # noqa: E402

METRIC = "hierarchical weighted grad-reduce throughput"
UNIT = "GB/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0


# ----------------------------------------------------------------------------- helpers
def algorithmic_bytes(wl) -> dict:
    """Bytes the method must move per step (N = gradient elements per rank)."""
    N, K, G, s = wl.N, wl.K, wl.G, wl.elem_size
    k1 = K * N * s + G * N * 4          # read every gradient once, write G fp32 partials
    k2 = G * N * 4 + N * s              # read G partials, write the result once
    return {"k1": k1, "k2": k2, "step": k1 + k2, "stage_each_way": G * N * 4 if wl.staged else 0}


def measured_peak() -> tuple:
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.file = None

    def start(self):
        try:
            self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=self.file, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.file.flush()
        self.file.seek(0)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.file.read().splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        self.file.close()
        os.unlink(self.file.name)
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons),
                       samples=len(sm))
        return out


# ----------------------------------------------------------------------------- our arm
class Problem:
    """Device state of one replica: gradients, context, transport / receive / pinned buffers."""

    def __init__(self, wl, kt, device_values: bool = True, chunk_bytes: int = 4 << 20, arena: bool = False,
                 transport_dtype=torch.float32):
        """arena=False: every gradient and output tensor is its own allocation (as per-parameter
        gradients are).  arena=True: the tensors of one rank are views into one buffer, each at
        a multiple of 64 elements, so that a whole rank moves between host and device in one
        copy (the end-to-end arm)."""
        self.wl, self.kt = wl, kt
        self.chunk_bytes = chunk_bytes
        self.shares = list(wl.shares) if wl.shares is not None else kt.kt_schedule(wl.step_times, wl.global_batch)
        dt = torch.float32 if wl.dtype == "f32" else torch.bfloat16
        self.grads = []
        starts, pos = [], 0
        for m in wl.numel:
            starts.append(pos)
            pos += -(-m // 64) * 64
        self.arena_numel = pos
        self.arena_starts = starts

        def views(buf):
            return [buf[s:s + m] for s, m in zip(starts, wl.numel)]

        self.grad_arenas = []
        for r in range(wl.K):
            flat = W.rank_gradients(wl, r, "cuda" if device_values else "cpu")
            if arena:
                buf = torch.zeros(self.arena_numel, dtype=dt, device="cuda")
                row = views(buf)
                for dst, src in zip(row, W.split_tensors(flat, wl.numel)):
                    dst.copy_(src)
                self.grad_arenas.append(buf)
                self.grads.append(row)
            else:
                self.grads.append([t.cuda() for t in W.split_tensors(flat, wl.numel)])
            del flat
        self.ctx = kt.kt_groups_init(wl.group_of, self.shares, wl.G)
        if transport_dtype != torch.float32:
            kt.kt_set_transport_dtype(self.ctx, kt.KT_BF16)
        kt.kt_bucket_pack(self.ctx, self.grads, wl.bucket_cap_bytes)
        self.plan = kt.kt_plan_query(self.ctx)
        n = self.plan.transport_numel
        # the G buffers of a set are rows of one allocation: the relay then moves a chunk of all
        # groups in one copy
        self.transport = kt.kt_ptrs(list(torch.zeros(wl.G, n, dtype=transport_dtype, device="cuda")))
        if arena:
            self.out_arena = torch.zeros(self.arena_numel, dtype=dt, device="cuda")
            self.out = [views(self.out_arena)]
        else:
            self.out = [[torch.zeros(m, dtype=dt, device="cuda") for m in wl.numel]]
        self.out_ptrs = kt.kt_ptrs([t for c in self.out for t in c])
        self.out_dtype = kt.KT_F32 if wl.dtype == "f32" else kt.KT_BF16
        self.main = torch.cuda.Stream()
        if wl.staged:
            self.recv = kt.kt_ptrs(list(torch.zeros(wl.G, n, dtype=transport_dtype, device="cuda")))
            self.pinned = kt.kt_ptrs(list(torch.zeros(wl.G, n, dtype=transport_dtype).pin_memory()))
            self.side_d2h = torch.cuda.Stream()
            self.side_h2d = torch.cuda.Stream()
        self.k1_events = []
        self.k2_events = []

    def step(self, time_k1: bool = False):
        """One launch of the fused reduce over all buckets, the relay of the whole transport
        as one chunk pipeline over the two copy streams, one launch of combine+unpack.  Kernels are
        deliberately not overlapped with the copies: next to a pinned-memory copy in flight
        they run 1.7-4x slower, and the relay dominates the step by a factor of ~20."""
        kt, ctx, wl = self.kt, self.ctx, self.wl
        if time_k1:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(self.main)
        kt.kt_hier_reduce(ctx, kt.KT_INTRA, self.transport, bucket=-1, stream=self.main)
        if time_k1:
            e1.record(self.main)
            self.k1_events.append((e0, e1))
            e2, e3 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        src = self.transport
        if wl.staged:
            kt.kt_relay_through_host(ctx, self.transport, self.pinned, self.recv, self.side_d2h,
                                     self.side_h2d, bucket=-1, chunk_bytes=self.chunk_bytes,
                                     main_stream=self.main)
            kt.kt_stage_wait(ctx, kt.KT_H2D, bucket=-1, main_stream=self.main)
            src = self.recv
        if time_k1:
            e2.record(self.main)
        kt.kt_unpack_scale(ctx, src, self.out_ptrs, scale=1.0, bucket=-1, out_dtype=self.out_dtype,
                           R=1, stream=self.main)
        if time_k1:
            e3.record(self.main)
            self.k2_events.append((e2, e3))

    def direct(self):
        """The one-pass route (no transport, no relay): what a collective that needs no host
        relay costs."""
        self.kt.kt_sync_direct(self.ctx, self.out_ptrs, scale=1.0, bucket=-1, out_dtype=self.out_dtype,
                               R=1, stream=self.main)

    def k1_seconds(self) -> float:
        return sum(a.elapsed_time(b) for a, b in self.k1_events) * 1e-3

    def k2_seconds(self) -> float:
        return sum(a.elapsed_time(b) for a, b in self.k2_events) * 1e-3


def host_link_bandwidth(nbytes: int = 256 << 20, reps: int = 10, chunk_bytes: int = 4 << 20) -> dict:
    """Pinned cudaMemcpyAsync, best of `reps` (GB/s): each direction alone; both directions at
    the same time on two streams, as one copy each ("both") and cut into independent copies of
    chunk_bytes ("both_chunked": per direction, what a relay that must work in chunks of that
    size can reach at most, before the lag of its pipeline)."""
    dev = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    host = torch.empty(nbytes, dtype=torch.uint8).pin_memory()
    dev2 = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    host2 = torch.empty(nbytes, dtype=torch.uint8).pin_memory()
    best = {"d2h": 0.0, "h2d": 0.0, "both": 0.0, "both_chunked": 0.0}
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    cuts = [(lo, min(nbytes, lo + chunk_bytes)) for lo in range(0, nbytes, chunk_bytes)]
    for _ in range(reps):
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        s1.wait_event(a)
        s2.wait_event(a)
        for lo, hi in cuts:
            with torch.cuda.stream(s1):
                host[lo:hi].copy_(dev[lo:hi], non_blocking=True)
            with torch.cuda.stream(s2):
                dev2[lo:hi].copy_(host2[lo:hi], non_blocking=True)
        torch.cuda.current_stream().wait_stream(s1)
        torch.cuda.current_stream().wait_stream(s2)
        b.record()
        b.synchronize()
        best["both_chunked"] = max(best["both_chunked"], nbytes / (a.elapsed_time(b) * 1e-3) / 1e9)
        for name, (dst, src) in (("d2h", (host, dev)), ("h2d", (dev, host))):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            dst.copy_(src, non_blocking=True)
            b.record()
            b.synchronize()
            best[name] = max(best[name], nbytes / (a.elapsed_time(b) * 1e-3) / 1e9)
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        s1.wait_event(a)
        s2.wait_event(a)
        with torch.cuda.stream(s1):
            host.copy_(dev, non_blocking=True)
        with torch.cuda.stream(s2):
            dev2.copy_(host2, non_blocking=True)
        torch.cuda.current_stream().wait_stream(s1)
        torch.cuda.current_stream().wait_stream(s2)
        b.record()
        b.synchronize()
        best["both"] = max(best["both"], nbytes / (a.elapsed_time(b) * 1e-3) / 1e9)
    return best


_FLUSH = {}


def l2_flush(stream) -> None:
    """Writes a buffer twice the size of the 126 MB L2 on `stream`, so that what follows finds
    none of its data cached."""
    buf = _FLUSH.get("buf")
    if buf is None:
        buf = _FLUSH["buf"] = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    with torch.cuda.stream(stream):
        buf.fill_(1)


def time_launches(fn, stream, reps: int, flush: bool = False) -> float:
    """Average CUDA-event duration (s) of `reps` launches queued on `stream`, each bracketed by
    its own pair of events; flush=True clears the L2 before every launch (outside the pair)."""
    pairs = []
    for _ in range(3):
        fn()
    torch.cuda.synchronize()
    for _ in range(reps):
        if flush:
            l2_flush(stream)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        fn()
        b.record(stream)
        pairs.append((a, b))
    torch.cuda.synchronize()
    return sum(a.elapsed_time(b) for a, b in pairs) * 1e-3 / reps


def kernel_rows(kt, prob, peak: float, reps: int = 20, flush: bool = False) -> dict:
    """K1, K2 and the one-pass kernel on a problem's buffers: algorithmic bytes over the
    CUDA-event time of a launch."""
    wl = prob.wl
    by = algorithmic_bytes(wl)
    with torch.cuda.stream(prob.main):
        k1 = time_launches(lambda: kt.kt_hier_reduce(prob.ctx, kt.KT_INTRA, prob.transport, stream=prob.main),
                           prob.main, reps, flush)
        k2 = time_launches(lambda: kt.kt_unpack_scale(prob.ctx, prob.transport, prob.out_ptrs, out_dtype=prob.out_dtype,
                                                      R=1, stream=prob.main), prob.main, reps, flush)
        direct = time_launches(prob.direct, prob.main, reps, flush)
    direct_bytes = wl.K * wl.N * wl.elem_size + wl.N * wl.elem_size

    def row(nbytes, sec):
        return {"us": round(sec * 1e6, 2), "GBps": round(nbytes / sec / 1e9, 1), "frac": round(nbytes / sec / 1e9 / peak, 4),
                "frac_of_nominal_8TBs": round(nbytes / sec / 1e9 / NOMINAL_HBM_GBS, 4), "bytes_per_launch": int(nbytes)}
    return {"k1_intra_reduce": row(by["k1"], k1), "k2_combine_unpack": row(by["k2"], k2),
            "k_direct_sync": row(direct_bytes, direct)}


def large_bucket_roofline(kt, peak: float, K: int = 4, bytes_per_rank: int = 256 << 20, dtype: str = "f32") -> dict:
    """The kernels on one flat bucket per rank of the size the bandwidth target is stated for
    (64 MiB and up): algorithmic bytes over the CUDA-event time of a launch.  The buffers
    exceed the L2 several times over."""
    wl = W.sweep_point(K, bytes_per_rank, dtype)
    prob = Problem(wl, kt)
    out = {"workload": "flat %s bucket, %d ranks x %d MiB in 2 groups" % ("fp32" if dtype == "f32" else "bf16", K,
                                                                          bytes_per_rank >> 20)}
    out.update(kernel_rows(kt, prob, peak))
    kt.kt_destroy(prob.ctx)
    del prob
    torch.cuda.empty_cache()
    return out


LARGE_BUCKETS = [(8, 64 << 20, "f32"), (16, 64 << 20, "f32"), (8, 256 << 20, "f32"), (16, 256 << 20, "f32"),
                 (8, 64 << 20, "bf16"), (16, 64 << 20, "bf16"), (8, 256 << 20, "bf16"), (16, 256 << 20, "bf16")]


def named_config_rows(kt, peak: float) -> dict:
    """The kernels on the other named configurations (the step itself runs on ResNet-18):
    ResNet-50 with bf16 gradients and 8 ranks, MobileNetV2's ragged list with 8 ranks in three
    groups.  The L2 is flushed before every timed launch."""
    out = {"l2": "flushed before every timed launch (a 256 MiB buffer is written outside the event pair)"}
    for name in ("resnet50", "mobilenet_v2"):
        wl = W.by_name(name)
        prob = Problem(wl, kt)
        rows = kernel_rows(kt, prob, peak, flush=True)
        rows["workload"] = "%s: %d tensors, %d elements per rank, %s, K=%d ranks in %d groups, shares %s" % (
            wl.name, wl.T, wl.N, wl.dtype, wl.K, wl.G, prob.shares)
        rows["k1_intra_reduce"]["traffic"] = TRAFFIC_K1.get(name)
        rows["default_route_without_staging"] = "k_direct_sync (one pass)"
        out[name] = rows
        kt.kt_destroy(prob.ctx)
        del prob
        torch.cuda.empty_cache()
    return out


def broadcast_phases(kt, wl, peak: float, chunk_bytes: int) -> dict:
    """Model synchronisation on the same tensor list: root rank 0's parameters to every rank,
    inside its group directly, to the other groups through pinned host memory."""
    dt = torch.float32 if wl.dtype == "f32" else torch.bfloat16
    params = [[t.cuda() for t in W.split_tensors(W.rank_gradients(wl, r, "cuda"), wl.numel)] for r in range(wl.K)]
    ctx = kt.kt_groups_init(wl.group_of, [1] * wl.K, wl.G)
    kt.kt_bucket_pack(ctx, params, wl.bucket_cap_bytes)
    n = kt.kt_plan_query(ctx).transport_numel
    send = torch.zeros(n, dtype=dt, device="cuda")
    pinned = torch.zeros(n, dtype=dt).pin_memory()
    g_root = wl.group_of[0]
    recv = [None if g == g_root else torch.zeros(n, dtype=dt, device="cuda") for g in range(wl.G)]
    main, s1, s2 = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
    k_root = sum(1 for g in wl.group_of if g == g_root)
    es, N = wl.elem_size, wl.N
    send_bytes = N * es * (1 + 1 + (k_root - 1))
    recv_bytes = N * es * ((wl.G - 1) + (wl.K - k_root))
    with torch.cuda.stream(main):
        t_send = time_launches(lambda: kt.kt_bcast_send(ctx, 0, send, stream=main), main, 20)
        t_recv = time_launches(lambda: kt.kt_bcast_recv(ctx, 0, recv, stream=main), main, 20)

        def whole():
            kt.kt_bcast_send(ctx, 0, send, stream=main)
            kt.kt_bcast_relay(ctx, 0, send, pinned, recv, s1, s2, chunk_bytes=chunk_bytes, main_stream=main)
            kt.kt_stage_wait(ctx, kt.KT_H2D, main_stream=main)
            kt.kt_bcast_recv(ctx, 0, recv, stream=main)
        t_all = time_launches(whole, main, 10)
    kt.kt_destroy(ctx)
    return {"what": "broadcast of rank 0's %d tensors (%s) to all %d ranks; %d other group(s) served through "
                    "pinned host memory" % (wl.T, wl.dtype, wl.K, wl.G - 1),
            "k_bcast_send": {"us": round(t_send * 1e6, 2), "GBps": round(send_bytes / t_send / 1e9, 1),
                             "frac": round(send_bytes / t_send / 1e9 / peak, 4), "bytes": send_bytes},
            "k_bcast_recv": {"us": round(t_recv * 1e6, 2), "GBps": round(recv_bytes / t_recv / 1e9, 1),
                             "frac": round(recv_bytes / t_recv / 1e9 / peak, 4), "bytes": recv_bytes},
            "ms_whole": round(t_all * 1e3, 4), "relay_bytes_down": N * es, "relay_bytes_up": N * es * (wl.G - 1)}


def sampler_phase(kt, shares, peak: float, dataset_size: int = 1281167) -> dict:
    """The load-adaptive sampler's index kernel on an ImageNet-sized epoch (1 281 167 indices)
    with the step's shares: every index read once from the epoch's permutation and written once
    into its rank's list."""
    perm = torch.randperm(dataset_size, device="cuda")
    steps = kt.kt_sampler_steps(dataset_size, sum(shares), False)
    out = [torch.empty(steps * b, dtype=torch.int64, device="cuda") for b in shares]
    main = torch.cuda.Stream()
    with torch.cuda.stream(main):
        sec = time_launches(lambda: kt.kt_sampler_indices(perm, dataset_size, shares, out, stream=main), main, 20)
    nbytes = 16 * steps * sum(shares)
    return {"what": "index lists of one epoch of %d samples for shares %s" % (dataset_size, list(shares)),
            "k_sampler": {"us": round(sec * 1e6, 2), "GBps": round(nbytes / sec / 1e9, 1), "frac": round(nbytes / sec / 1e9 / peak, 4),
                          "bytes": nbytes, "note": "20 MB once per epoch: two to three times the fixed cost of a launch; not on the per-step path"}}


def narrow_transport_step(kt, wl, chunk_bytes: int, steps: int) -> dict:
    """The same step with the library's bf16 transport (an extension: partials rounded once
    to bf16, half the bytes on the host link).  Reported beside the headline, never as it."""
    prob = Problem(wl, kt, chunk_bytes=chunk_bytes, transport_dtype=torch.bfloat16)
    with torch.cuda.stream(prob.main):
        for _ in range(3):
            prob.step()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(prob.main)
        for _ in range(steps):
            prob.step(time_k1=True)
        b.record(prob.main)
        torch.cuda.synchronize()
    ms = a.elapsed_time(b) / steps
    out = {"ms_per_step": round(ms, 4), "k1_us": round(prob.k1_seconds() / steps * 1e6, 2),
           "k2_us": round(prob.k2_seconds() / steps * 1e6, 2),
           "staging_bytes_each_way": wl.G * wl.N * 2 if wl.staged else 0,
           "note": "extension, not the paper's method: fp32 accumulation, partials stored as bf16 "
                   "(one extra rounding, <= 2^-8 relative)"}
    kt.kt_destroy(prob.ctx)
    return out


def recorded_step(kt, prob, steps: int) -> dict:
    """The step recorded once and replayed with one submission per step (kt_graph_*): what the
    sync costs when the host-side cost of the individual calls is out of the way."""
    main = prob.main
    torch.cuda.synchronize()
    kt.kt_graph_begin(prob.ctx, main)
    prob.step()
    graph = kt.kt_graph_end(prob.ctx, main)
    for _ in range(3):
        kt.kt_graph_launch(graph, main)
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(main)
    for _ in range(steps):
        kt.kt_graph_launch(graph, main)
    b.record(main)
    torch.cuda.synchronize()
    out = {"ms_per_step": round(a.elapsed_time(b) / steps, 4), "recorded_operations": kt.kt_graph_nodes(graph)}
    kt.kt_graph_destroy(graph)
    return out


def free_port() -> int:
    import socket
    with socket.socket(socket.AF_INET, socket.SOCK_STREAM) as sock:
        sock.bind(("127.0.0.1", 0))
        return sock.getsockname()[1]


def launch_ranks(n: int, script: str, script_args, need_devices: bool = True, capture: bool = False):
    """Starts `n` ranks of `script` on this node, one process per GPU, the way a multi-GPU run
    of this benchmark is launched from outside: `python -m torch.distributed.run --nnodes=1
    --nproc-per-node n --master-addr 127.0.0.1 --master-port P script args...`.  Refuses when
    fewer than `n` CUDA devices are visible (never fewer replicas than asked for).  Returns the
    finished process (capture=True keeps its output instead of passing it through)."""
    if need_devices:
        have = torch.cuda.device_count()
        if have < n:
            raise SystemExit("bench.py: --gpus %d was asked for but %d CUDA device(s) are visible; refusing to "
                             "run fewer replicas than requested" % (n, have))
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(n),
           "--master-addr", "127.0.0.1", "--master-port", str(free_port()), script] + list(script_args)
    kw = dict(stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True) if capture else {}
    return subprocess.run(cmd, **kw)


def init_ranks(backend: str):
    """Reads the launcher's environment.  Returns (world, rank, local_rank, dist or None); with
    more than one rank the process group is up when this returns.  NCCL's own start-up log is
    kept (in a file per process, so that standard output stays one JSON line): it is the record
    of how many ranks the communicator really has."""
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world == 1:
        return world, rank, local, None
    import torch.distributed as dist
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    if backend == "nccl":
        os.environ.setdefault("NCCL_DEBUG", "INFO")
        os.environ.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
        os.environ.setdefault("NCCL_DEBUG_FILE", os.path.join(tempfile.gettempdir(), "kt_bench_nccl_%h_%p.log"))
        torch.cuda.set_device(local)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    else:
        dist.init_process_group(backend, rank=rank, world_size=world)
    return world, rank, local, dist


def nccl_log_summary() -> dict:
    """What this process's NCCL start-up log says about the communicator (ranks, version, whether
    in-switch reduction was set up); empty when NCCL wrote no log."""
    import glob
    import re
    pattern = os.environ.get("NCCL_DEBUG_FILE", "")
    if not pattern:
        return {}
    path = pattern.replace("%p", str(os.getpid()))
    out = {}
    for name in glob.glob(path.replace("%h", "*")):
        try:
            text = open(name, errors="replace").read()
        except OSError:
            continue
        m = re.search(r"nranks (\d+)", text)
        if m:
            out["nranks"] = int(m.group(1))
        m = re.search(r"NCCL version ([0-9.]+)", text)
        if m:
            out["version"] = m.group(1)
        out["nvls"] = bool(re.search(r"NVLS", text))
        out["log"] = name
    return out


def recorded_launches(kt, prob, fn, n: int = 20, reps: int = 10) -> float:
    """Seconds per launch when `n` launches of one kernel are recorded once and replayed: no
    event pair and no host call between the launches, so what CUDA events add around a single
    short launch (about 5 us) is spread over n.  Meaningful for roofline purposes only when the
    kernel's inputs exceed the L2."""
    main = prob.main
    fn()
    torch.cuda.synchronize()
    kt.kt_graph_begin(prob.ctx, main)
    for _ in range(n):
        fn()
    graph = kt.kt_graph_end(prob.ctx, main)
    times = []
    for i in range(reps + 2):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(main)
        kt.kt_graph_launch(graph, main)
        b.record(main)
        torch.cuda.synchronize()
        if i >= 2:
            times.append(a.elapsed_time(b) * 1e-3 / n)
    kt.kt_graph_destroy(graph)
    return statistics.median(times)


def max_over_ranks(seconds, dist, device) -> list:
    """Every replica times its own steps; the job is as slow as its slowest replica."""
    if dist is None:
        return list(seconds)
    t = torch.tensor(list(seconds), device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def job_throughput(bytes_per_step: int, steps: int, world: int, slowest_seconds: float) -> float:
    """Whole-job GB/s: all replicas' bytes over the slowest replica's time (weak scaling)."""
    return world * bytes_per_step * steps / slowest_seconds / 1e9


def run_ours(args) -> dict:
    from paper_2505_10183_b200 import build as kt_build
    if kt_build.is_stale():
        if int(os.environ.get("LOCAL_RANK", "0")) == 0:
            kt_build.build()                 # in-tree, sm_100a; a failed build ends the run
        else:                                # the other ranks wait for rank 0's build
            deadline = time.time() + 600
            while kt_build.is_stale() and time.time() < deadline:
                time.sleep(0.5)
    from paper_2505_10183_b200 import binding as kt

    world, rank, local, dist = init_ranks("nccl")
    torch.cuda.set_device(local)

    wl = W.by_name(args.workload)
    prob = Problem(wl, kt, chunk_bytes=args_chunk(args))
    nbytes = algorithmic_bytes(wl)
    link = host_link_bandwidth(chunk_bytes=args_chunk(args)) if wl.staged else None

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    with torch.cuda.stream(prob.main):
        for _ in range(args.warmup):
            prob.step()
        barrier()
        sampler = ClockSampler(local)
        if rank == 0:
            sampler.start()
        launches0 = kt.kt_launch_count(prob.ctx)
        t_start, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        marks = []
        t_start.record(prob.main)
        for _ in range(args.steps):
            prob.step(time_k1=True)
            m = torch.cuda.Event(enable_timing=True)
            m.record(prob.main)
            marks.append(m)
        t_end.record(prob.main)
        barrier()
        clocks = sampler.stop() if rank == 0 else None
        launches = kt.kt_launch_count(prob.ctx) - launches0
        total_s = t_start.elapsed_time(t_end) * 1e-3
        per_step = [a.elapsed_time(b) for a, b in zip([t_start] + marks[:-1], marks)]
        k1_s = prob.k1_seconds()
        direct_s = time_launches(prob.direct, prob.main, args.steps)
        recorded = recorded_step(kt, prob, args.steps)
        k1_seq_s = recorded_launches(kt, prob, lambda: kt.kt_hier_reduce(prob.ctx, kt.KT_INTRA, prob.transport,
                                                                          bucket=-1, stream=prob.main))

        # end to end: gradients start in pinned host memory, the result ends there
        e2e = run_e2e(prob, kt, args, barrier)

    total_s, e2e["seconds"] = max_over_ranks([total_s, e2e["seconds"]], dist, "cuda")

    peak, peak_kind = measured_peak()
    k1_launch_bytes = nbytes["k1"]                                # one launch per step covers all buckets
    k1_launch_s = k1_s / args.steps
    k2_launch_s = prob.k2_seconds() / args.steps
    achieved = k1_launch_bytes / k1_launch_s / 1e9
    relay_s = total_s / args.steps - k1_launch_s - k2_launch_s
    value = job_throughput(nbytes["step"], args.steps, world, total_s)
    result = {
        "metric": METRIC, "value": round(value, 2), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": round(total_s / args.steps * 1e3, 4),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": wl.dtype,
        "data": "synthetic",
        "config": {
            "workload": "%s: %d tensors, %d elements per rank, K=%d ranks in %d groups, shares %s, "
                        "%d buckets of <= 25 MiB%s" % (wl.name, wl.T, wl.N, wl.K, wl.G, prob.shares,
                                                      prob.plan.n_buckets,
                                                      ", fp32 partials relayed through pinned host memory"
                                                      if wl.staged else ""),
            "bytes_per_step": nbytes["step"],
            "bytes_counted": "algorithmic HBM bytes of the two kernels (K*N*s + 4*G*N read/written by the "
                             "fused reduce, 4*G*N + N*s by combine+unpack); staging copies add time, not bytes",
            "staging_bytes_each_way": nbytes["stage_each_way"],
            "l2": ("inputs (%.0f MB) exceed the 126 MB L2 and every step streams all buffers through it"
                   if wl.K * wl.N * wl.elem_size > (126 << 20) else
                   "inputs (%.0f MB) fit the 126 MB L2 and nothing flushes it between steps: this workload's "
                   "figures are not roofline figures (the default workload's inputs exceed the L2)")
                  % (wl.K * wl.N * wl.elem_size / 1e6),
            "multi_gpu": "independent replicas, no collective",
            "launches_per_step": "1 fused reduce + 1 combine/unpack over all buckets; relay of the whole "
                                 "transport in %d MiB chunks on two copy streams" % (prob.chunk_bytes >> 20),
            "phases": {"k1_us": round(k1_launch_s * 1e6, 2), "k2_us": round(k2_launch_s * 1e6, 2),
                       "k2_GBps": round(nbytes["k2"] / k2_launch_s / 1e9, 1),
                       "relay_ms": round(relay_s * 1e3, 4) if wl.staged else 0.0,
                       "relay_GBps_each_way": round(nbytes["stage_each_way"] / relay_s / 1e9, 1) if wl.staged else None,
                       "direct_us": round(direct_s * 1e6, 2),
                       "direct_note": "kt_sync_direct: the same arithmetic in one pass without transport or "
                                      "relay (what a collective inside one vendor group costs); not part of the step"},
            "recorded_step": recorded,
            "latency_ms": {"p50": round(statistics.median(per_step), 4),
                           "p95": round(sorted(per_step)[int(0.95 * (len(per_step) - 1))], 4)},
        },
        "roofline": {"bound": "hbm", "kernel": "k1_intra_reduce", "achieved": round(achieved, 1),
                     "peak": peak, "unit": "GB/s", "frac": round(achieved / peak, 4),
                     "peak_kind": peak_kind, "frac_of_nominal_8TBs": round(achieved / NOMINAL_HBM_GBS, 4),
                     "bytes_per_launch": int(k1_launch_bytes), "us_per_launch": round(k1_launch_s * 1e6, 2),
                     "traffic": TRAFFIC_K1.get(wl.name), "traffic_source": TRAFFIC_SOURCE,
                     "in_recorded_sequence": {
                         "us_per_launch": round(k1_seq_s * 1e6, 2),
                         "achieved": round(k1_launch_bytes / k1_seq_s / 1e9, 1),
                         "frac": round(k1_launch_bytes / k1_seq_s / 1e9 / peak, 4),
                         "how": "the same launch recorded 20 times and replayed (median of 10 replays / 20): no event "
                                "pair and no host call between launches; inputs (%.0f MB) %s; beside the "
                                "headline figures above, which bracket every launch with its own events"
                                % (wl.K * wl.N * wl.elem_size / 1e6,
                                   "exceed the L2" if wl.K * wl.N * wl.elem_size > (126 << 20) else
                                   "do NOT exceed the 126 MB L2, so part of them is re-read from it and this figure "
                                   "flatters the kernel")}},
        "e2e": {"value": round(job_throughput(nbytes["step"], args.steps, world, e2e["seconds"]), 2), "unit": UNIT,
                "h2d_bytes_per_step": e2e["h2d"], "d2h_bytes_per_step": e2e["d2h"],
                "ms_per_step": round(e2e["seconds"] / args.steps * 1e3, 4),
                "layout": "one pinned host buffer and one device buffer per rank, tensors at multiples of "
                          "64 elements (views); per bucket K copies in and 1 copy out through kt_copy_tensors, "
                          "buckets pipelined over the two directions of the host link"},
        "gpu_launches": int(launches),
        "clocks": clocks,
    }
    if link is not None:
        result["host_link"] = {"d2h_GBps": round(link["d2h"], 1), "h2d_GBps": round(link["h2d"], 1),
                               "both_ways_at_once_GBps_each": round(link["both"], 1),
                               "relay_frac_of_both_ways": round(nbytes["stage_each_way"] / relay_s / 1e9 / link["both"], 3),
                               "both_ways_in_relay_chunks_GBps_each": round(link["both_chunked"], 1),
                               "relay_frac_of_both_ways_in_relay_chunks": round(
                                   nbytes["stage_each_way"] / relay_s / 1e9 / link["both_chunked"], 3),
                               "how": "pinned copies of 256 MiB, best of 10; both ways = one copy down and one up on "
                                      "two streams at the same time; in relay chunks = the same bytes as independent "
                                      "copies of the relay's chunk size (a relay must work in chunks: the way up of a "
                                      "chunk starts when its way down is done)"}
    if rank == 0 and world == 1 and not args.no_large_bucket:
        result["roofline_large_bucket"] = large_bucket_roofline(kt, peak)
        result["roofline_large_bucket"]["more"] = [large_bucket_roofline(kt, peak, K, nb, dt) for K, nb, dt in LARGE_BUCKETS]
        result["configs"] = named_config_rows(kt, peak)
        result["broadcast"] = broadcast_phases(kt, wl, peak, args_chunk(args))
        result["bf16_transport"] = narrow_transport_step(kt, wl, args_chunk(args), min(args.steps, 20))
        result["sampler"] = sampler_phase(kt, prob.shares, peak)
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        result["cpu_baseline"] = cpu_baseline(wl, prob.shares, budget_s=args.cpu_seconds)
    if dist is not None:
        result["nccl"] = nccl_log_summary()
        result["nccl"]["used_for"] = "the barriers around the timed region and the max over ranks; no data-path collective"
        dist.destroy_process_group()
    return result if rank == 0 else None


# dram__bytes_read.sum + dram__bytes_write.sum per launch of the fused reduce on each named
# workload, from ncu captures of the kernel as committed (not measured in this run: a run under
# a profiler reports no times).  A workload without a capture reports null.
TRAFFIC_K1 = {"resnet18": 216022272, "mobilenet_v2": 120217856, "resnet50": 560153856}
TRAFFIC_SOURCE = ("ncu --set full captures of the fused reduce as committed, first launch: profiles/k1_k2_resnet18.md, "
                  "profiles/k1_k2_mobilenet_v2_resnet50.md (read + write bytes; below the algorithmic bytes because part "
                  "of the output is still dirty in the 126 MB L2 when a 27-92 us kernel ends)")


def args_chunk(args) -> int:
    return int(getattr(args, "relay_chunk_mib", 4)) << 20


class HostResidentStep:
    """The end-to-end arm: every rank's gradients start in pinned host memory, the reduced
    gradients end there.

    Host side: one pinned buffer per rank holding that rank's tensors, each at a multiple of 64
    elements; device side: the same layout, the per-parameter tensors being views.  A bucket of a
    rank is then one contiguous range and crosses the host link in one copy (with hundreds of
    small tensors a copy per tensor would cost more than the bytes).  The step is pipelined
    bucket by bucket over the two directions of the link: while the gradients of bucket b+1
    still come up, bucket b is reduced and its partials already go down; the reduced gradients
    of a bucket go down while the partials of the next come back up."""

    def __init__(self, wl, kt, chunk_bytes: int, device_values: bool = True):
        self.wl, self.kt = wl, kt
        prob = self.prob = Problem(wl, kt, device_values=device_values, chunk_bytes=chunk_bytes, arena=True)
        self.host_in = [a.cpu().pin_memory() for a in prob.grad_arenas]
        self.host_out = torch.zeros_like(prob.out_arena, device="cpu").pin_memory()
        for a in prob.grad_arenas:       # whatever reaches the kernels must have crossed the link
            a.zero_()
        es = prob.grad_arenas[0].element_size()
        self.copies_in, self.copies_out, self.h2d_bytes, self.d2h_bytes = [], [], 0, 0
        for b in range(prob.plan.n_buckets):
            ts = [t for t in range(wl.T) if prob.plan.bucket_of[t] == b]
            lo, hi = min(ts), max(ts)
            off = prob.arena_starts[lo] * es
            size = (prob.arena_starts[hi] + -(-wl.numel[hi] // 64) * 64) * es - off
            P = kt.PtrArray.from_addresses
            self.copies_in.append((P([a.data_ptr() + off for a in prob.grad_arenas], prob.grad_arenas),
                                   P([h.data_ptr() + off for h in self.host_in], self.host_in), [size] * wl.K))
            self.copies_out.append((P([self.host_out.data_ptr() + off], self.host_out),
                                    P([prob.out_arena.data_ptr() + off], prob.out_arena), [size]))
            self.h2d_bytes += size * wl.K
            self.d2h_bytes += size
        self.up = prob.side_h2d if wl.staged else torch.cuda.Stream()
        self.down = prob.side_d2h if wl.staged else torch.cuda.Stream()

    def step(self):
        kt, prob, wl = self.kt, self.prob, self.wl
        main, up, down, ctx = prob.main, self.up, self.down, prob.ctx
        nb = prob.plan.n_buckets
        start = torch.cuda.Event()
        start.record(main)
        up.wait_event(start)
        down.wait_event(start)
        arrived = []
        for b in range(nb):
            kt.kt_copy_tensors(*self.copies_in[b], kt.KT_H2D, stream=up)
            e = torch.cuda.Event()
            e.record(up)
            arrived.append(e)
        for b in range(nb):
            main.wait_event(arrived[b])
            kt.kt_hier_reduce(ctx, kt.KT_INTRA, prob.transport, bucket=b, stream=main)
            if wl.staged:
                kt.kt_relay_through_host(ctx, prob.transport, prob.pinned, prob.recv, down, up, bucket=b,
                                         chunk_bytes=prob.chunk_bytes, main_stream=main)
        for b in range(nb):
            if wl.staged:
                kt.kt_stage_wait(ctx, kt.KT_H2D, bucket=b, main_stream=main)
            kt.kt_unpack_scale(ctx, prob.recv if wl.staged else prob.transport, prob.out_ptrs, scale=1.0, bucket=b,
                               out_dtype=prob.out_dtype, R=1, stream=main)
            e = torch.cuda.Event()
            e.record(main)
            down.wait_event(e)
            kt.kt_copy_tensors(*self.copies_out[b], kt.KT_D2H, stream=down)
        done = torch.cuda.Event()
        done.record(down)
        main.wait_event(done)       # the step ends when the reduced gradients are on the host

    def result_tensors(self):
        """The reduced per-parameter gradients as they arrived in pinned host memory."""
        return [self.host_out[s:s + m] for s, m in zip(self.prob.arena_starts, self.wl.numel)]


def run_e2e(prob, kt, args, barrier) -> dict:
    """Same step, but every step first copies all ranks' gradients from pinned host memory
    to the device and ends with the reduced gradients copied back to pinned host memory."""
    wl = prob.wl
    del prob
    arm = HostResidentStep(wl, kt, args_chunk(args))
    main = arm.prob.main
    for _ in range(max(1, min(args.warmup, 3))):
        arm.step()
    barrier()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(main)
    for _ in range(args.steps):
        arm.step()
    b.record(main)
    barrier()
    if not bool(arm.host_out.any()):
        raise RuntimeError("end-to-end arm: the result buffer on the host is all zero")
    kt.kt_destroy(arm.prob.ctx)
    return {"seconds": a.elapsed_time(b) * 1e-3, "h2d": arm.h2d_bytes, "d2h": arm.d2h_bytes}


# ----------------------------------------------------------------------------- one rank per GPU
def sharded_workload(name: str, world: int):
    """The named tensor list with one rank per GPU: the first half of the ranks is one vendor
    group, the second half a slower one (step times 1.0 and 1.6, global batch 256)."""
    base = W.by_name(name)
    first = max(1, world // 2)
    group_of = [0] * first + [1] * (world - first)
    times = [1.0] * first + [1.6] * (world - first)
    return W.Workload(base.name + "_sharded", base.config_id, base.shapes, base.dtype, group_of, None,
                      step_times=times, global_batch=256, bucket_cap_bytes=base.bucket_cap_bytes, staged=world > first)


def run_sharded(args) -> dict:
    """`--sharded`: every GPU is one rank and reduces its share of every bucket from its group
    mates' gradients (peer-mapped), relays only that share through host memory, and writes its
    share of the result into every group mate's tensors.  Timed on the device (events on the
    rank's stream around the K steps, host barriers included), maximum over ranks."""
    from paper_2505_10183_b200 import binding as kt
    from paper_2505_10183_b200.sharded import ShardedSync
    import torch.distributed as dist
    # the ranks talk to each other on the host only (handles and names at set-up, then the
    # shared-memory barrier): a gloo group is all this arm needs
    world, rank, local, started = init_ranks("gloo")
    torch.cuda.set_device(local)
    if started is None:
        dist.init_process_group("gloo", rank=0, world_size=1, init_method="tcp://127.0.0.1:%d" % free_port())
    host_group = None
    wl = sharded_workload(args.workload, world)
    shares = kt.kt_schedule(wl.step_times, wl.global_batch)
    dt = torch.float32 if wl.dtype == "f32" else torch.bfloat16
    grads = [t.cuda() for t in W.split_tensors(W.rank_gradients(wl, rank, "cuda"), wl.numel)]
    outs = [torch.zeros(m, dtype=dt, device="cuda") for m in wl.numel]
    job = ShardedSync(rank, wl.group_of, shares, grads, outs, wl.bucket_cap_bytes, host_group=host_group)
    M, G, s = len(job.members), wl.G, wl.elem_size
    mine = sum(kt.kt_shard_query(job.ctx, b)[1] for b in job.buckets)          # transport elements of my shares
    if G == 1:
        my_bytes = M * mine * s + M * mine * s
    else:
        my_bytes = (M * mine * s + 4 * mine) + (4 * G * mine + M * mine * s)
    for _ in range(args.warmup):
        job.step()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(job.main)
    for _ in range(args.steps):
        job.step()
    b.record(job.main)
    torch.cuda.synchronize()
    t = torch.tensor([a.elapsed_time(b) * 1e-3, 0.0], dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX, group=host_group)
    total = torch.tensor([float(my_bytes)], dtype=torch.float64)
    dist.all_reduce(total, op=dist.ReduceOp.SUM, group=host_group)
    seconds = float(t[0])
    if not all(bool(torch.isfinite(o).all()) and bool(o.any()) for o in outs if o.numel() > 64):
        raise RuntimeError("sharded arm: an output tensor was not written")
    job_buckets = list(job.buckets)
    job.close()
    dist.destroy_process_group()
    if rank != 0:
        return None
    return {"metric": METRIC, "arm": "sharded", "value": round(float(total[0]) * args.steps / seconds / 1e9, 2),
            "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": round(seconds / args.steps * 1e3, 4), "higher_is_better": True, "scaling": "strong",
            "vs_baseline": None, "dtype": wl.dtype, "data": "synthetic",
            "config": {"workload": "%s: %d tensors, %d elements per rank, one rank per GPU, groups %s, shares %s"
                                   % (wl.name, wl.T, wl.N, wl.group_of, shares),
                       "bytes_counted": "per GPU: M*n*s read + 4*n written by the fused reduce over its share of n "
                                        "elements, 4*G*n read + M*n*s written by combine+unpack (M group members); "
                                        "summed over GPUs",
                       "host_barriers_per_step": 2 + (len(job_buckets) if G > 1 else 0),
                       "note": "timing includes the host-side barriers between ranks"}}


# ----------------------------------------------------------------------------- the oracle as CPU baseline
def oracle_inputs(wl):
    host = []
    for r in range(wl.K):
        flat = W.rank_gradients(wl, r, "cpu")
        host.append([W.as_numpy(t) for t in W.split_tensors(flat, wl.numel)])
    return host


def cpu_baseline(wl, shares, budget_s: float = 12.0) -> dict:
    """The oracle as it stands, one thread, on the full workload, repeated for about
    budget_s seconds; GB/s over the same algorithmic bytes as the GPU path."""
    from oracle import kt_oracle as oracle
    host = oracle_inputs(wl)
    dt = 0 if wl.dtype == "f32" else 1
    nbytes = algorithmic_bytes(wl)["step"]
    oracle.sync_step(host, wl.numel, dt, wl.group_of, shares, wl.G, wl.bucket_cap_bytes)   # warm
    times = []
    t_all = time.perf_counter()
    while time.perf_counter() - t_all < budget_s or len(times) < 2:
        t0 = time.perf_counter()
        oracle.sync_step(host, wl.numel, dt, wl.group_of, shares, wl.G, wl.bucket_cap_bytes)
        times.append(time.perf_counter() - t0)
    best = statistics.median(times)
    out = {"value": round(nbytes / best / 1e9, 3), "unit": UNIT, "cores": 1, "kind": "oracle",
           "sample": "full %s step (all %d elements x %d ranks), %d repetitions, median" %
                     (wl.name, wl.N, wl.K, len(times)),
           "ms_per_step": round(best * 1e3, 2), "host_cores_available": os.cpu_count()}
    # beside it: the same per-element loops cut into static slices over all host cores (results
    # are identical because the order inside an element does not change)
    import numpy as np
    cores = os.cpu_count() or 1
    if cores > 1:
        flat = [np.concatenate(h) for h in host]
        many = []
        t_all = time.perf_counter()
        while time.perf_counter() - t_all < min(4.0, budget_s / 3) or len(many) < 2:
            t0 = time.perf_counter()
            oracle.sync_step_flat_threads(flat, dt, wl.group_of, shares, wl.G, 1.0, dt, cores)
            many.append(time.perf_counter() - t0)
        m = statistics.median(many)
        out["all_cores"] = {"value": round(nbytes / m / 1e9, 3), "cores": cores, "ms_per_step": round(m * 1e3, 2),
                            "sample": "the same elements as one flat tensor per rank, %d static slices" % cores}
    return out


def run_reference(args) -> dict:
    """The reference arm: the CPU oracle, unmodified, on the machine's host cores."""
    if int(os.environ.get("RANK", "0")) != 0:
        return None
    from oracle import kt_oracle as oracle
    wl = W.by_name(args.workload)
    shares = list(wl.shares) if wl.shares is not None else oracle.schedule(wl.step_times, wl.global_batch).tolist()
    host = oracle_inputs(wl)
    dt = 0 if wl.dtype == "f32" else 1
    nbytes = algorithmic_bytes(wl)["step"]
    for _ in range(args.warmup):
        oracle.sync_step(host, wl.numel, dt, wl.group_of, shares, wl.G, wl.bucket_cap_bytes)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.sync_step(host, wl.numel, dt, wl.group_of, shares, wl.G, wl.bucket_cap_bytes)
    total = time.perf_counter() - t0
    value = round(nbytes * args.steps / total / 1e9, 3)
    sample = "full %s step on one host thread, host-resident inputs" % wl.name
    return {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT,
        "n_gpus": max(int(os.environ.get("WORLD_SIZE", "1")), int(getattr(args, "gpus", 1))),
        "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": round(total / args.steps * 1e3, 3), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": wl.dtype, "data": "synthetic",
        "config": {"workload": "%s: %d tensors, %d elements per rank, K=%d ranks in %d groups, shares %s"
                               % (wl.name, wl.T, wl.N, wl.K, wl.G, shares), "bytes_per_step": nbytes},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }


# ----------------------------------------------------------------------------- bucket sweep
def run_sweep(args) -> None:
    """Fused reduce (K1) and combine+unpack (K2) alone on flat buffers, 4 KB .. 1 GB per rank.
    Buffers that fit the L2 are rotated over enough copies to exceed it."""
    from paper_2505_10183_b200 import binding as kt
    torch.cuda.set_device(0)
    peak, peak_kind = measured_peak()
    l2 = 126 << 20
    sizes = [4 << 10 << (2 * i) for i in range(10)]
    for dtype in ("f32", "bf16"):
        for K in (2, 4, 8, 16):
            for nb in sizes:
                if args.sweep_max_bytes and nb > args.sweep_max_bytes:
                    continue
                wl = W.sweep_point(K, nb, dtype)
                by = algorithmic_bytes(wl)
                foot = by["k1"] + wl.N * wl.elem_size
                copies = max(1, min(64, -(-2 * l2 // foot)))
                probs = [Problem(wl, kt) for _ in range(copies)]
                main = torch.cuda.Stream()
                reps = max(5, min(200, int(2e9 // max(by["k1"], 1))))
                res = {}
                with torch.cuda.stream(main):
                    for name in ("k1", "k2"):
                        def launch(p):
                            if name == "k1":
                                kt.kt_hier_reduce(p.ctx, kt.KT_INTRA, p.transport, stream=main)
                            else:
                                kt.kt_unpack_scale(p.ctx, p.transport, p.out_ptrs, out_dtype=p.out_dtype, R=1,
                                                   stream=main)
                        for i in range(3 * copies):
                            launch(probs[i % copies])
                        torch.cuda.synchronize()
                        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                        a.record(main)
                        for i in range(reps):
                            launch(probs[i % copies])
                        b.record(main)
                        torch.cuda.synchronize()
                        us = a.elapsed_time(b) * 1e3 / reps
                        res[name] = {"us": round(us, 2), "GBps": round(by[name] / us / 1e3, 1),
                                     "frac": round(by[name] / us / 1e3 / peak, 4)}
                print(json.dumps({"sweep": wl.name, "K": K, "dtype": dtype, "bytes_per_rank": nb,
                                  "shares": wl.shares, "rotated_copies": copies, "peak": peak,
                                  "peak_kind": peak_kind, **res}), flush=True)
                for p in probs:
                    kt.kt_destroy(p.ctx)
                del probs
                torch.cuda.empty_cache()


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="resnet18", choices=["tiny", "resnet18", "resnet50", "mobilenet_v2"])
    ap.add_argument("--sweep", action="store_true")
    ap.add_argument("--sweep-max-bytes", type=int, default=0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-large-bucket", action="store_true")
    ap.add_argument("--cpu-seconds", type=float, default=12.0)
    ap.add_argument("--relay-chunk-mib", type=int, default=4)
    ap.add_argument("--sharded", action="store_true",
                    help="one rank per GPU with element-range shares instead of independent replicas")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.sweep:
        run_sweep(args)
        return
    if args.gpus < 1:
        raise SystemExit("bench.py: --gpus must be >= 1")
    env_world = os.environ.get("WORLD_SIZE")
    if env_world is not None and args.gpus not in (1, int(env_world)):
        raise SystemExit("bench.py: --gpus %d disagrees with WORLD_SIZE=%s set by the launcher" % (args.gpus, env_world))
    if args.impl == "ours" and env_world is None and args.gpus > 1:
        # not started by a launcher: start the N ranks here, one process per GPU
        sys.exit(launch_ranks(args.gpus, os.path.abspath(__file__), sys.argv[1:]).returncode)
    if args.sharded and args.impl == "ours":
        out = run_sharded(args)
    else:
        out = run_reference(args) if args.impl == "reference" else run_ours(args)
    if out is not None:
        print(json.dumps(out), flush=True)


if __name__ == "__main__":
    main()
