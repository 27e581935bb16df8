"""Runs a few launches of the two hot kernels on one small flat case, for profilers.

    python -m paper_2505_10183_b200.profile_case --K 4 --bytes 67108864 --dtype f32 --launches 3

One flat gradient buffer per rank (ranks 0..K/2-1 in group 0, the rest in group 1), the
fused intra-group reduce, the combine+unpack kernel, the one-pass direct kernel and the two
broadcast kernels launched `launches` times each, after one warm-up launch of each.  Prints
the CUDA-event time of every launch.
"""
from __future__ import annotations

import argparse
import json

import torch

from . import binding as kt
from . import workloads as W


def fixed_cost(args) -> None:
    """What CUDA events see around one launch when the queue is kept full (a long fill kernel
    runs first, so the launch under test is already queued when the GPU gets to it): two
    events with nothing between them, then the fused reduce and the combine+unpack on the
    40 KB `tiny` list (all fixed cost: event pair, launch, one chain of dependent loads, drain)
    and on the chosen workload, beside the time the copy peak would allow for its bytes."""
    import statistics
    torch.cuda.set_device(0)
    blocker = torch.empty(1 << 30, dtype=torch.uint8, device="cuda")

    def timed(fn, reps=20):
        out = []
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        for _ in range(reps):
            blocker.fill_(1)
            blocker.fill_(2)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            fn()
            b.record()
            torch.cuda.synchronize()
            out.append(a.elapsed_time(b) * 1e3)
        return {"median_us": round(statistics.median(out), 2), "min_us": round(min(out), 2)}

    res = {"two_events_back_to_back": timed(lambda: None)}
    names = ["tiny"] + ([args.workload] if args.workload else [])
    for name in names:
        wl = W.by_name(name)
        shares = list(wl.shares) if wl.shares is not None else kt.kt_schedule(wl.step_times, wl.global_batch)
        dt = torch.float32 if wl.dtype == "f32" else torch.bfloat16
        grads = [[t.cuda() for t in W.split_tensors(W.rank_gradients(wl, r, "cuda"), wl.numel)] for r in range(wl.K)]
        ctx = kt.kt_groups_init(wl.group_of, shares, wl.G)
        kt.kt_bucket_pack(ctx, grads, wl.bucket_cap_bytes)
        n = kt.kt_plan_query(ctx).transport_numel
        transport = kt.kt_ptrs(list(torch.zeros(wl.G, n, device="cuda")))
        out = kt.kt_ptrs([torch.zeros(m, dtype=dt, device="cuda") for m in wl.numel])
        odt = kt.KT_F32 if wl.dtype == "f32" else kt.KT_BF16
        k1_bytes = wl.K * wl.N * wl.elem_size + wl.G * wl.N * 4
        k2_bytes = wl.G * wl.N * 4 + wl.N * wl.elem_size
        res[name] = {"k1": timed(lambda: kt.kt_hier_reduce(ctx, kt.KT_INTRA, transport)),
                     "k2": timed(lambda: kt.kt_unpack_scale(ctx, transport, out, out_dtype=odt, R=1)),
                     "k1_bytes": k1_bytes, "k2_bytes": k2_bytes}
        kt.kt_destroy(ctx)
    print(json.dumps(res))


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--K", type=int, default=4)
    ap.add_argument("--bytes", type=int, default=64 << 20, help="bytes per rank")
    ap.add_argument("--dtype", default="f32", choices=["f32", "bf16"])
    ap.add_argument("--launches", type=int, default=3)
    ap.add_argument("--workload", default=None, help="a named workload instead of a flat case")
    ap.add_argument("--fixed-cost", action="store_true",
                    help="measure what a launch costs besides streaming: see fixed_cost()")
    args = ap.parse_args()
    if args.fixed_cost:
        fixed_cost(args)
        return

    torch.cuda.set_device(0)
    wl = W.by_name(args.workload) if args.workload else W.sweep_point(args.K, args.bytes, args.dtype)
    shares = list(wl.shares) if wl.shares is not None else kt.kt_schedule(wl.step_times, wl.global_batch)
    dt = torch.float32 if wl.dtype == "f32" else torch.bfloat16
    grads = [[t.cuda() for t in W.split_tensors(W.rank_gradients(wl, r, "cuda"), wl.numel)] for r in range(wl.K)]
    ctx = kt.kt_groups_init(wl.group_of, shares, wl.G)
    kt.kt_bucket_pack(ctx, grads, 1 << 62)
    n = kt.kt_plan_query(ctx).transport_numel
    transport = kt.kt_ptrs([torch.zeros(n, device="cuda") for _ in range(wl.G)])
    out = kt.kt_ptrs([torch.zeros(m, dtype=dt, device="cuda") for m in wl.numel])
    odt = kt.KT_F32 if wl.dtype == "f32" else kt.KT_BF16
    send = torch.zeros(n, dtype=dt, device="cuda")
    recv = [None if g == wl.group_of[0] else send for g in range(wl.G)]
    steps = [("k1_us", lambda: kt.kt_hier_reduce(ctx, kt.KT_INTRA, transport)),
             ("k2_us", lambda: kt.kt_unpack_scale(ctx, transport, out, out_dtype=odt, R=1)),
             ("direct_us", lambda: kt.kt_sync_direct(ctx, out, out_dtype=odt, R=1)),
             ("bcast_send_us", lambda: kt.kt_bcast_send(ctx, 0, send)),
             ("bcast_recv_us", lambda: kt.kt_bcast_recv(ctx, 0, recv))]
    times = {name: [] for name, _ in steps}
    for i in range(args.launches + 1):
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(len(steps) + 1)]
        ev[0].record()
        for j, (_, fn) in enumerate(steps):
            fn()
            ev[j + 1].record()
        torch.cuda.synchronize()
        if i:
            for j, (name, _) in enumerate(steps):
                times[name].append(round(ev[j].elapsed_time(ev[j + 1]) * 1e3, 2))
    k1_bytes = wl.K * wl.N * wl.elem_size + wl.G * wl.N * 4
    k2_bytes = wl.G * wl.N * 4 + wl.N * wl.elem_size
    print(json.dumps({"case": wl.name, "k1_bytes": k1_bytes, "k2_bytes": k2_bytes, **times}))
    kt.kt_destroy(ctx)


if __name__ == "__main__":
    main()
