"""Shared helpers for the GPU parity tests: build a workload on the device, run it
through the C-ABI binding, run the oracle on host copies of the same bytes."""
from __future__ import annotations

import numpy as np
import torch

from paper_2505_10183_b200 import workloads as W

TORCH_DT = {"f32": torch.float32, "bf16": torch.bfloat16}
ORACLE_DT = {"f32": 0, "bf16": 1}


def device_gradients(wl, misalign: int = 0):
    """Per-rank per-tensor device gradients from the CPU generators (same bytes feed the
    oracle).  misalign > 0 shifts every tensor by that many elements inside a larger
    allocation, so that base pointers are only element aligned."""
    host, dev = [], []
    for r in range(wl.K):
        flat = W.rank_gradients(wl, r, "cpu")
        ts = W.split_tensors(flat, wl.numel)
        host.append([W.as_numpy(t) for t in ts])
        row = []
        for t in ts:
            if misalign:
                buf = torch.empty(t.numel() + misalign, dtype=t.dtype, device="cuda")
                view = buf[misalign:]
                view.copy_(t)
                row.append(view)
            else:
                row.append(t.cuda())
        dev.append(row)
    return host, dev


def shares_of(wl, kt=None):
    if wl.shares is not None:
        return list(wl.shares)
    return kt.kt_schedule(wl.step_times, wl.global_batch)


def run_gpu_path(kt, wl, dev_grads, shares, out_dtype=None, R=1, scale=1.0, per_bucket=False,
                 use_combined=False, staged=False, relay_chunk=4 << 20, rows=False, transport_dtype=torch.float32,
                 skew16=False):
    """Returns (out[c][t] tensors, transport list, plan, ctx).  skew16: every transport, pinned
    and receive buffer starts 16 bytes past a 32-byte boundary (the least alignment the library
    accepts), so that 8-float accesses cannot be single 256-bit instructions."""
    ctx = kt.kt_groups_init(wl.group_of, shares, wl.G)
    if transport_dtype != torch.float32:
        kt.kt_set_transport_dtype(ctx, kt.KT_BF16)
    kt.kt_bucket_pack(ctx, dev_grads, wl.bucket_cap_bytes)
    plan = kt.kt_plan_query(ctx)
    n = plan.transport_numel
    # rows=True: the G buffers of each set are rows of one allocation (the relay then moves a
    # chunk of all groups in one copy)
    def buffers(pinned=False):
        tdt = transport_dtype
        if skew16:
            shift = 16 // torch.empty(0, dtype=tdt).element_size()
            out = []
            for _ in range(wl.G):
                whole = torch.full((n + 64,), float("nan"), dtype=tdt, device=None if pinned else "cuda")
                whole = whole.pin_memory() if pinned else whole
                assert whole.data_ptr() % 32 == 0
                out.append(whole[shift:shift + n])
            return out
        if rows:
            whole = torch.full((wl.G, n), float("nan"), dtype=tdt, device=None if pinned else "cuda")
            return list(whole.pin_memory() if pinned else whole)
        return [torch.full((n,), float("nan"), dtype=tdt).pin_memory() if pinned
                else torch.full((n,), float("nan"), dtype=tdt, device="cuda") for _ in range(wl.G)]
    transport = buffers()
    odt = TORCH_DT[wl.dtype] if out_dtype is None else out_dtype
    out = [[torch.full((m,), float("nan"), dtype=odt, device="cuda") for m in wl.numel] for _ in range(R)]
    buckets = list(range(plan.n_buckets)) if per_bucket else [-1]
    src = transport
    if staged:
        host = buffers(pinned=True)
        recv = buffers()
        side = torch.cuda.Stream()
        src = recv
    if staged in ("relay", "relay_all"):
        # the benchmark's launch configuration: one fused-reduce launch over all buckets, the
        # relay bucket by bucket as a chunk pipeline on two copy streams, one combine/unpack launch
        side2 = torch.cuda.Stream()
        kt.kt_hier_reduce(ctx, kt.KT_INTRA, transport, bucket=-1)
        relay_buckets = [-1] if staged == "relay_all" else list(range(plan.n_buckets))
        for b in relay_buckets:
            kt.kt_relay_through_host(ctx, transport, host, recv, side, side2, bucket=b, chunk_bytes=relay_chunk)
        for b in relay_buckets:
            kt.kt_stage_wait(ctx, kt.KT_H2D, bucket=b)
        kt.kt_unpack_scale(ctx, recv, out, scale=scale, bucket=-1)
        torch.cuda.synchronize()
        for g in range(wl.G):      # what crossed the host is what the reduce wrote
            assert torch.equal(host[g], transport[g].cpu()) and torch.equal(recv[g], transport[g])
        return out, transport, plan, ctx
    for b in buckets:
        kt.kt_hier_reduce(ctx, kt.KT_INTRA, transport, bucket=b)
        if staged:
            kt.kt_stage_to_host(ctx, kt.KT_D2H, transport, host, bucket=b, side_stream=side)
            kt.kt_stage_to_host(ctx, kt.KT_H2D, recv, host, bucket=b, side_stream=side)
    for b in buckets:
        if staged:
            kt.kt_stage_wait(ctx, kt.KT_H2D, bucket=b)
        if use_combined:
            combined = torch.full((n,), float("nan"), device="cuda")
            kt.kt_hier_reduce(ctx, kt.KT_INTER, src, combined, bucket=b)
            kt.kt_unpack_scale(ctx, [combined], out, scale=scale, from_combined=True, bucket=b)
        else:
            kt.kt_unpack_scale(ctx, src, out, scale=scale, bucket=b)
    torch.cuda.synchronize()
    return out, transport, plan, ctx


def run_oracle_path(oracle, wl, host_grads, shares, out_dtype=None, scale=1.0, transport_dtype=0):
    odt = ORACLE_DT[wl.dtype] if out_dtype is None else out_dtype
    return oracle.sync_step(host_grads, wl.numel, ORACLE_DT[wl.dtype], wl.group_of, shares, wl.G,
                            wl.bucket_cap_bytes, scale, odt, transport_dtype)


def bits(a: np.ndarray) -> np.ndarray:
    return a.view(np.uint32) if a.dtype == np.float32 else a.view(np.uint16)


def assert_bit_equal(got: torch.Tensor, want: np.ndarray, what: str = ""):
    g = W.as_numpy(got)
    assert g.shape == want.shape, what
    gb, wb = bits(g), bits(want)
    if not np.array_equal(gb, wb):
        bad = np.nonzero(gb != wb)[0]
        raise AssertionError("%s: %d of %d elements differ, first at %d: got %r want %r"
                             % (what, bad.size, gb.size, bad[0], g[bad[0]], want[bad[0]]))
