"""Thin ctypes binding over the C-ABI library declared in ``include/kaitian.h``.

Argument marshalling only: every function here has the name of the C entry point it
calls, turns torch tensors into raw pointers and raises :class:`KtError` on a negative
status.  All arithmetic runs in the CUDA library.  If the library has not been built the
import fails: there is no CPU fallback.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import List, Optional, Sequence, Union

import torch

from . import build as _build

KT_F32, KT_BF16 = 0, 1
KT_INTRA, KT_INTER, KT_BOTH = 1, 2, 3
KT_D2H, KT_H2D = 0, 1
KT_ROUTE_DIRECT, KT_ROUTE_RELAY = 0, 1
KT_OK, KT_ERR_INVALID, KT_ERR_SHAPE, KT_ERR_ALIGN = 0, -1, -2, -3
KT_ERR_CUDA, KT_ERR_TIMEOUT, KT_ERR_STATE, KT_ERR_NOMEM = -4, -5, -6, -7
KT_MAX_RANKS, KT_MAX_GROUPS = 64, 16

EXPORTS = ["kt_schedule", "kt_scores", "kt_adapt_create", "kt_adapt_observe", "kt_adapt_state", "kt_adapt_destroy",
           "kt_sampler_steps", "kt_sampler_indices", "kt_graph_begin", "kt_graph_end", "kt_graph_launch",
           "kt_graph_nodes", "kt_graph_destroy", "kt_groups_init", "kt_set_shares", "kt_set_coefficients",
           "kt_get_coefficients", "kt_set_transport_dtype", "kt_route", "kt_bucket_pack", "kt_plan_buckets", "kt_plan_query", "kt_hier_reduce",
           "kt_stage_to_host", "kt_relay_through_host", "kt_stage_wait", "kt_unpack_scale", "kt_sync_direct", "kt_allreduce", "kt_bcast_send", "kt_bcast_relay", "kt_bcast_recv", "kt_cast", "kt_copy_tensors", "kt_sync_flat_static", "kt_launch_count",
           "kt_last_error", "kt_destroy", "kt_work_unit", "kt_shard_ranges", "kt_shard_bind", "kt_shard_query",
           "kt_ipc_export", "kt_ipc_open", "kt_ipc_close", "kt_host_register", "kt_host_unregister", "kt_host_barrier", "kt_shard_step", "kt_shard_bcast"]

_DTYPES = {torch.float32: KT_F32, torch.bfloat16: KT_BF16}


class KtError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__("kaitian status %d: %s" % (status, message))
        self.status = status


def _load() -> C.CDLL:
    path = _build.LIB
    if not os.path.exists(path):
        raise ImportError(
            "%s is missing: build it with `python -m paper_2505_10183_b200.build` "
            "(needs nvcc); this package has no CPU fallback" % path)
    L = C.CDLL(path)
    vp, i32p, i64p, f32p = C.c_void_p, C.POINTER(C.c_int32), C.POINTER(C.c_int64), C.POINTER(C.c_float)
    vpp = C.POINTER(C.c_void_p)
    sigs = {
        "kt_schedule": ([C.POINTER(C.c_double), C.c_int, C.c_int, i32p], C.c_int),
        "kt_scores": ([C.POINTER(C.c_double), C.c_int, C.POINTER(C.c_double)], C.c_int),
        "kt_adapt_create": ([i32p, C.c_int, C.c_int, C.c_double, C.c_int, C.c_double, vpp], C.c_int),
        "kt_adapt_observe": ([vp, C.POINTER(C.c_double), i32p, C.POINTER(C.c_int)], C.c_int),
        "kt_adapt_state": ([vp, C.POINTER(C.c_double), i32p, i64p], C.c_int),
        "kt_adapt_destroy": ([vp], None),
        "kt_sampler_steps": ([C.c_int64, C.c_int64, C.c_int], C.c_int64),
        "kt_sampler_indices": ([vp, C.c_int64, i32p, C.c_int, C.c_int, vpp, vp], C.c_int),
        "kt_graph_begin": ([vp, vp], C.c_int),
        "kt_graph_end": ([vp, vp, vpp], C.c_int),
        "kt_graph_launch": ([vp, vp], C.c_int),
        "kt_graph_nodes": ([vp], C.c_int64),
        "kt_graph_destroy": ([vp], None),
        "kt_groups_init": ([i32p, i32p, C.c_int, C.c_int, vpp], C.c_int),
        "kt_set_shares": ([vp, i32p], C.c_int),
        "kt_set_coefficients": ([vp, f32p, f32p], C.c_int),
        "kt_get_coefficients": ([vp, f32p, f32p], C.c_int),
        "kt_set_transport_dtype": ([vp, C.c_int], C.c_int),
        "kt_route": ([i32p, C.c_int, C.c_int, i32p, C.c_int, C.POINTER(C.c_int), i32p, C.POINTER(C.c_int)], C.c_int),
        "kt_bucket_pack": ([vp, vpp, i64p, C.c_int, C.c_int, C.c_int64, vpp, vp], C.c_int),
        "kt_plan_buckets": ([i64p, C.c_int, C.c_int64, i32p, i64p, i64p, i64p, i32p, i64p], C.c_int),
        "kt_plan_query": ([vp, i32p, i64p, i64p, i64p, i32p, i64p], C.c_int),
        "kt_hier_reduce": ([vp, C.c_int, C.c_int, vpp, vp, vp], C.c_int),
        "kt_stage_to_host": ([vp, C.c_int, C.c_int, vpp, vpp, vp, vp], C.c_int),
        "kt_relay_through_host": ([vp, C.c_int, vpp, vpp, vpp, C.c_int64, vp, vp, vp], C.c_int),
        "kt_stage_wait": ([vp, C.c_int, C.c_int, vp, C.c_int], C.c_int),
        "kt_unpack_scale": ([vp, vpp, C.c_int, vpp, C.c_int, C.c_int, C.c_float, C.c_int, vp], C.c_int),
        "kt_sync_direct": ([vp, vpp, C.c_int, C.c_int, C.c_float, C.c_int, vp], C.c_int),
        "kt_allreduce": ([vp, vpp, vpp, vpp, vpp, C.c_int, C.c_int, C.c_float, C.c_int64, vp, vp, vp], C.c_int),
        "kt_bcast_send": ([vp, C.c_int, C.c_int, vp, vp], C.c_int),
        "kt_bcast_relay": ([vp, C.c_int, C.c_int, vp, vp, vpp, C.c_int64, vp, vp, vp], C.c_int),
        "kt_bcast_recv": ([vp, C.c_int, C.c_int, vpp, vp], C.c_int),
        "kt_cast": ([vp, C.c_int, vp, C.c_int, C.c_int64, vp], C.c_int),
        "kt_copy_tensors": ([vpp, vpp, i64p, C.c_int, C.c_int, vp], C.c_int),
        "kt_sync_flat_static": ([i32p, i32p, C.c_int, C.c_int, vpp, C.c_int, C.c_int64, vp, C.c_int,
                                 C.c_float, vp], C.c_int),
        "kt_work_unit": ([C.c_int], C.c_int),
        "kt_shard_ranges": ([i64p, C.c_int, C.c_int64, C.c_int64, C.c_int, C.c_int, i64p, i64p], C.c_int),
        "kt_shard_bind": ([vp, C.c_int], C.c_int),
        "kt_shard_query": ([vp, C.c_int, C.c_int, C.POINTER(C.c_int), i64p, i64p], C.c_int),
        "kt_ipc_export": ([vp, vp, i64p], C.c_int),
        "kt_ipc_open": ([vp, C.c_int64, vpp], C.c_int),
        "kt_ipc_close": ([vp], C.c_int),
        "kt_host_register": ([vp, C.c_int64], C.c_int),
        "kt_host_unregister": ([vp], C.c_int),
        "kt_host_barrier": ([vp, C.c_int, C.c_int], C.c_int),
        "kt_shard_step": ([vp, vp, vpp, vpp, vpp, C.c_int, C.c_int, C.c_float, C.c_int, vp, vp, vp, C.c_int], C.c_int),
        "kt_shard_bcast": ([vp, C.c_int, vp, vp, vp, vp, C.c_int, vp, vp, vp, C.c_int], C.c_int),
        "kt_launch_count": ([vp], C.c_int64),
        "kt_last_error": ([vp], C.c_char_p),
        "kt_destroy": ([vp], None),
    }
    for name, (args, res) in sigs.items():
        fn = getattr(L, name)
        fn.argtypes = args
        fn.restype = res
    return L


_lib = _load()


def _check(rc: int) -> None:
    if rc != 0:
        raise KtError(rc, _lib.kt_last_error(None).decode("utf-8", "replace"))


class PtrArray:
    """A host array of raw pointers built once from tensors (keeps them alive)."""

    def __init__(self, tensors: Sequence[torch.Tensor]):
        self.tensors = list(tensors)
        self.n = len(self.tensors)
        self.array = (C.c_void_p * max(self.n, 1))()
        for i, t in enumerate(self.tensors):
            self.array[i] = t.data_ptr() if t.numel() > 0 else (t.data_ptr() or None)


    @classmethod
    def from_addresses(cls, addresses: Sequence[int], keep=None) -> "PtrArray":
        """A pointer array from raw addresses (e.g. offsets into tensors held elsewhere);
        `keep` is stored so that whatever owns the memory stays alive with the array."""
        self = cls([])
        self.tensors = keep
        self.n = len(addresses)
        self.array = (C.c_void_p * max(self.n, 1))(*[int(a) if a else None for a in addresses])
        return self


Ptrs = Union[PtrArray, Sequence[torch.Tensor]]


def kt_ptrs(tensors: Ptrs) -> PtrArray:
    return tensors if isinstance(tensors, PtrArray) else PtrArray(tensors)


def _stream(stream) -> C.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


def _i32(values) -> C.Array:
    return (C.c_int32 * len(values))(*[int(v) for v in values])


@dataclass
class Plan:
    n_buckets: int
    bucket_start: List[int]
    bucket_numel: List[int]
    tensor_offset: List[int]
    bucket_of: List[int]
    transport_numel: int


class Ctx:
    """Opaque handle returned by :func:`kt_groups_init`."""

    def __init__(self, handle: int, K: int, G: int):
        self.handle = C.c_void_p(handle)
        self.K, self.G, self.T = K, G, 0
        self.sources = K              # rank lists kt_bucket_pack expects (the group's members once bound to a rank)
        self._keep = {}

    def __del__(self):
        try:
            kt_destroy(self)
        except Exception:
            pass


# --------------------------------------------------------------------------- entry points
def kt_schedule(step_times: Sequence[float], global_batch: int) -> List[int]:
    K = len(step_times)
    t = (C.c_double * max(K, 1))(*[float(x) for x in step_times])
    out = (C.c_int32 * max(K, 1))()
    _check(_lib.kt_schedule(t, K, int(global_batch), out))
    return [int(out[i]) for i in range(K)]


class Adapt:
    """Handle of the online adaptation state (kt_adapt_create)."""

    def __init__(self, handle: int, K: int):
        self.handle = C.c_void_p(handle)
        self.K = K

    def __del__(self):
        try:
            kt_adapt_destroy(self)
        except Exception:
            pass


def kt_adapt_create(shares: Sequence[int], global_batch: int, alpha: float, period: int, hysteresis: float) -> Adapt:
    h = C.c_void_p()
    _check(_lib.kt_adapt_create(_i32(shares), len(shares), int(global_batch), float(alpha), int(period),
                                float(hysteresis), C.byref(h)))
    return Adapt(h.value, len(shares))


def kt_adapt_observe(state: Adapt, step_times: Sequence[float]):
    """Returns (shares to use from now on, whether they changed)."""
    if len(step_times) != state.K:
        raise KtError(KT_ERR_SHAPE, "expected %d step times" % state.K)
    t = (C.c_double * state.K)(*[float(x) for x in step_times])
    out = (C.c_int32 * state.K)()
    changed = C.c_int(0)
    _check(_lib.kt_adapt_observe(state.handle, t, out, C.byref(changed)))
    return [int(v) for v in out], bool(changed.value)


def kt_adapt_state(state: Adapt):
    """Returns (smoothed per-sample times, shares in use, number of observations)."""
    tau = (C.c_double * state.K)()
    b = (C.c_int32 * state.K)()
    n = C.c_int64(0)
    _check(_lib.kt_adapt_state(state.handle, tau, b, C.byref(n)))
    return [float(v) for v in tau], [int(v) for v in b], int(n.value)


def kt_adapt_destroy(state: Adapt) -> None:
    if state.handle is not None and state.handle.value:
        _lib.kt_adapt_destroy(state.handle)
        state.handle = C.c_void_p(None)


def kt_sampler_steps(dataset_size: int, global_batch: int, drop_last: bool) -> int:
    s = int(_lib.kt_sampler_steps(int(dataset_size), int(global_batch), int(bool(drop_last))))
    _check(s if s < 0 else 0)
    return s


def kt_sampler_indices(index_list: Optional[torch.Tensor], dataset_size: int, shares: Sequence[int],
                       out: Sequence[torch.Tensor], drop_last: bool = False, stream=None) -> None:
    """index_list: int64 device tensor of dataset_size entries (the epoch's permutation) or None;
    out[r]: int64 device tensor of kt_sampler_steps(...) * shares[r] entries."""
    K = len(shares)
    if len(out) != K:
        raise KtError(KT_ERR_SHAPE, "expected %d output tensors" % K)
    if any(t.dtype != torch.int64 or not t.is_contiguous() for t in out):
        raise KtError(KT_ERR_SHAPE, "out: int64 contiguous tensors expected")
    if index_list is not None and (index_list.dtype != torch.int64 or index_list.numel() != dataset_size
                                   or not index_list.is_contiguous()):
        raise KtError(KT_ERR_SHAPE, "index_list: int64 contiguous tensor of dataset_size entries expected")
    if K >= 1 and all(int(b) >= 1 for b in shares) and dataset_size >= 1:
        steps = kt_sampler_steps(dataset_size, sum(int(b) for b in shares), drop_last)
        if any(t.numel() != steps * int(b) for t, b in zip(out, shares)):
            raise KtError(KT_ERR_SHAPE, "out[r] must hold steps * shares[r] = %d * shares[r] entries" % steps)
    pa = PtrArray(out)
    _check(_lib.kt_sampler_indices(C.c_void_p(index_list.data_ptr()) if index_list is not None else None,
                                   int(dataset_size), _i32(shares), K, int(bool(drop_last)), pa.array,
                                   _stream(stream)))


def kt_scores(step_times: Sequence[float]) -> List[float]:
    K = len(step_times)
    t = (C.c_double * max(K, 1))(*[float(x) for x in step_times])
    out = (C.c_double * max(K, 1))()
    _check(_lib.kt_scores(t, K, out))
    return [float(out[i]) for i in range(K)]


def kt_groups_init(group_of: Sequence[int], shares: Sequence[int], G: Optional[int] = None) -> Ctx:
    K = len(group_of)
    if len(shares) != K:
        raise KtError(KT_ERR_SHAPE, "group_of and shares differ in length")
    G = (max(group_of) + 1 if K else 0) if G is None else G
    h = C.c_void_p()
    _check(_lib.kt_groups_init(_i32(group_of), _i32(shares), K, int(G), C.byref(h)))
    return Ctx(h.value, K, int(G))


def kt_set_shares(ctx: Ctx, shares: Sequence[int]) -> None:
    if len(shares) != ctx.K:
        raise KtError(KT_ERR_SHAPE, "expected %d shares" % ctx.K)
    _check(_lib.kt_set_shares(ctx.handle, _i32(shares)))


def kt_set_coefficients(ctx: Ctx, a: Sequence[float], W: Sequence[float]) -> None:
    if len(a) != ctx.K or len(W) != ctx.G:
        raise KtError(KT_ERR_SHAPE, "expected %d rank and %d group weights" % (ctx.K, ctx.G))
    _check(_lib.kt_set_coefficients(ctx.handle, (C.c_float * ctx.K)(*a), (C.c_float * ctx.G)(*W)))


def kt_set_transport_dtype(ctx: Ctx, dtype: int) -> None:
    """KT_F32 (default) or KT_BF16: element type of the transport / pinned / receive buffers."""
    _check(_lib.kt_set_transport_dtype(ctx.handle, int(dtype)))


def kt_route(group_of: Sequence[int], participants: Sequence[int], G: Optional[int] = None):
    """Returns (KT_ROUTE_DIRECT or KT_ROUTE_RELAY, ascending list of the groups that take part)."""
    K = len(group_of)
    G = (max(group_of) + 1 if K else 0) if G is None else G
    route, ng = C.c_int(-1), C.c_int(0)
    groups = (C.c_int32 * max(G, 1))()
    _check(_lib.kt_route(_i32(group_of) if K else None, K, int(G), _i32(participants) if participants else None,
                         len(participants), C.byref(route), groups, C.byref(ng)))
    return int(route.value), [int(groups[i]) for i in range(ng.value)]


def kt_get_coefficients(ctx: Ctx):
    a = (C.c_float * ctx.K)()
    W = (C.c_float * ctx.G)()
    _check(_lib.kt_get_coefficients(ctx.handle, a, W))
    return list(a), list(W)


def kt_bucket_pack(ctx: Ctx, grads: Sequence[Sequence[torch.Tensor]], bucket_cap_bytes: int,
                   flat_out: Optional[Ptrs] = None, stream=None) -> None:
    """grads[r][t]: tensor t of rank r (contiguous, all of one dtype, same shapes per rank)."""
    if len(grads) != ctx.sources:
        raise KtError(KT_ERR_SHAPE, "expected gradient lists of %d ranks" % ctx.sources)
    T = len(grads[0])
    flat = []
    for r in range(ctx.sources):
        if len(grads[r]) != T:
            raise KtError(KT_ERR_SHAPE, "rank %d holds %d tensors, rank 0 holds %d" % (r, len(grads[r]), T))
        for t in range(T):
            g = grads[r][t]
            if g.dtype != grads[0][0].dtype or g.numel() != grads[0][t].numel() or not g.is_contiguous():
                raise KtError(KT_ERR_SHAPE, "grads[%d][%d]: dtype, size or layout mismatch" % (r, t))
            flat.append(g)
    if T and grads[0][0].dtype not in _DTYPES:
        raise KtError(KT_ERR_INVALID, "unsupported gradient dtype %s" % grads[0][0].dtype)
    pa = PtrArray(flat)
    numel = (C.c_int64 * max(T, 1))(*[int(g.numel()) for g in grads[0]])
    fo = kt_ptrs(flat_out) if flat_out is not None else None
    dt = _DTYPES[grads[0][0].dtype] if T else KT_F32
    _check(_lib.kt_bucket_pack(ctx.handle, pa.array, numel, T, dt, int(bucket_cap_bytes),
                               fo.array if fo is not None else None, _stream(stream)))
    ctx.T = T
    ctx._keep["grads"] = pa


def kt_bucket_pack_ptrs(ctx: Ctx, grads: PtrArray, numel: Sequence[int], dtype: int, bucket_cap_bytes: int,
                        stream=None) -> None:
    """kt_bucket_pack from raw device addresses (grads: rank-major, ctx.sources * len(numel)
    pointers), for tensors that are not torch tensors of this process: memory of other
    processes mapped with kt_ipc_open."""
    T = len(numel)
    if grads.n != ctx.sources * T:
        raise KtError(KT_ERR_SHAPE, "expected %d gradient pointers" % (ctx.sources * T))
    n = (C.c_int64 * max(T, 1))(*[int(v) for v in numel])
    _check(_lib.kt_bucket_pack(ctx.handle, grads.array, n, T, int(dtype), int(bucket_cap_bytes), None, _stream(stream)))
    ctx.T = T
    ctx._keep["grads"] = grads


def kt_work_unit(dtype: int) -> int:
    u = int(_lib.kt_work_unit(int(dtype)))
    _check(u if u < 0 else 0)
    return u


def kt_shard_ranges(numel: Sequence[int], bucket_cap_bytes: int, unit: int, bucket: int, n_members: int):
    """Pure host: [(lo, n)] per member, the element range of the transport each of the
    n_members devices of a group works on."""
    T = len(numel)
    n = (C.c_int64 * max(T, 1))(*[int(v) for v in numel])
    lo = (C.c_int64 * max(n_members, 1))()
    cnt = (C.c_int64 * max(n_members, 1))()
    _check(_lib.kt_shard_ranges(n, T, int(bucket_cap_bytes), int(unit), int(bucket), int(n_members), lo, cnt))
    return [(int(lo[m]), int(cnt[m])) for m in range(n_members)]


def kt_shard_bind(ctx: Ctx, rank: int, group_of: Sequence[int]) -> None:
    """Binds the context to one rank (one rank per device); group_of is the map given to
    kt_groups_init, used here only to know how many rank lists kt_bucket_pack will expect."""
    _check(_lib.kt_shard_bind(ctx.handle, int(rank)))
    ctx.sources = sum(1 for g in group_of if g == group_of[rank])


def kt_shard_query(ctx: Ctx, bucket: int = -1, member: int = -1):
    """Returns (lo, n, members): this context's (or `member`'s) element range for `bucket`."""
    M, lo, n = C.c_int(0), C.c_int64(0), C.c_int64(0)
    _check(_lib.kt_shard_query(ctx.handle, int(bucket), int(member), C.byref(M), C.byref(lo), C.byref(n)))
    return int(lo.value), int(n.value), int(M.value)


KT_IPC_HANDLE_BYTES = 64


def kt_ipc_export(address: int):
    """Returns (handle bytes, offset) for a device address inside a cudaMalloc allocation."""
    h = (C.c_ubyte * KT_IPC_HANDLE_BYTES)()
    off = C.c_int64(0)
    _check(_lib.kt_ipc_export(C.c_void_p(int(address)), h, C.byref(off)))
    return bytes(h), int(off.value)


def kt_ipc_open(handle: bytes, offset: int) -> int:
    """Maps another process's allocation on the current device; returns the address."""
    out = C.c_void_p()
    buf = (C.c_ubyte * KT_IPC_HANDLE_BYTES).from_buffer_copy(handle)
    _check(_lib.kt_ipc_open(buf, int(offset), C.byref(out)))
    return int(out.value)


def kt_ipc_close(handle: bytes) -> None:
    buf = (C.c_ubyte * KT_IPC_HANDLE_BYTES).from_buffer_copy(handle)
    _check(_lib.kt_ipc_close(buf))


def kt_host_register(address: int, nbytes: int) -> None:
    _check(_lib.kt_host_register(C.c_void_p(int(address)), int(nbytes)))


def kt_host_unregister(address: int) -> None:
    _check(_lib.kt_host_unregister(C.c_void_p(int(address))))


KT_HOST_BARRIER_BYTES = 128


def kt_host_barrier(address: int, n_ranks: int, timeout_ms: int = -1) -> None:
    """Barrier between the processes of a node on a zeroed, 64-byte aligned block of shared host
    memory; raises KtError(KT_ERR_TIMEOUT) when the others do not arrive in time."""
    _check(_lib.kt_host_barrier(C.c_void_p(int(address)), int(n_ranks), int(timeout_ms)))


def kt_shard_step(ctx: Ctx, barrier_address: int, partials: Optional[Ptrs], host_shared: Optional[Ptrs],
                  out_grads: PtrArray, R: int, out_dtype: int, scale: float = 1.0, per_bucket: bool = True,
                  main_stream=None, down_stream=None, up_stream=None, timeout_ms: int = -1) -> None:
    """One whole step of a rank-bound context; blocks until every rank has finished it."""
    pa = kt_ptrs(partials) if partials is not None else None
    hs = kt_ptrs(host_shared) if host_shared is not None else None
    if out_grads.n != R * ctx.T:
        raise KtError(KT_ERR_SHAPE, "expected %d output pointers" % (R * ctx.T))
    _check(_lib.kt_shard_step(ctx.handle, C.c_void_p(int(barrier_address)), pa.array if pa is not None else None,
                              hs.array if hs is not None else None, out_grads.array, int(R), int(out_dtype),
                              C.c_float(scale), int(bool(per_bucket)), _stream(main_stream), _stream(down_stream),
                              _stream(up_stream), int(timeout_ms)))
    ctx._keep["out"] = out_grads


def kt_shard_bcast(ctx: Ctx, root: int, barrier_address: int, send_address: int, host_address: int,
                   recv_address: int, per_bucket: bool, main_stream, d2h_stream, h2d_stream,
                   timeout_ms: int = -1) -> None:
    """Broadcast of rank `root`'s registered tensors to every rank (rank-bound contexts); blocks
    until every rank has finished.  Addresses may be 0 where the header allows NULL."""
    _check(_lib.kt_shard_bcast(ctx.handle, int(root), C.c_void_p(int(barrier_address)),
                               C.c_void_p(int(send_address) or None), C.c_void_p(int(host_address) or None),
                               C.c_void_p(int(recv_address) or None), int(bool(per_bucket)), _stream(main_stream),
                               _stream(d2h_stream), _stream(h2d_stream), int(timeout_ms)))


def kt_plan_buckets(numel: Sequence[int], bucket_cap_bytes: int) -> Plan:
    T = len(numel)
    n = (C.c_int64 * max(T, 1))(*[int(v) for v in numel])
    nb = C.c_int32()
    total = C.c_int64()
    bs = (C.c_int64 * max(T, 1))()
    bn = (C.c_int64 * max(T, 1))()
    off = (C.c_int64 * max(T, 1))()
    bof = (C.c_int32 * max(T, 1))()
    _check(_lib.kt_plan_buckets(n, T, int(bucket_cap_bytes), C.byref(nb), bs, bn, off, bof, C.byref(total)))
    return Plan(nb.value, list(bs)[: nb.value], list(bn)[: nb.value], list(off)[:T], list(bof)[:T], total.value)


def kt_plan_query(ctx: Ctx) -> Plan:
    nb = C.c_int32()
    total = C.c_int64()
    _check(_lib.kt_plan_query(ctx.handle, C.byref(nb), None, None, None, None, C.byref(total)))
    bs = (C.c_int64 * nb.value)()
    bn = (C.c_int64 * nb.value)()
    off = (C.c_int64 * ctx.T)()
    bof = (C.c_int32 * ctx.T)()
    _check(_lib.kt_plan_query(ctx.handle, None, bs, bn, off, bof, None))
    return Plan(nb.value, list(bs), list(bn), list(off), list(bof), total.value)


def kt_hier_reduce(ctx: Ctx, phase: int, transport: Ptrs, combined: Optional[torch.Tensor] = None,
                   bucket: int = -1, stream=None) -> None:
    tr = kt_ptrs(transport)
    if tr.n != ctx.G:
        raise KtError(KT_ERR_SHAPE, "expected %d transport buffers" % ctx.G)
    _check(_lib.kt_hier_reduce(ctx.handle, int(phase), int(bucket), tr.array,
                               C.c_void_p(combined.data_ptr()) if combined is not None else None,
                               _stream(stream)))


def kt_stage_to_host(ctx: Ctx, direction: int, transport: Ptrs, host_pinned: Ptrs, bucket: int = -1,
                     main_stream=None, side_stream=None) -> None:
    tr, hp = kt_ptrs(transport), kt_ptrs(host_pinned)
    if tr.n != ctx.G or hp.n != ctx.G:
        raise KtError(KT_ERR_SHAPE, "expected %d device and %d host buffers" % (ctx.G, ctx.G))
    _check(_lib.kt_stage_to_host(ctx.handle, int(direction), int(bucket), tr.array, hp.array,
                                 _stream(main_stream), _stream(side_stream)))


def kt_relay_through_host(ctx: Ctx, send: Ptrs, host_pinned: Ptrs, recv: Ptrs, d2h_stream, h2d_stream,
                          bucket: int = -1, chunk_bytes: int = 4 << 20, main_stream=None) -> None:
    sd, hp, rv = kt_ptrs(send), kt_ptrs(host_pinned), kt_ptrs(recv)
    if sd.n != ctx.G or hp.n != ctx.G or rv.n != ctx.G:
        raise KtError(KT_ERR_SHAPE, "expected %d buffers in every list" % ctx.G)
    _check(_lib.kt_relay_through_host(ctx.handle, int(bucket), sd.array, hp.array, rv.array, int(chunk_bytes),
                                      _stream(main_stream), _stream(d2h_stream), _stream(h2d_stream)))


def kt_stage_wait(ctx: Ctx, direction: int, bucket: int = -1, main_stream=None, timeout_ms: int = -1) -> None:
    _check(_lib.kt_stage_wait(ctx.handle, int(direction), int(bucket), _stream(main_stream), int(timeout_ms)))


def _out_args(ctx: Ctx, out_grads, out_dtype, R):
    """Marshals out_grads[c][t] (or a ready PtrArray) into (PtrArray, R, out_dtype)."""
    if isinstance(out_grads, PtrArray):
        op = out_grads
        if R is None or out_dtype is None:
            raise KtError(KT_ERR_INVALID, "R and out_dtype are required with a PtrArray")
    else:
        R = len(out_grads)
        flat = [t for copy in out_grads for t in copy]
        if any(len(copy) != ctx.T for copy in out_grads):
            raise KtError(KT_ERR_SHAPE, "every copy needs %d tensors" % ctx.T)
        if any(t.dtype != flat[0].dtype or not t.is_contiguous() for t in flat):
            raise KtError(KT_ERR_SHAPE, "out_grads: dtype or layout mismatch")
        if flat and flat[0].dtype not in _DTYPES:
            raise KtError(KT_ERR_INVALID, "unsupported output dtype %s" % flat[0].dtype)
        out_dtype = _DTYPES[flat[0].dtype] if flat else KT_F32
        op = PtrArray(flat)
    if op.n != R * ctx.T:
        raise KtError(KT_ERR_SHAPE, "expected %d output pointers" % (R * ctx.T))
    return op, int(R), int(out_dtype)


def kt_unpack_scale(ctx: Ctx, src: Ptrs, out_grads: Union[PtrArray, Sequence[Sequence[torch.Tensor]]],
                    scale: float = 1.0, from_combined: bool = False, bucket: int = -1,
                    out_dtype: Optional[int] = None, R: Optional[int] = None, stream=None) -> None:
    """out_grads[c][t]: copy c of tensor t (or a PtrArray of R*T pointers with R, out_dtype given)."""
    sp = kt_ptrs(src)
    if sp.n != (1 if from_combined else ctx.G):
        raise KtError(KT_ERR_SHAPE, "wrong number of source buffers")
    op, R, out_dtype = _out_args(ctx, out_grads, out_dtype, R)
    _check(_lib.kt_unpack_scale(ctx.handle, sp.array, 1 if from_combined else 0, op.array, R,
                                out_dtype, C.c_float(scale), int(bucket), _stream(stream)))
    ctx._keep["out"] = op


def kt_sync_direct(ctx: Ctx, out_grads: Union[PtrArray, Sequence[Sequence[torch.Tensor]]],
                   scale: float = 1.0, bucket: int = -1, out_dtype: Optional[int] = None,
                   R: Optional[int] = None, stream=None) -> None:
    """The one-pass route without transport buffers; out_grads as in kt_unpack_scale."""
    op, R, out_dtype = _out_args(ctx, out_grads, out_dtype, R)
    _check(_lib.kt_sync_direct(ctx.handle, op.array, R, out_dtype, C.c_float(scale), int(bucket),
                               _stream(stream)))
    ctx._keep["out"] = op


def kt_allreduce(ctx: Ctx, out_grads, transport: Optional[Ptrs] = None, host_pinned: Optional[Ptrs] = None,
                 recv: Optional[Ptrs] = None, d2h_stream=None, h2d_stream=None, scale: float = 1.0,
                 chunk_bytes: int = 4 << 20, out_dtype: Optional[int] = None, R: Optional[int] = None,
                 main_stream=None) -> None:
    """One AllReduce of the registered gradients: the direct route with one group, else reduce,
    relay through pinned host memory, combine + unpack.  The three buffer lists and the two copy
    streams are needed only with more than one group."""
    op, R, out_dtype = _out_args(ctx, out_grads, out_dtype, R)
    lists = [kt_ptrs(x) if x is not None else None for x in (transport, host_pinned, recv)]
    if ctx.G > 1 and (any(x is None or x.n != ctx.G for x in lists) or d2h_stream is None or h2d_stream is None):
        raise KtError(KT_ERR_SHAPE, "with %d groups, %d transport, pinned and receive buffers and two copy streams "
                                    "are required" % (ctx.G, ctx.G))
    arrs = [x.array if x is not None else None for x in lists]
    _check(_lib.kt_allreduce(ctx.handle, arrs[0], arrs[1], arrs[2], op.array, R, out_dtype, C.c_float(scale),
                             int(chunk_bytes), _stream(main_stream),
                             _stream(d2h_stream) if d2h_stream is not None else None,
                             _stream(h2d_stream) if h2d_stream is not None else None))
    ctx._keep["out"] = op
    ctx._keep["allreduce"] = lists


def _recv_array(ctx: Ctx, recv: Sequence[Optional[torch.Tensor]]) -> C.Array:
    if len(recv) != ctx.G:
        raise KtError(KT_ERR_SHAPE, "expected %d receive buffers (the root group's may be None)" % ctx.G)
    arr = (C.c_void_p * max(ctx.G, 1))()
    for g, t in enumerate(recv):
        arr[g] = t.data_ptr() if t is not None else None
    return arr


def kt_bcast_send(ctx: Ctx, root: int, send: torch.Tensor, bucket: int = -1, stream=None) -> None:
    _check(_lib.kt_bcast_send(ctx.handle, int(root), int(bucket), C.c_void_p(send.data_ptr()), _stream(stream)))


def kt_bcast_relay(ctx: Ctx, root: int, send: Optional[torch.Tensor], host_pinned: torch.Tensor,
                   recv: Sequence[Optional[torch.Tensor]], d2h_stream, h2d_stream, bucket: int = -1,
                   chunk_bytes: int = 4 << 20, main_stream=None) -> None:
    """send may be None on a rank-bound context that is not the root's."""
    _check(_lib.kt_bcast_relay(ctx.handle, int(root), int(bucket),
                               C.c_void_p(send.data_ptr()) if send is not None else None,
                               C.c_void_p(host_pinned.data_ptr()), _recv_array(ctx, recv), int(chunk_bytes),
                               _stream(main_stream), _stream(d2h_stream), _stream(h2d_stream)))


def kt_bcast_recv(ctx: Ctx, root: int, recv: Sequence[Optional[torch.Tensor]], bucket: int = -1, stream=None) -> None:
    _check(_lib.kt_bcast_recv(ctx.handle, int(root), int(bucket), _recv_array(ctx, recv), _stream(stream)))


def kt_cast(inp: torch.Tensor, out: torch.Tensor, stream=None) -> None:
    if inp.numel() != out.numel() or inp.dtype not in _DTYPES or out.dtype not in _DTYPES:
        raise KtError(KT_ERR_SHAPE, "kt_cast: size or dtype mismatch")
    _check(_lib.kt_cast(C.c_void_p(inp.data_ptr()), _DTYPES[inp.dtype], C.c_void_p(out.data_ptr()),
                        _DTYPES[out.dtype], inp.numel(), _stream(stream)))


def kt_copy_tensors(dst: Ptrs, src: Ptrs, nbytes: Sequence[int], direction: int, stream=None) -> None:
    d, s = kt_ptrs(dst), kt_ptrs(src)
    if d.n != s.n or d.n != len(nbytes):
        raise KtError(KT_ERR_SHAPE, "kt_copy_tensors: list lengths differ")
    sizes = nbytes if isinstance(nbytes, C.Array) else (C.c_int64 * max(d.n, 1))(*[int(b) for b in nbytes])
    _check(_lib.kt_copy_tensors(d.array, s.array, sizes, d.n, int(direction), _stream(stream)))


KT_STATIC_MAX_ELEMS = 1 << 20


def kt_sync_flat_static(group_of: Sequence[int], shares: Sequence[int], grads: Sequence[torch.Tensor],
                        out: torch.Tensor, scale: float = 1.0, G: Optional[int] = None, stream=None) -> None:
    """The flat path for callers that may not allocate device memory: one gradient buffer per
    rank in, one reduced buffer out, scratch in the library's fixed device array.  Marshals
    pointers only (no tensor is created here); see the header for limits and sharing rules."""
    K = len(group_of)
    if len(shares) != K or len(grads) != K:
        raise KtError(KT_ERR_SHAPE, "group_of, shares and grads differ in length")
    G = (max(group_of) + 1 if K else 0) if G is None else G
    n = out.numel()
    if any(g.numel() != n or g.dtype != grads[0].dtype or not g.is_contiguous() for g in grads):
        raise KtError(KT_ERR_SHAPE, "grads: size, dtype or layout mismatch")
    if grads[0].dtype not in _DTYPES or out.dtype not in _DTYPES or not out.is_contiguous():
        raise KtError(KT_ERR_INVALID, "unsupported dtype or layout")
    ptrs = (C.c_void_p * max(K, 1))(*[g.data_ptr() for g in grads])
    _check(_lib.kt_sync_flat_static(_i32(group_of), _i32(shares), K, int(G), ptrs, _DTYPES[grads[0].dtype],
                                    n, C.c_void_p(out.data_ptr()), _DTYPES[out.dtype], C.c_float(scale),
                                    _stream(stream)))


class Graph:
    """Handle of a recorded step (kt_graph_end)."""

    def __init__(self, handle: int):
        self.handle = C.c_void_p(handle)

    def __del__(self):
        try:
            kt_graph_destroy(self)
        except Exception:
            pass


def kt_graph_begin(ctx: Ctx, stream=None) -> None:
    _check(_lib.kt_graph_begin(ctx.handle, _stream(stream)))


def kt_graph_end(ctx: Ctx, stream=None) -> Graph:
    h = C.c_void_p()
    _check(_lib.kt_graph_end(ctx.handle, _stream(stream), C.byref(h)))
    return Graph(h.value)


def kt_graph_launch(graph: Graph, stream=None) -> None:
    _check(_lib.kt_graph_launch(graph.handle, _stream(stream)))


def kt_graph_nodes(graph: Graph) -> int:
    return int(_lib.kt_graph_nodes(graph.handle))


def kt_graph_destroy(graph: Graph) -> None:
    if graph.handle is not None and graph.handle.value:
        _lib.kt_graph_destroy(graph.handle)
        graph.handle = C.c_void_p(None)


def kt_launch_count(ctx: Ctx) -> int:
    return int(_lib.kt_launch_count(ctx.handle))


def kt_last_error() -> str:
    return _lib.kt_last_error(None).decode("utf-8", "replace")


def kt_destroy(ctx: Ctx) -> None:
    if ctx.handle is not None and ctx.handle.value:
        _lib.kt_destroy(ctx.handle)
        ctx.handle = C.c_void_p(None)
