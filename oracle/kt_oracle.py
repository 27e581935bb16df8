"""ctypes loader for the CPU oracle (``kt_oracle.c``).

TEST INFRASTRUCTURE ONLY: tests, the smoke check and the bench's CPU-baseline leg
use this module; the CUDA library never does, and this module never touches the
CUDA library.  It only marshals numpy arrays into the plain C functions; all of
the method's arithmetic is in ``kt_oracle.c``.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "kt_oracle.c")
_LIB = os.path.join(_HERE, "libkt_oracle.so")

F32, BF16 = 0, 1
_ELEM = {F32: 4, BF16: 2}
_NP = {F32: np.float32, BF16: np.uint16}


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fused contraction, no fast-math)."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(
            ["gcc", "-std=c99", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fPIC", "-shared",
             "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        i32p, i64p, f32p, f64p = (C.POINTER(C.c_int32), C.POINTER(C.c_int64),
                                  C.POINTER(C.c_float), C.POINTER(C.c_double))
        vpp = C.POINTER(C.c_void_p)
        L.kto_scores.argtypes = [f64p, C.c_int, f64p]
        L.kto_scores.restype = C.c_int
        L.kto_schedule.argtypes = [f64p, C.c_int, C.c_int, i32p]
        L.kto_schedule.restype = C.c_int
        L.kto_adapt_observe.argtypes = [f64p, i32p, i64p, C.c_int, C.c_int, C.c_double, C.c_int,
                                        C.c_double, f64p]
        L.kto_adapt_observe.restype = C.c_int
        L.kto_sampler_steps.argtypes = [C.c_int64, C.c_int64, C.c_int]
        L.kto_sampler_steps.restype = C.c_int64
        L.kto_sampler_indices.argtypes = [i64p, C.c_int64, i32p, C.c_int, C.c_int, vpp]
        L.kto_sampler_indices.restype = C.c_int
        L.kto_route.argtypes = [i32p, C.c_int, i32p, C.c_int]
        L.kto_route.restype = C.c_int
        L.kto_coefficients.argtypes = [i32p, i32p, C.c_int, C.c_int, f32p, f32p, f32p]
        L.kto_coefficients.restype = C.c_int
        L.kto_bucket_plan.argtypes = [i64p, C.c_int, C.c_int64, i64p, i32p, i64p, i64p, i32p, i64p]
        L.kto_bucket_plan.restype = C.c_int
        L.kto_shard_ranges.argtypes = [i64p, C.c_int, C.c_int64, C.c_int64, C.c_int, C.c_int, i64p, i64p]
        L.kto_shard_ranges.restype = C.c_int
        L.kto_bf16_to_f32.argtypes = [C.c_void_p, C.c_void_p, C.c_int64]
        L.kto_bf16_to_f32.restype = None
        L.kto_f32_to_bf16.argtypes = [C.c_void_p, C.c_void_p, C.c_int64]
        L.kto_f32_to_bf16.restype = None
        L.kto_pack.argtypes = [vpp, i64p, i64p, C.c_int, C.c_int, C.c_int64, C.c_void_p]
        L.kto_pack.restype = None
        L.kto_unpack_copy.argtypes = [C.c_void_p, i64p, i64p, C.c_int, C.c_int, vpp]
        L.kto_unpack_copy.restype = None
        L.kto_intra_reduce.argtypes = [vpp, C.c_int, i64p, i64p, C.c_int, C.c_int64, i32p, f32p,
                                       C.c_int, C.c_int, vpp]
        L.kto_intra_reduce.restype = None
        L.kto_combine.argtypes = [vpp, f32p, C.c_int, C.c_int64, C.c_void_p]
        L.kto_combine.restype = None
        L.kto_unpack_scale.argtypes = [C.c_void_p, i64p, i64p, C.c_int, C.c_float, C.c_int, vpp]
        L.kto_unpack_scale.restype = None
        L.kto_flat_reduce_f32.argtypes = [vpp, C.c_int, f32p, C.c_int, C.c_int64, C.c_void_p]
        L.kto_flat_reduce_f32.restype = None
        L.kto_flat_reduce_f64.argtypes = [vpp, C.c_int, i32p, C.c_int, C.c_int64, C.c_void_p,
                                          C.c_void_p]
        L.kto_flat_reduce_f64.restype = None
        _lib = L
    return _lib


class OracleError(ValueError):
    pass


def _p(arr, ctype):
    return arr.ctypes.data_as(C.POINTER(ctype))


def _ptr_array(arrays):
    out = (C.c_void_p * len(arrays))()
    for i, a in enumerate(arrays):
        assert a.flags["C_CONTIGUOUS"]
        out[i] = a.ctypes.data
    return out


def _check_dtype(arrays, dtype):
    for a in arrays:
        if a.dtype != _NP[dtype]:
            raise TypeError("expected %s array, got %s" % (_NP[dtype], a.dtype))


# --------------------------------------------------------------------------- schedule
def scores(step_times) -> np.ndarray:
    t = np.ascontiguousarray(step_times, dtype=np.float64)
    out = np.zeros(t.size, dtype=np.float64)
    if lib().kto_scores(_p(t, C.c_double), int(t.size), _p(out, C.c_double)) != 0:
        raise OracleError("kto_scores: invalid arguments")
    return out


def schedule(step_times, global_batch: int) -> np.ndarray:
    t = np.ascontiguousarray(step_times, dtype=np.float64)
    out = np.zeros(t.size, dtype=np.int32)
    rc = lib().kto_schedule(_p(t, C.c_double), int(t.size), int(global_batch), _p(out, C.c_int32))
    if rc != 0:
        raise OracleError("kto_schedule: invalid arguments")
    return out


class Adapter:
    """Caller-held state of the online adaptation: smoothed per-sample times, the shares in
    use and the number of observations so far."""

    def __init__(self, shares, global_batch: int, alpha: float, period: int, hysteresis: float):
        self.shares = np.ascontiguousarray(shares, dtype=np.int32).copy()
        self.ema = np.zeros(self.shares.size, np.float64)
        self.count = C.c_int64(0)
        self.B, self.alpha, self.period, self.hysteresis = int(global_batch), float(alpha), int(period), float(hysteresis)

    def observe(self, step_times) -> bool:
        t = np.ascontiguousarray(step_times, dtype=np.float64)
        if t.size != self.shares.size:
            raise OracleError("expected %d step times" % self.shares.size)
        rc = lib().kto_adapt_observe(_p(self.ema, C.c_double), _p(self.shares, C.c_int32), C.byref(self.count),
                                     int(t.size), self.B, self.alpha, self.period, self.hysteresis,
                                     _p(t, C.c_double))
        if rc < 0:
            raise OracleError("kto_adapt_observe: invalid arguments")
        return bool(rc)


def sampler_steps(dataset_size: int, global_batch: int, drop_last: bool) -> int:
    s = lib().kto_sampler_steps(int(dataset_size), int(global_batch), int(bool(drop_last)))
    if s < 0:
        raise OracleError("kto_sampler_steps: invalid arguments")
    return int(s)


def sampler_indices(index_list, dataset_size: int, shares, drop_last: bool):
    """Returns the list of K per-rank epoch index arrays (int64)."""
    b = np.ascontiguousarray(shares, dtype=np.int32)
    if b.size < 1 or (b < 1).any() or dataset_size < 1:
        raise OracleError("kto_sampler_indices: invalid arguments")
    S = sampler_steps(dataset_size, int(b.sum()), drop_last)
    out = [np.empty(S * int(v), np.int64) for v in b]
    lst = None
    if index_list is not None:
        lst = np.ascontiguousarray(index_list, dtype=np.int64)
        assert lst.size == dataset_size
    rc = lib().kto_sampler_indices(_p(lst, C.c_int64) if lst is not None else None, int(dataset_size),
                                   _p(b, C.c_int32), int(b.size), int(bool(drop_last)), _ptr_array(out))
    if rc != 0:
        raise OracleError("kto_sampler_indices: invalid arguments")
    return out


def route(group_of, participants) -> int:
    """0: all participants in one group (homogeneous), 1: they span groups (relay needed)."""
    g = np.ascontiguousarray(group_of, dtype=np.int32)
    p = np.ascontiguousarray(participants, dtype=np.int32)
    rc = lib().kto_route(_p(g, C.c_int32), int(g.size), _p(p, C.c_int32), int(p.size))
    if rc < 0:
        raise OracleError("kto_route: invalid arguments")
    return rc


def coefficients(group_of, shares, G: int):
    """Returns (a[K], W[G], w_flat[K]) as float32 arrays."""
    g = np.ascontiguousarray(group_of, dtype=np.int32)
    b = np.ascontiguousarray(shares, dtype=np.int32)
    K = g.size
    a = np.zeros(K, np.float32)
    W = np.zeros(G, np.float32)
    w = np.zeros(K, np.float32)
    rc = lib().kto_coefficients(_p(g, C.c_int32), _p(b, C.c_int32), K, int(G),
                                _p(a, C.c_float), _p(W, C.c_float), _p(w, C.c_float))
    if rc != 0:
        raise OracleError("kto_coefficients: invalid arguments")
    return a, W, w


# --------------------------------------------------------------------------- bucket plan
class Plan:
    """Result of the bucket plan: offsets are in transport (fp32) elements."""

    def __init__(self, numel, tensor_offset, bucket_of, bucket_start, bucket_numel, transport_numel):
        self.numel = numel
        self.tensor_offset = tensor_offset
        self.bucket_of = bucket_of
        self.bucket_start = bucket_start
        self.bucket_numel = bucket_numel
        self.transport_numel = int(transport_numel)
        self.n_buckets = int(bucket_start.size)
        self.T = int(numel.size)


def bucket_plan(numel, bucket_cap_bytes: int) -> Plan:
    n = np.ascontiguousarray(numel, dtype=np.int64)
    T = n.size
    off = np.zeros(T, np.int64)
    bof = np.zeros(T, np.int32)
    bstart = np.zeros(max(T, 1), np.int64)
    bnumel = np.zeros(max(T, 1), np.int64)
    nb = C.c_int32(0)
    total = C.c_int64(0)
    rc = lib().kto_bucket_plan(_p(n, C.c_int64), T, int(bucket_cap_bytes), _p(off, C.c_int64),
                               _p(bof, C.c_int32), _p(bstart, C.c_int64), _p(bnumel, C.c_int64),
                               C.byref(nb), C.byref(total))
    if rc != 0:
        raise OracleError("kto_bucket_plan: invalid arguments")
    return Plan(n, off, bof, bstart[: nb.value].copy(), bnumel[: nb.value].copy(), total.value)


def shard_ranges(numel, bucket_cap_bytes: int, unit: int, bucket: int, n_members: int):
    """One rank per device: the element range of the transport that each of the n_members
    devices of a group reduces, for one bucket (or the whole transport, bucket = -1).
    Returns a list of (lo, n), one per member."""
    n = np.ascontiguousarray(numel, dtype=np.int64)
    lo = np.zeros(max(n_members, 1), np.int64)
    cnt = np.zeros(max(n_members, 1), np.int64)
    rc = lib().kto_shard_ranges(_p(n, C.c_int64), n.size, int(bucket_cap_bytes), int(unit), int(bucket),
                                int(n_members), _p(lo, C.c_int64), _p(cnt, C.c_int64))
    if rc != 0:
        raise OracleError("kto_shard_ranges: invalid arguments")
    return [(int(a), int(b)) for a, b in zip(lo[:n_members], cnt[:n_members])]


# --------------------------------------------------------------------------- casts
def bf16_to_f32(x: np.ndarray) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.uint16)
    out = np.empty(x.shape, np.float32)
    lib().kto_bf16_to_f32(x.ctypes.data, out.ctypes.data, x.size)
    return out


def f32_to_bf16(x: np.ndarray) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float32)
    out = np.empty(x.shape, np.uint16)
    lib().kto_f32_to_bf16(x.ctypes.data, out.ctypes.data, x.size)
    return out


# --------------------------------------------------------------------------- data path
def pack(tensors, plan: Plan, dtype: int) -> np.ndarray:
    """tensors: list of T flat arrays of one rank.  Returns the flat bucket buffer."""
    _check_dtype(tensors, dtype)
    flat = np.empty(plan.transport_numel, _NP[dtype])
    lib().kto_pack(_ptr_array(tensors), _p(plan.numel, C.c_int64), _p(plan.tensor_offset, C.c_int64),
                   plan.T, _ELEM[dtype], plan.transport_numel, flat.ctypes.data)
    return flat


def unpack_copy(flat: np.ndarray, plan: Plan, dtype: int):
    """Bit copy of every tensor out of a flat buffer; returns the list of T flat arrays."""
    assert flat.dtype == _NP[dtype] and flat.size == plan.transport_numel
    out = [np.empty(int(n), _NP[dtype]) for n in plan.numel]
    lib().kto_unpack_copy(flat.ctypes.data, _p(plan.numel, C.c_int64), _p(plan.tensor_offset, C.c_int64),
                          plan.T, _ELEM[dtype], _ptr_array(out))
    return out


def broadcast(tensors, root: int, numel, dtype: int, bucket_cap_bytes: int):
    """Model synchronisation from rank `root`: tensors[r][t] are the ranks' lists.  Returns
    (new lists of every rank, the flat buffer that crosses the host, plan): the root keeps
    its own arrays, every other rank gets bit copies taken out of the flat buffer."""
    plan = bucket_plan(numel, bucket_cap_bytes)
    flat = pack(tensors[root], plan, dtype)
    out = [list(tensors[r]) if r == root else unpack_copy(flat, plan, dtype) for r in range(len(tensors))]
    return out, flat, plan


def intra_reduce(grads, plan: Plan, dtype: int, group_of, a, G: int):
    """grads[r][t]: flat arrays.  Returns the list of G fp32 transport partials."""
    K = len(grads)
    flat_list = [grads[r][t] for r in range(K) for t in range(plan.T)]
    _check_dtype(flat_list, dtype)
    g = np.ascontiguousarray(group_of, dtype=np.int32)
    a = np.ascontiguousarray(a, dtype=np.float32)
    out = [np.empty(plan.transport_numel, np.float32) for _ in range(G)]
    lib().kto_intra_reduce(_ptr_array(flat_list), dtype, _p(plan.numel, C.c_int64),
                           _p(plan.tensor_offset, C.c_int64), plan.T, plan.transport_numel,
                           _p(g, C.c_int32), _p(a, C.c_float), K, int(G), _ptr_array(out))
    return out


def combine(partials, W) -> np.ndarray:
    _check_dtype(partials, F32)
    W = np.ascontiguousarray(W, dtype=np.float32)
    n = partials[0].size
    S = np.empty(n, np.float32)
    lib().kto_combine(_ptr_array(partials), _p(W, C.c_float), len(partials), n, S.ctypes.data)
    return S


def unpack_scale(S: np.ndarray, plan: Plan, scale: float, out_dtype: int):
    """Returns the list of T per-parameter flat arrays."""
    assert S.dtype == np.float32 and S.size == plan.transport_numel
    out = [np.empty(int(n), _NP[out_dtype]) for n in plan.numel]
    lib().kto_unpack_scale(S.ctypes.data, _p(plan.numel, C.c_int64),
                           _p(plan.tensor_offset, C.c_int64), plan.T, C.c_float(scale), out_dtype,
                           _ptr_array(out))
    return out


def flat_reduce_f32(x, dtype: int, w_flat) -> np.ndarray:
    _check_dtype(x, dtype)
    w = np.ascontiguousarray(w_flat, dtype=np.float32)
    n = x[0].size
    F = np.empty(n, np.float32)
    lib().kto_flat_reduce_f32(_ptr_array(x), dtype, _p(w, C.c_float), len(x), n, F.ctypes.data)
    return F


def flat_reduce_f64(x, dtype: int, shares):
    """Returns (F, absF): the fp64 weighted mean and sum_r w_r |x_r| per element."""
    _check_dtype(x, dtype)
    b = np.ascontiguousarray(shares, dtype=np.int32)
    n = x[0].size
    F = np.empty(n, np.float64)
    A = np.empty(n, np.float64)
    lib().kto_flat_reduce_f64(_ptr_array(x), dtype, _p(b, C.c_int32), len(x), n, F.ctypes.data,
                              A.ctypes.data)
    return F, A


# --------------------------------------------------------------------------- whole path
def sync_step(grads, numel, dtype: int, group_of, shares, G: int, bucket_cap_bytes: int,
              scale: float = 1.0, out_dtype: int | None = None, transport_dtype: int = F32):
    """The whole path on one thread: plan, intra-group reduce, combine, unpack.

    transport_dtype BF16 (an extension, not the paper's method): every group partial is
    rounded to bf16 (nearest-even) when it is stored in the transport and widened exactly when
    the combine reads it; the returned partials are then the uint16 patterns.

    Returns (out tensors, transport partials, combined buffer, plan)."""
    out_dtype = dtype if out_dtype is None else out_dtype
    plan = bucket_plan(numel, bucket_cap_bytes)
    a, W, _ = coefficients(group_of, shares, G)
    partials = intra_reduce(grads, plan, dtype, group_of, a, G)
    if transport_dtype == BF16:
        partials = [f32_to_bf16(p) for p in partials]
        S = combine([bf16_to_f32(p) for p in partials], W)
    else:
        S = combine(partials, W)
    out = unpack_scale(S, plan, scale, out_dtype)
    return out, partials, S, plan


def sync_step_flat_threads(x, dtype: int, group_of, shares, G: int, scale: float, out_dtype: int,
                           threads: int):
    """The same per-element loops on one flat tensor per rank, the element range cut
    into ``threads`` static slices, one C call chain per slice (ctypes drops the GIL).
    Per-element operation order is unchanged, so results equal the one-thread run."""
    n = x[0].size
    a, W, _ = coefficients(group_of, shares, G)
    out = np.empty(n, _NP[out_dtype])
    step = -(-n // (threads * 64)) * 64
    bounds = [(lo, min(n, lo + step)) for lo in range(0, n, step)]

    def work(b):
        lo, hi = b
        m = hi - lo
        sub = bucket_plan([m], 1 << 62)  # one tensor, one bucket, offset 0
        parts = intra_reduce([[xr[lo:hi]] for xr in x], sub, dtype, group_of, a, G)
        S = combine(parts, W)
        out[lo:hi] = unpack_scale(S, sub, scale, out_dtype)[0]

    with ThreadPoolExecutor(max_workers=threads) as ex:
        list(ex.map(work, bounds))
    return out


def sharded_sync_step(grads, numel, dtype: int, group_of, shares, G: int, bucket_cap_bytes: int, unit: int,
                      scale: float = 1.0, out_dtype: int | None = None, per_bucket: bool = False):
    """The whole path with one rank per device, in the order the devices work (Section III-A:
    collective inside the group, device -> host, exchange between groups in host memory, host ->
    device), every device doing only its own share of each range (shard_ranges):

      1. member m of group g forms the group partial over ITS element range from the tensors
         of all members of g (ascending rank) and stores that range in host memory;
      2. once every range of every group is there, it reads ITS range of every group's
         partial, combines them (ascending group), scales, casts, and writes that range into
         the tensors of every member of its group.

    Returns (out[r][t] for every rank r, the G partials as they stand in host memory, plan).
    Per element the operations are those of sync_step, so every rank must end up with
    sync_step's result."""
    out_dtype = dtype if out_dtype is None else out_dtype
    K = len(grads)
    plan = bucket_plan(numel, bucket_cap_bytes)
    a, W, _ = coefficients(group_of, shares, G)
    members = [[r for r in range(K) if group_of[r] == g] for g in range(G)]
    flat = [pack(grads[r], plan, dtype) for r in range(K)]            # a rank's tensors at the plan's offsets
    host = [np.full(plan.transport_numel, np.nan, np.float32) for _ in range(G)]
    S = [np.full(plan.transport_numel, np.nan, np.float32) for _ in range(G)]   # what group g's members combined
    ranges = [-1] if not per_bucket else list(range(plan.n_buckets))
    for b in ranges:
        for g in range(G):                                            # step 1, every device of every group
            mine = shard_ranges(numel, bucket_cap_bytes, unit, b, len(members[g]))
            for m, (lo, n) in enumerate(mine):
                if n == 0:
                    continue
                sub = bucket_plan([n], 1 << 62)
                part = intra_reduce([[flat[r][lo:lo + n]] for r in members[g]], sub, dtype, [0] * len(members[g]),
                                    [a[r] for r in members[g]], 1)[0]
                host[g][lo:lo + n] = part[:n]
        for g in range(G):                                            # step 2, after the exchange
            mine = shard_ranges(numel, bucket_cap_bytes, unit, b, len(members[g]))
            for m, (lo, n) in enumerate(mine):
                if n:
                    S[g][lo:lo + n] = combine([np.ascontiguousarray(host[h][lo:lo + n]) for h in range(G)], W)
    out = [None] * K
    for g in range(G):
        tensors = unpack_scale(S[g], plan, scale, out_dtype)
        for r in members[g]:
            out[r] = [t.copy() for t in tensors]
    return out, host, plan
