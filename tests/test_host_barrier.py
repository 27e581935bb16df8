"""The barrier between the processes of a node (kt_host_barrier) on CPU: pure host code on a
block of shared memory.  Four processes run a thousand rounds and check after every round that
all of them have finished the round before; then a rank stays away and the others get
KT_ERR_TIMEOUT within the limit they asked for, which is how a dead or hung rank shows up
without any GPU being involved."""
import ctypes as C
import mmap
import os
import sys
import time

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _map(path, nbytes):
    fd = os.open(path, os.O_RDWR)
    m = mmap.mmap(fd, nbytes)
    os.close(fd)
    view = C.c_char.from_buffer(m)
    return m, view, C.addressof(view)


def _rounds(rank, world, path, rounds, results):
    sys.path.insert(0, ROOT)
    from paper_2505_10183_b200 import binding as kt
    m, view, base = _map(path, 4096)
    slots = (C.c_int64 * world).from_address(base + 1024)
    ok = True
    for i in range(1, rounds + 1):
        slots[rank] = i                                   # my progress, written before the barrier
        kt.kt_host_barrier(base, world, 20000)
        ok = ok and all(slots[r] >= i for r in range(world))   # nobody is behind the round just closed
        if rank == i % world:
            time.sleep(0.0002)                            # stagger arrivals
    results[rank] = ok
    del slots, view
    m.close()


def _absent(rank, world, path, results):
    sys.path.insert(0, ROOT)
    from paper_2505_10183_b200 import binding as kt
    m, view, base = _map(path, 4096)
    if rank == world - 1:
        results[rank] = "stayed away"                     # never joins
    else:
        t0 = time.time()
        try:
            kt.kt_host_barrier(base, world, 300)
            results[rank] = "passed"
        except kt.KtError as e:
            results[rank] = (e.status, time.time() - t0, str(e))
    del view
    m.close()


def _shared_file(tmp_path, name):
    path = str(tmp_path / name)
    with open(path, "wb") as f:
        f.write(b"\0" * 4096)
    return path


def test_a_thousand_rounds_with_four_processes(tmp_path):
    path = _shared_file(tmp_path, "barrier")
    with mp.Manager() as mgr:
        results = mgr.dict()
        mp.spawn(_rounds, args=(4, path, 1000, results), nprocs=4, join=True)
        assert [results[r] for r in range(4)] == [True] * 4


def test_a_rank_that_never_joins_ends_the_wait_with_a_timeout_status(tmp_path):
    from paper_2505_10183_b200 import binding as kt
    path = _shared_file(tmp_path, "barrier_absent")
    with mp.Manager() as mgr:
        results = mgr.dict()
        mp.spawn(_absent, args=(3, path, results), nprocs=3, join=True)
        for r in (0, 1):
            status, waited, message = results[r]
            assert status == kt.KT_ERR_TIMEOUT and 0.25 <= waited < 5.0
            assert "of 3 ranks had arrived" in message
    # argument checks, and the single-rank barrier returns at once
    buf = (C.c_char * 256)()
    base = (C.addressof(buf) + 63) // 64 * 64
    kt.kt_host_barrier(base, 1, 0)
    for bad in ((0, 1, 0), (base + 8, 1, 0), (base, 0, 0)):
        try:
            kt.kt_host_barrier(*bad)
            raise AssertionError("accepted %r" % (bad,))
        except kt.KtError as e:
            assert e.status in (kt.KT_ERR_INVALID, kt.KT_ERR_ALIGN)
