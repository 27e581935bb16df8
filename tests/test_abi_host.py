"""No-GPU checks of the C-ABI library: it builds, loads, exports every symbol the header
declares, and its pure host functions (scheduler, bucket plan, argument validation) agree
with the oracle bit for bit."""
import ctypes
import os
import random
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def kt():
    from paper_2505_10183_b200 import build
    build.build()
    from paper_2505_10183_b200 import binding
    return binding


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "kaitian.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(kt_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(kt):
    from paper_2505_10183_b200 import build
    lib = ctypes.CDLL(build.LIB)
    names = declared_symbols()
    assert len(names) >= 15
    for name in names:
        assert hasattr(lib, name), name
    assert sorted(kt.EXPORTS) == names          # the binding covers the same set
    for name in names:
        assert callable(getattr(kt, name)), name


def test_schedule_bit_exact_against_oracle(kt, oracle):
    rnd = random.Random(42)
    for _ in range(2000):
        K = rnd.randint(1, 64)
        times = [rnd.choice([1.0, 1.4, 1.6, 2.1, rnd.uniform(0.05, 9.0)]) for _ in range(K)]
        B = rnd.randint(K, 4096)
        assert kt.kt_schedule(times, B) == oracle.schedule(times, B).tolist(), (times, B)
    # tiny batches exercise the nobody-idles rule
    for _ in range(500):
        K = rnd.randint(2, 12)
        times = [rnd.choice([1.0, 3.0, 50.0, 1000.0]) for _ in range(K)]
        B = rnd.randint(K, K + 6)
        assert kt.kt_schedule(times, B) == oracle.schedule(times, B).tolist(), (times, B)


@pytest.mark.parametrize("times,B", [([1.0, 0.0], 8), ([1.0, -1.0], 8), ([1.0, float("nan")], 8),
                                     ([1.0, float("inf")], 8), ([1.0] * 3, 2), ([], 4), ([1.0] * 65, 100)])
def test_schedule_rejects_invalid(kt, times, B):
    with pytest.raises(kt.KtError) as e:
        kt.kt_schedule(times, B)
    assert e.value.status == kt.KT_ERR_INVALID
    assert kt.kt_last_error() != ""


def test_plan_buckets_against_oracle(kt, oracle):
    from paper_2505_10183_b200 import workloads as W
    cases = [(W.tiny().numel, 25 << 20), (W.resnet18().numel, 25 << 20), (W.resnet50().numel, 25 << 20),
             (W.mobilenet_v2().numel, 25 << 20), (W.mobilenet_v2().numel, 1 << 20), ([1 << 28], 1 << 62)]
    rnd = random.Random(3)
    for _ in range(300):
        T = rnd.randint(1, 50)
        cases.append(([rnd.choice([0, 1, 7, 8, 9, 63, 64, 65, 100, 1000, 4097, 70000]) for _ in range(T)],
                      rnd.choice([4, 32, 256, 1000, 4096, 20000, 1 << 22, 1 << 40])))
    for numel, cap in cases:
        p = kt.kt_plan_buckets(numel, cap)
        o = oracle.bucket_plan(numel, cap)
        assert p.n_buckets == o.n_buckets
        assert p.tensor_offset == o.tensor_offset.tolist()
        assert p.bucket_of == o.bucket_of.tolist()
        assert p.bucket_start == o.bucket_start.tolist()
        assert p.bucket_numel == o.bucket_numel.tolist()
        assert p.transport_numel == o.transport_numel


def test_argument_validation_needs_no_device(kt):
    E = kt.KtError
    for args in (([0, 2], [1, 1], 3), ([0, 1], [1, 0], 2), ([0, -1], [1, 1], 2), ([0, 0], [1, 1], 3),
                 ([], [], 0), ([0] * 65, [1] * 65, 1)):
        with pytest.raises(E) as e:
            kt.kt_groups_init(*args)
        assert e.value.status == kt.KT_ERR_INVALID
    with pytest.raises(E):
        kt.kt_plan_buckets([4, -1], 1024)
    with pytest.raises(E):
        kt.kt_plan_buckets([4], 2)


def test_missing_library_fails_loudly(tmp_path, monkeypatch):
    """The product path has no fallback: without the built library the binding refuses to import."""
    import importlib
    import sys
    from paper_2505_10183_b200 import build
    monkeypatch.setattr(build, "LIB", str(tmp_path / "nope.so"))
    saved = sys.modules.pop("paper_2505_10183_b200.binding", None)
    try:
        with pytest.raises(ImportError):
            importlib.import_module("paper_2505_10183_b200.binding")
    finally:
        sys.modules.pop("paper_2505_10183_b200.binding", None)
        if saved is not None:
            sys.modules["paper_2505_10183_b200.binding"] = saved


def test_header_is_plain_c_and_links_against_the_library(tmp_path):
    """The boundary is a C ABI: the header must compile as C99 on its own, and a C program
    that calls the pure host entry points must link against the built library and run."""
    import subprocess
    from paper_2505_10183_b200 import build
    src = tmp_path / "abi.c"
    src.write_text(r'''
#include "kaitian.h"
#include <stdio.h>
int main(void) {
    double t[4] = {1.0, 1.0, 1.6, 1.6};
    int32_t b[4];
    if (kt_schedule(t, 4, 256, b) != KT_OK) return 1;
    if (b[0] != 79 || b[1] != 79 || b[2] != 49 || b[3] != 49) return 2;
    int64_t numel[3] = {10, 100, 5}, off[3], total = 0;
    int32_t nb = 0;
    if (kt_plan_buckets(numel, 3, 1 << 20, &nb, 0, 0, off, 0, &total) != KT_OK) return 3;
    if (nb != 1 || off[2] != 0 || off[1] != 8 || off[0] != 112 || total != 128) return 4;
    if (kt_schedule(t, 4, 2, b) != KT_ERR_INVALID || kt_last_error(0)[0] == 0) return 5;
    if (kt_sampler_steps(50000, 256, 0) != 196) return 6;
    printf("ok\n");
    return 0;
}
''')
    exe = tmp_path / "abi"
    inc = os.path.join(ROOT, "include")
    subprocess.check_call(["gcc", "-std=c99", "-Wall", "-Werror", "-pedantic", "-I", inc, "-fsyntax-only", str(src)])
    subprocess.check_call(["gcc", "-std=c99", "-I", inc, str(src), "-o", str(exe), build.LIB, "-lm", "-ldl", "-lpthread", "-lrt",
                           "-lstdc++", "-Wl,-rpath," + os.path.dirname(build.LIB)])
    assert subprocess.check_output([str(exe)]).decode().strip() == "ok"


def test_shard_ranges_match_the_oracle(kt, oracle):
    """One rank per device: the element ranges the library hands to the members of a group are
    the oracle's, on random lists, caps, units and member counts; pure host functions."""
    import random
    rnd = random.Random(1)
    sizes = [0, 1, 7, 8, 9, 63, 64, 65, 500, 2047, 2048, 2049, 4096, 5000, 10000, 40000]
    assert kt.kt_work_unit(kt.KT_F32) == 2048 and kt.kt_work_unit(kt.KT_BF16) == 4096
    for _ in range(400):
        numel = [rnd.choice(sizes) for _ in range(rnd.randint(1, 12))]
        cap, unit, M = rnd.choice([64, 4096, 40000, 1 << 20, 1 << 40]), rnd.choice([2048, 4096, 64]), rnd.randint(1, 9)
        nb = kt.kt_plan_buckets(numel, cap).n_buckets
        for b in [-1] + list(range(nb)):
            assert kt.kt_shard_ranges(numel, cap, unit, b, M) == oracle.shard_ranges(numel, cap, unit, b, M)
    for bad in (([5], 1 << 20, 0, -1, 2), ([5], 1 << 20, 2048, 1, 2), ([5], 1 << 20, 2048, -1, 0), ([-1], 1 << 20, 2048, -1, 1)):
        with pytest.raises(kt.KtError):
            kt.kt_shard_ranges(*bad)
    with pytest.raises(kt.KtError):
        kt.kt_work_unit(7)


def test_shared_memory_calls_validate_arguments(kt):
    """kt_ipc_* and kt_host_register refuse null addresses, negative offsets and empty ranges on
    the host, before any CUDA call (so this runs without a device)."""
    for call in (lambda: kt.kt_ipc_export(0), lambda: kt.kt_ipc_open(b"\0" * kt.KT_IPC_HANDLE_BYTES, -1),
                 lambda: kt.kt_host_register(0, 4096), lambda: kt.kt_host_register(4096, 0),
                 lambda: kt.kt_host_unregister(0)):
        with pytest.raises(kt.KtError) as e:
            call()
        assert e.value.status == kt.KT_ERR_INVALID


def test_host_arithmetic_at_extreme_values_matches_the_oracle(kt, oracle):
    """Sizes beyond 2^31 and 2^40 elements, caps from 4 bytes to 2^63 - 1, step times from the
    smallest subnormal to the largest double, batches up to 2^31 - 1: the library's host
    functions and the oracle must agree on every result and on what they reject."""
    rnd = random.Random(99)
    big = [0, 1, 7, 8, 9, 63, 64, 65, 2047, 2048, 2049, 4096, (1 << 31) - 1, 1 << 31, (1 << 31) + 1, (1 << 33) + 5,
           (1 << 40) + 3, 1 << 45]
    caps = [4, 63, 64, 256, 4096, 1 << 20, 25 << 20, 1 << 40, 1 << 62, (1 << 63) - 1]

    def outcome(fn):
        try:
            return fn()
        except (kt.KtError, oracle.OracleError):
            return "rejected"

    for _ in range(1500):
        T = rnd.randint(1, 8)
        numel = [rnd.choice(big) if rnd.random() < 0.6 else rnd.randint(0, 100000) for _ in range(T)]
        if sum(numel) == 0:
            numel[0] = 3
        cap = rnd.choice(caps)
        po, pl = outcome(lambda: oracle.bucket_plan(numel, cap)), outcome(lambda: kt.kt_plan_buckets(numel, cap))
        assert (po == "rejected") == (pl == "rejected"), (numel, cap)
        if po == "rejected":
            continue
        assert (pl.n_buckets, pl.tensor_offset, pl.bucket_of, pl.bucket_start, pl.bucket_numel, pl.transport_numel) == \
            (po.n_buckets, po.tensor_offset.tolist(), po.bucket_of.tolist(), po.bucket_start.tolist(),
             po.bucket_numel.tolist(), po.transport_numel), (numel, cap)
        if sum(numel) <= 1 << 32:                    # the oracle walks the range unit by unit
            unit, M, b = rnd.choice([2048, 4096]), rnd.randint(1, 9), rnd.randint(-1, po.n_buckets - 1)
            assert outcome(lambda: oracle.shard_ranges(numel, cap, unit, b, M)) == \
                outcome(lambda: kt.kt_shard_ranges(numel, cap, unit, b, M)), (numel, cap, unit, b, M)
    times = [5e-324, 1e-300, 1e-30, 1e-9, 0.5, 1.0, 1.0000000000000002, 3.0, 1e9, 1e30, 1e300, 1.7976931348623157e308]
    for _ in range(1500):
        K = rnd.randint(1, 64)
        ts = [rnd.choice(times) if rnd.random() < 0.5 else rnd.uniform(0.001, 1000) for _ in range(K)]
        B = rnd.choice([K, K + 1, 2 * K, 256, 65536, (1 << 31) - 1, rnd.randint(K, 100000)])
        a = outcome(lambda: oracle.schedule(ts, B).tolist())
        assert a == outcome(lambda: kt.kt_schedule(ts, B)), (ts, B)
        assert a == "rejected" or (sum(a) == B and min(a) >= 1)
        assert outcome(lambda: oracle.scores(ts).tolist()) == outcome(lambda: kt.kt_scores(ts))
