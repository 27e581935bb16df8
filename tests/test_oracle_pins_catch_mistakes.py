"""The oracle's pins must fail when the oracle is wrong.

Each case below plants one plausible mistake in a copy of the oracle's C source (a dropped
weight, a swapped order, a wrong rounding, an index off by one ...), builds that copy, and runs
the pin tests (tests/test_oracle_*.py) against it in a process of their own.  The run has to
fail: a mistake that every pin lets through would mean that this part of the oracle is checked
against nothing but itself.  Tests whose only expected value is the CUDA library's result are
left out of these runs: agreement between the two implementations pins neither.

The mistakes live in temporary copies on the CPU; nothing here touches the committed oracle or
the CUDA path.
"""
import os
import shutil
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

import pytest

from _planted import write_oracle_copy

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
PIN_FILES = ["test_oracle_schedule.py", "test_oracle_sampler_adapt.py", "test_oracle_sharding.py",
             "test_oracle_datapath.py"]

# (name, pin file that has to catch it, text in kt_oracle.c, replacement, which occurrence of the
#  text: None = it occurs once)
MISTAKES = [
    # --- scores and shares (Section III-C)
    ("score inverted", "test_oracle_schedule.py",
     "scores[i] = t_min / step_times[i];", "scores[i] = step_times[i] / t_min;", None),
    ("shares follow the time, not the speed", "test_oracle_schedule.py",
     "score[i] = t_min / step_times[i];", "score[i] = step_times[i] / t_min;", None),
    ("quotas truncated, remainder all to rank 0", "test_oracle_schedule.py",
     "if (frac[i] >= 0.0 && (best < 0 || frac[i] > frac[best]))", "if (frac[i] >= 0.0 && best < 0)", None),
    ("equal remainders go to the higher rank", "test_oracle_schedule.py",
     "frac[i] > frac[best]", "frac[i] >= frac[best]", None),
    ("a rank may get zero samples", "test_oracle_schedule.py",
     "if (shares[i] >= 1)", "if (shares[i] >= 0)", None),
    ("the one sample for an idle rank comes from the fastest of the largest", "test_oracle_schedule.py",
     "step_times[j] >= step_times[big]", "step_times[j] < step_times[big]", None),
    # --- weights of the two-level mean
    ("in-group weight divided by the global batch", "test_oracle_schedule.py",
     "a[r] = (float)((double)shares[r] / (double)Bg[group_of[r]]);", "a[r] = (float)((double)shares[r] / (double)B);", None),
    ("groups weighted equally", "test_oracle_schedule.py",
     "W[g] = (float)((double)Bg[g] / (double)B);", "W[g] = (float)(1.0 / (double)G);", None),
    ("flat weight divided by the rank count", "test_oracle_schedule.py",
     "w_flat[r] = (float)((double)shares[r] / (double)B);", "w_flat[r] = (float)(1.0 / (double)K);", None),
    ("weights rounded twice", "test_oracle_schedule.py",
     "a[r] = (float)((double)shares[r] / (double)Bg[group_of[r]]);",
     "a[r] = (float)shares[r] * (1.0f / (float)Bg[group_of[r]]);", None),
    ("route looks at the first two participants only", "test_oracle_schedule.py",
     "for (int i = 1; i < n; ++i)\n        if (group_of[participants[i]]", "for (int i = 1; i < n && i < 2; ++i)\n        if (group_of[participants[i]]", None),
    # --- online adaptation
    ("moving average with the factor on the wrong term", "test_oracle_sampler_adapt.py",
     "(1.0 - alpha) * ema[r] + alpha * tau", "alpha * ema[r] + (1.0 - alpha) * tau", None),
    ("step time not divided by the samples it was spent on", "test_oracle_sampler_adapt.py",
     "double tau = step_times[r] / (double)shares[r];", "double tau = step_times[r];", None),
    ("no hysteresis", "test_oracle_sampler_adapt.py",
     "then < (1.0 - hysteresis) * now", "then < now", None),
    ("hysteresis widens the threshold instead of narrowing it", "test_oracle_sampler_adapt.py",
     "then < (1.0 - hysteresis) * now", "then < (1.0 + hysteresis) * now", None),
    ("new shares taken at exactly the threshold", "test_oracle_sampler_adapt.py",
     "then < (1.0 - hysteresis) * now", "then <= (1.0 - hysteresis) * now", None),
    ("the first observation is averaged with zero", "test_oracle_sampler_adapt.py",
     "if (*count == 0)\n            ema[r] = tau;", "if (0)\n            ema[r] = tau;", None),
    ("shares recomputed on every observation", "test_oracle_sampler_adapt.py",
     "if (*count % period != 0)", "if (0)", None),
    # --- sampler
    ("one step too many when the batch divides the data set", "test_oracle_sampler_adapt.py",
     "return (dataset_size + global_batch - 1) / global_batch;", "return dataset_size / global_batch + 1;", None),
    ("every rank reads from the start of the step", "test_oracle_sampler_adapt.py",
     "(s * B + c + j) % dataset_size", "(s * B + j) % dataset_size", None),
    ("sampler positions shifted by one", "test_oracle_sampler_adapt.py",
     "(s * B + c + j) % dataset_size", "(s * B + c + j + 1) % dataset_size", None),
    ("steps advance by the rank's share, not the global batch", "test_oracle_sampler_adapt.py",
     "(s * B + c + j) % dataset_size", "(s * shares[r] + c + j) % dataset_size", None),
    # --- bucket plan
    ("tensors start at multiples of 4", "test_oracle_datapath.py",
     "int64_t off = round_up(cursor, 8);", "int64_t off = round_up(cursor, 4);", None),
    ("buckets start at multiples of 32", "test_oracle_datapath.py",
     "start = round_up(cursor, 64);", "start = round_up(cursor, 32);", None),
    ("a bucket closes one element early", "test_oracle_datapath.py",
     "(off - start) + numel[t] > cap", "(off - start) + numel[t] >= cap", None),
    ("cap counted in bytes", "test_oracle_datapath.py",
     "const int64_t cap = bucket_cap_bytes / 4;", "const int64_t cap = bucket_cap_bytes;", None),
    ("tensors visited in list order", "test_oracle_datapath.py",
     "for (int t = T - 1; t >= 0; --t) {\n        int64_t off", "for (int t = 0; t < T; ++t) {\n        int64_t off", None),
    ("transport not padded to 64", "test_oracle_datapath.py",
     "const int64_t total = round_up(cursor, 64);", "const int64_t total = round_up(cursor, 8);", None),
    # --- share ranges of one rank per device
    ("short last unit counted as a full one", "test_oracle_sharding.py",
     "const int64_t len = extent - at < unit ? extent - at : unit;", "const int64_t len = unit;", None),
    ("units split with the remainder to the first members", "test_oracle_sharding.py",
     "const int64_t first = (int64_t)m * U / n_members;\n                    const int64_t past = (int64_t)(m + 1) * U / n_members;",
     "const int64_t first = ((int64_t)m * U + n_members - 1) / n_members;\n"
     "                    const int64_t past = ((int64_t)(m + 1) * U + n_members - 1) / n_members;", None),
    ("a tensor's padding left out of its units", "test_oracle_sharding.py",
     "const int64_t extent = end - offset[t];", "const int64_t extent = numel[t];", None),
    # --- casts
    ("narrowing truncates", "test_oracle_datapath.py", "u += 0x7FFFu + lsb;", "u += 0u;", None),
    ("ties away from zero", "test_oracle_datapath.py", "u += 0x7FFFu + lsb;", "u += 0x8000u;", None),
    ("ties towards zero", "test_oracle_datapath.py", "u += 0x7FFFu + lsb;", "u += 0x7FFFu;", None),
    ("NaN not made quiet", "test_oracle_datapath.py", "((u >> 16) | 0x0040u)", "(u >> 16)", None),
    ("NaN test takes infinity for a NaN", "test_oracle_datapath.py",
     "(u & 0x7FFFFFFFu) > 0x7F800000u", "(u & 0x7FFFFFFFu) >= 0x7F800000u", None),
    # --- pack, broadcast copy
    ("padding of the pack not zero", "test_oracle_datapath.py",
     "memset(flat, 0, (size_t)transport_numel", "memset(flat, 0x55, (size_t)transport_numel", None),
    ("pack offset in elements used as bytes", "test_oracle_datapath.py",
     "unsigned char *dst = (unsigned char *)flat + tensor_offset[t] * elem_size;",
     "unsigned char *dst = (unsigned char *)flat + tensor_offset[t];", None),
    ("pack drops a tensor's last element", "test_oracle_datapath.py",
     "for (int64_t j = 0; j < numel[t] * elem_size; ++j)", "for (int64_t j = 0; j < (numel[t] - 1) * elem_size; ++j)", 0),
    ("copy out of the flat buffer drops a tensor's last element", "test_oracle_datapath.py",
     "for (int64_t j = 0; j < numel[t] * elem_size; ++j)", "for (int64_t j = 0; j < (numel[t] - 1) * elem_size; ++j)", 1),
    ("copy out of the flat buffer reads at the element offset as bytes", "test_oracle_datapath.py",
     "(const unsigned char *)flat + tensor_offset[t] * elem_size;", "(const unsigned char *)flat + tensor_offset[t];", None),
    # --- intra-group reduce
    ("later terms as multiply then add (two roundings)", "test_oracle_datapath.py",
     "acc = fmaf(a[r], x, acc);", "acc = acc + a[r] * x;", None),
    ("ranks of a group taken in descending order", "test_oracle_datapath.py",
     "for (int r = 0; r < K; ++r) {\n                    if (group_of[r] != g)",
     "for (int r = K - 1; r >= 0; --r) {\n                    if (group_of[r] != g)", None),
    ("in-group weight dropped from the first term", "test_oracle_datapath.py",
     "acc = a[r] * x;\n                        first = 0;", "acc = x;\n                        first = 0;", None),
    ("partial holds the other groups' ranks", "test_oracle_datapath.py",
     "if (group_of[r] != g)\n                        continue;\n                    float x", "if (group_of[r] == g && G > 1)\n                        continue;\n                    float x", None),
    ("padding of the partial not zero", "test_oracle_datapath.py", "P[i] = 0.0f;", "P[i] = 1.0f;", None),
    ("partial written one element late", "test_oracle_datapath.py",
     "P[tensor_offset[t] + j] = acc;", "P[tensor_offset[t] + j + (j + 1 < numel[t])] = acc;", None),
    # --- inter-group combine
    ("combine as multiply then add", "test_oracle_datapath.py",
     "acc = fmaf(W[g], partials[g][i], acc);", "acc = acc + W[g] * partials[g][i];", None),
    ("group weight dropped from the first group", "test_oracle_datapath.py",
     "float acc = W[0] * partials[0][i];", "float acc = partials[0][i];", None),
    ("groups combined in descending order", "test_oracle_datapath.py",
     "float acc = W[0] * partials[0][i];\n        for (int g = 1; g < G; ++g)\n            acc = fmaf(W[g], partials[g][i], acc);",
     "float acc = W[G - 1] * partials[G - 1][i];\n        for (int g = G - 2; g >= 0; --g)\n            acc = fmaf(W[g], partials[g][i], acc);", None),
    # --- unpack + scale
    ("scale dropped", "test_oracle_datapath.py",
     "float y = S[tensor_offset[t] + j] * scale;", "float y = S[tensor_offset[t] + j];", None),
    ("bf16 output truncated, not rounded", "test_oracle_datapath.py",
     "((uint16_t *)out[t])[j] = kto_f32_to_bf16_one(y);", "((uint16_t *)out[t])[j] = (uint16_t)(f32_to_bits(y) >> 16);", None),
    ("unpack reads from the tensor's list position", "test_oracle_datapath.py",
     "float y = S[tensor_offset[t] + j] * scale;", "float y = S[tensor_offset[T - 1 - t] + j] * scale;", None),
    # --- flat means
    ("flat fp32 mean as multiply then add", "test_oracle_datapath.py",
     "acc = fmaf(w_flat[r], load_as_f32(x[r], in_dtype, i), acc);", "acc = acc + w_flat[r] * load_as_f32(x[r], in_dtype, i);", None),
    ("flat fp64 mean divided by the rank count", "test_oracle_datapath.py",
     "F[i] = acc / (double)B;", "F[i] = acc / (double)K;", None),
    ("flat fp64 mean unweighted", "test_oracle_datapath.py",
     "acc += (double)shares[r] * v;", "acc += (double)B / (double)K * v;", None),
    # --- the whole-path drivers (Python side of the oracle)
    ("bf16 transport: the combine reads the partials before they were rounded", "test_oracle_datapath.py",
     "partials = [f32_to_bf16(p) for p in partials]\n        S = combine([bf16_to_f32(p) for p in partials], W)",
     "S = combine(partials, W)\n        partials = [f32_to_bf16(p) for p in partials]", None),
    ("broadcast sends rank 0's tensors whoever the root is", "test_oracle_datapath.py",
     "flat = pack(tensors[root], plan, dtype)", "flat = pack(tensors[0], plan, dtype)", None),
    ("whole path combines with equal group weights", "test_oracle_datapath.py",
     "    else:\n        S = combine(partials, W)\n    out = unpack_scale(S, plan, scale, out_dtype)",
     "    else:\n        S = combine(partials, np.full(G, 1.0 / G, np.float32))\n    out = unpack_scale(S, plan, scale, out_dtype)", None),
    ("sharded path: a member weights its mates' tensors with the first ranks' weights", "test_oracle_sharding.py",
     "[a[r] for r in members[g]], 1)[0]", "[a[i] for i in range(len(members[g]))], 1)[0]", None),
    ("sharded path: a member combines its own group's partial only", "test_oracle_sharding.py",
     "combine([np.ascontiguousarray(host[h][lo:lo + n]) for h in range(G)], W)",
     "combine([np.ascontiguousarray(host[g][lo:lo + n]) for h in range(G)], W)", None),
]


def make_tree(tmp, name, old, new, occurrence):
    """A miniature of the repository in `tmp`: the pin tests and their fixtures, the package (by
    link: the pin tests take the workloads' shapes from it), and the oracle with one mistake."""
    os.makedirs(os.path.join(tmp, "tests"))
    for f in PIN_FILES + ["conftest.py"]:
        shutil.copy(os.path.join(ROOT, "tests", f), os.path.join(tmp, "tests", f))
    shutil.copytree(os.path.join(ROOT, "tests", "golden"), os.path.join(tmp, "tests", "golden"))
    os.symlink(os.path.join(ROOT, "paper_2505_10183_b200"), os.path.join(tmp, "paper_2505_10183_b200"))
    os.symlink(os.path.join(ROOT, "include"), os.path.join(tmp, "include"))
    write_oracle_copy(os.path.join(tmp, "oracle"), name, old, new, occurrence)


def run_pins(tmp, pin_file):
    env = dict(os.environ, PYTHONDONTWRITEBYTECODE="1")
    env.pop("PYTHONPATH", None)
    return subprocess.run(
        [sys.executable, "-m", "pytest", os.path.join("tests", pin_file), "-x", "-q", "-m", "not gpu",
         "-p", "no:cacheprovider", "-k", "not test_library_"],
        cwd=tmp, env=env, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True, timeout=600)


def test_unchanged_copy_passes_its_pins(tmp_path):
    """The miniature tree itself is sound: with no mistake planted every pin file is green (so a
    failure in the cases below comes from the mistake, not from the copy)."""
    tmp = str(tmp_path / "clean")
    make_tree(tmp, "none", "int kto_scores(", "int kto_scores(", None)
    with ThreadPoolExecutor(len(PIN_FILES)) as pool:
        for f, res in zip(PIN_FILES, pool.map(lambda f: run_pins(tmp, f), PIN_FILES)):
            assert res.returncode == 0, "%s fails on an unchanged copy:\n%s" % (f, res.stdout[-3000:])


def test_every_planted_mistake_fails_a_pin(tmp_path):
    def one(case):
        i, (name, pin_file, old, new, occurrence) = case
        tmp = str(tmp_path / ("m%02d" % i))
        make_tree(tmp, name, old, new, occurrence)
        res = run_pins(tmp, pin_file)
        # 1 = tests failed; anything else (2 interrupted, 4 usage, 5 nothing collected) is a broken run
        return name, pin_file, res.returncode, res.stdout[-1500:]

    with ThreadPoolExecutor(min(8, os.cpu_count() or 2)) as pool:
        results = list(pool.map(one, enumerate(MISTAKES)))
    survived = [(n, f) for n, f, rc, _ in results if rc == 0]
    broken = [(n, f, rc, out) for n, f, rc, out in results if rc not in (0, 1)]
    assert not broken, "runs that did not get as far as the pins: %r" % broken
    assert not survived, "mistakes that every pin let through: %r" % survived
