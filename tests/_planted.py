"""Planting a mistake in a temporary copy of the CPU oracle (tests of the tests: the pins and the
parity comparisons have to notice a wrong oracle).  Nothing here changes the committed oracle,
and nothing here runs on a GPU."""
from __future__ import annotations

import importlib.util
import os
import shutil

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
ORACLE = os.path.join(ROOT, "oracle")
SOURCES = ("kt_oracle.c", "kt_oracle.py")


def write_oracle_copy(dst: str, name: str, old: str, new: str, occurrence=None) -> None:
    """Copies the oracle package into the new folder `dst` with one piece of text replaced.
    `old` is looked for in the C source first, then in the Python side (the whole-path
    drivers).  occurrence None: the text must occur exactly once; k: the k-th occurrence."""
    os.makedirs(dst)
    for f in ("__init__.py",) + SOURCES:
        shutil.copy(os.path.join(ORACLE, f), os.path.join(dst, f))
    for target in SOURCES:
        src = open(os.path.join(ORACLE, target)).read()
        if old in src:
            break
    at = -1
    for _ in range((occurrence or 0) + 1):
        at = src.find(old, at + 1)
        assert at >= 0, "mistake %r: the text to change is not in the oracle's source (any more)" % name
    if occurrence is None:
        assert src.find(old, at + 1) < 0, "mistake %r: the text to change is not unique" % name
    with open(os.path.join(dst, target), "w") as f:
        f.write(src[:at] + new + src[at + len(old):])


def load_oracle_copy(dst: str, module_name: str):
    """Imports the copy's loader under a name of its own (it builds and loads the C file that
    lies beside it, not the committed one)."""
    spec = importlib.util.spec_from_file_location(module_name, os.path.join(dst, "kt_oracle.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    mod.lib()
    return mod
