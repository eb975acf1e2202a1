"""CPU-side checks of the C-ABI library: it builds, loads, exports every symbol
the header declares, and its host-only entry points agree with the oracle.
No compute call is made here (no GPU)."""
import ctypes
import os
import re

import numpy as np
import pytest

from oracle import d3tom_oracle as orc
from paper_2511_12280_b200 import binding as B_
from paper_2511_12280_b200 import build as build_mod

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build_mod.build()
    return B_.load()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "d3tom.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(d3tom_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(lib):
    names = declared_functions()
    assert len(names) >= 14
    for n in names:
        assert hasattr(lib, n), "missing export: " + n
    # the Python binding mirrors the same set of names
    assert sorted(B_.exported_symbols()) == names


def test_status_strings(lib):
    assert B_.status_string(0) == "ok"
    for code in (B_.ERR_INVALID_ARG, B_.ERR_UNSUPPORTED, B_.ERR_WORKSPACE, B_.ERR_CUDA, B_.ERR_TIMEOUT):
        assert B_.status_string(code) not in ("ok", "unknown status")
    assert B_.status_string(-99) == "unknown status"


def test_keep_count_matches_oracle(lib):
    rng = np.random.default_rng(0)
    for V in [1, 2, 7, 100, 256, 1000, 1024, 2048, 4096]:
        for r in [0.0, 0.05, 0.1, 1 - 0.9, 0.25, 1 / 3, 0.5, 0.999, 1.0, 1.7] + rng.random(20).tolist():
            assert B_.d3tom_keep_count(V, r) == orc.keep_count(V, r), (V, r)
    assert B_.d3tom_keep_count(1024, 0.10) == 102
    assert B_.d3tom_keep_count(1000, 1 - 0.9) == 100
    assert B_.d3tom_keep_count(0, 0.5) == 0


def test_schedule_alpha_matches_oracle(lib):
    for T in (1, 2, 32, 64):
        for rev in (False, True):
            for s in range(T):
                got = B_.d3tom_schedule_alpha(s, T, 0.5, 1.0, rev)
                assert abs(got - orc.schedule_alpha(s, T, 0.5, 1.0, rev)) < 1e-15
    with pytest.raises(B_.D3tomError):
        B_.d3tom_schedule_alpha(5, 5, 0.0, 1.0)
    # the step schedule of the T=64 config: keep counts fall from 2*mean to the clamp at 1
    ks = [B_.d3tom_keep_count(2048, 1.0 - B_.d3tom_schedule_alpha(s, 64, 0.5, 1.0)) for s in range(64)]
    assert ks[0] == 1024 and ks[-1] == 1 and all(a >= b for a, b in zip(ks, ks[1:]))


def test_host_argument_errors_need_no_gpu(lib):
    # null / inconsistent arguments are rejected on the host before any CUDA work
    assert lib.d3tom_create(None, 0, None) == B_.ERR_INVALID_ARG
    h = ctypes.c_void_p()
    bad = B_.Limits(0, 1, 1, 64, 1, 1)
    assert lib.d3tom_create(ctypes.byref(h), 0, ctypes.byref(bad)) == B_.ERR_INVALID_ARG
    assert lib.d3tom_destroy(None) == B_.ERR_INVALID_ARG
    assert lib.d3tom_select(None, None, None, None, None, 1, 1, None, None, None) == B_.ERR_INVALID_ARG
    assert lib.d3tom_proj_qkv(None, 0, None, None, 1, 64, None, None, None, None) == B_.ERR_INVALID_ARG


def test_create_fails_cleanly_without_a_device(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    h = ctypes.c_void_p()
    lim = B_.Limits(128, 1, 1, 64, 1, 64)
    assert lib.d3tom_create(ctypes.byref(h), 0, ctypes.byref(lim)) < 0
    assert not h.value


def test_product_package_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2511_12280_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert not re.search(r"(import\s+oracle|from\s+oracle|oracle[./]d3tom|oracle/)", src), os.path.join(dirpath, f)


def test_log_line_per_call_when_the_environment_asks_for_it():
    # D3TOM_LOG=1: one line per call on stderr with sizes and status; silent otherwise.  Without a GPU
    # d3tom_create fails on the host, which is enough to see both behaviours.
    import subprocess
    import sys
    code = ("from paper_2511_12280_b200 import binding as B\n"
            "try:\n    B.Context(128, 1, 2, 64, 1, 64).close()\nexcept B.D3tomError:\n    pass\n")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    for val, expect in (("1", True), ("0", False), (None, False)):
        env = dict(os.environ)
        env.pop("D3TOM_LOG", None)
        if val is not None:
            env["D3TOM_LOG"] = val
        r = subprocess.run([sys.executable, "-c", code], cwd=root, env=env, capture_output=True, text=True)
        assert r.returncode == 0, r.stderr
        has = "[d3tom] d3tom_create device 0: tokens 128 batch 1 heads 2 x 64" in r.stderr
        assert has == expect, (val, r.stderr)
