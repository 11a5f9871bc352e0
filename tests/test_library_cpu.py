"""Host-only checks of the CUDA library: it loads, exports what include/rubick.h declares,
its structs have the documented sizes, and its host logic (plan enumeration, argument checks)
behaves.  No compute call is made, so no GPU is needed."""
import ctypes as C
import os
import re

import numpy as np
import pytest

import oracle
from paper_2408_08586_b200 import binding as rb
from paper_2408_08586_b200 import build as rbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    rbuild.build()
    return rb.lib()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "rubick.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(rubick_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert set(names) == set(rb.EXPORTS)
    for n in names:
        assert getattr(lib, n) is not None


def test_struct_sizes_match_the_header():
    assert rb.JOB_DTYPE.itemsize == 128 and rb.JOB_DTYPE.fields["tau"][1] == 40 and rb.JOB_DTYPE.fields["w"][1] == 72
    assert rb.PLAN_DTYPE.itemsize == 8
    assert rb.ASSIGN_DTYPE.itemsize == 40 and rb.ASSIGN_DTYPE.fields["thr"][1] == 28
    assert rb.NODE_DTYPE.itemsize == 24
    assert C.sizeof(rb.Env) == 64 and C.sizeof(rb.Grid) == 40 and C.sizeof(rb.Cluster) == 24
    assert rb.JOB_DTYPE.fields["tenant"][1] == 88


@pytest.mark.parametrize("levels", [[1, 2, 3, 4, 5, 6, 7, 8], [1, 2, 4, 8, 16, 32, 64], [1 << i for i in range(9)], [4, 12, 16]])
def test_plan_enumeration_matches_the_oracle(lib, levels):
    a, aoff = rb.enumerate_plans(levels)
    b, boff = oracle.enumerate_plans(levels)
    assert np.array_equal(aoff, boff) and len(a) == len(b)
    got = np.stack([1 << a["log2d"].astype(np.int64), 1 << a["log2t"].astype(np.int64), 1 << a["log2p"].astype(np.int64),
                    a["zero"], a["gc"], a["off"]], axis=1)
    assert np.array_equal(got, b[:, :6]) and not b[:, 6].any()
    assert np.array_equal(a["g_level"], np.repeat(np.arange(len(levels)), np.diff(aoff)))


def test_plan_enumeration_capacity_and_errors(lib):
    gl = np.array([1, 2, 4], dtype=np.int32)
    n = C.c_int(0)
    few = np.zeros(5, dtype=rb.PLAN_DTYPE)
    assert lib.rubick_enumerate_plans(gl.ctypes.data, 3, few.ctypes.data, 5, C.byref(n), None) == rb.OK
    assert n.value == 16 * (1 + 3 + 6)                      # the full count is reported, 5 were written
    assert few["zero"].tolist() == [0, 0, 0, 0, 1]
    bad = np.array([1, 1, 2], dtype=np.int32)
    assert lib.rubick_enumerate_plans(bad.ctypes.data, 3, None, 0, C.byref(n), None) == rb.EINVAL
    assert lib.rubick_enumerate_plans(gl.ctypes.data, 0, None, 0, C.byref(n), None) == rb.EINVAL
    assert lib.rubick_enumerate_plans(None, 3, None, 0, C.byref(n), None) == rb.EINVAL


def test_create_rejects_bad_environments_and_missing_devices(lib):
    from paper_2408_08586_b200 import workloads
    h = C.c_void_p()
    e = rb.Env(400e9, 100e9, 25e9, 80 * 10**9, 1 << 40, 6, 96, 2, 0)        # 6 GPUs per node: not a power of two
    assert lib.rubick_create(C.byref(h), C.byref(e), 0, None) == rb.EINVAL and not h.value
    e = rb.Env(0.0, 100e9, 25e9, 80 * 10**9, 1 << 40, 8, 96, 2, 0)
    assert lib.rubick_create(C.byref(h), C.byref(e), 0, None) == rb.EINVAL
    assert lib.rubick_create(None, C.byref(e), 0, None) == rb.EINVAL
    import torch
    if not torch.cuda.is_available():
        ok = rb.Env(400e9, 100e9, 25e9, 80 * 10**9, 1 << 40, 8, 96, 2, 0)
        assert lib.rubick_create(C.byref(h), C.byref(ok), 0, None) == rb.ECUDA     # no fallback: fails loudly
        with pytest.raises(rb.RubickError):
            rb.Context(workloads.ENV)
    assert lib.rubick_sync(None) == rb.EINVAL
    lib.rubick_destroy(None)


def test_job_packing_round_trips():
    from paper_2408_08586_b200 import workloads
    cfg = workloads.make("paper-scale")
    rec = rb.pack_jobs(cfg["jobs"])
    assert rec.dtype == rb.JOB_DTYPE and len(rec) == 64
    for k in ("P", "l", "h", "s", "b", "mu_cap", "alpha_act", "gmin_idx", "cmin_idx", "host_base_bytes"):
        assert np.array_equal(rec[k].astype(np.float64), np.asarray(cfg["jobs"][k], dtype=np.float64))
    for k in ("tau", "k_bwd", "k_sync", "k_opt", "k_opt_off", "k_off", "k_swap", "k_const", "w"):
        assert np.array_equal(rec[k].astype(np.float64), cfg["jobs"][k])      # generator values are float32-exact
