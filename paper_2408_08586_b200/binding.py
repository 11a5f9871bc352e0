"""Thin ctypes binding of ``librubick.so`` (see ``include/rubick.h``).

Argument marshalling only: every step of the path runs in the library's CUDA kernels.  Device
buffers are ordinary torch CUDA tensors (torch is used for device memory and streams, nothing
else); the binding passes their ``data_ptr()``.  There is no CPU fallback: if the shared
library has not been built, importing the native handle raises.
"""
import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "librubick.so")

OK, EINVAL, ENOMEM, ECUDA, ESTEPS, ESTATE = 0, -1, -2, -3, -4, -5
UNALLOCATED, RUNNING, PENDING = 0, 1, 2
BEST_RAW = 1
NOALLOC_MAX_JOBS = 32768

JOB_DTYPE = np.dtype([
    ("P", "<f8"), ("host_base_bytes", "<i8"), ("l", "<i4"), ("h", "<i4"), ("s", "<i4"), ("b", "<i4"),
    ("mu_cap", "<i4"), ("alpha_act", "<i4"), ("tau", "<f4"), ("k_bwd", "<f4"), ("k_sync", "<f4"),
    ("k_opt", "<f4"), ("k_opt_off", "<f4"), ("k_off", "<f4"), ("k_swap", "<f4"), ("k_const", "<f4"),
    ("w", "<f4"), ("gmin_idx", "<i4"), ("cmin_idx", "<i4"), ("flags", "<u4"), ("tenant", "<i4"), ("pad", "u1", (36,))])
PLAN_DTYPE = np.dtype([("log2d", "u1"), ("log2t", "u1"), ("log2p", "u1"), ("zero", "u1"), ("gc", "u1"),
                       ("off", "u1"), ("g_level", "u1"), ("disabled", "u1")])
ASSIGN_DTYPE = np.dtype([("g", "<i4"), ("c", "<i4"), ("m_bytes", "<i8"), ("plan", "<i4"), ("first_node", "<i4"),
                         ("n_nodes", "<i4"), ("thr", "<f4"), ("status", "<i4"), ("m_level", "<i4")])
REQUEST_DTYPE = np.dtype([("g_idx", "<i4"), ("c_idx", "<i4"), ("m_idx", "<i4"), ("plan", "<i4")])
SAMPLE_DTYPE = np.dtype([("plan", "<i4"), ("cores", "<i4"), ("thr", "<f8")])
FIT_NAMES = ("k_bwd", "k_sync", "k_opt", "k_opt_off", "k_off", "k_swap", "k_const")
RECONF_DTYPE = np.dtype([("T", "<f4"), ("delta", "<f4"), ("n_reconf", "<i4"), ("active", "<i4")])
NODE_DTYPE = np.dtype([("free_g", "<i4"), ("free_c", "<i4"), ("free_m", "<i8"), ("owner", "<i4"), ("reserved", "<i4")])
PLAN_WIDE_DTYPE = np.dtype([("d", "<u2"), ("t", "<u2"), ("p", "<u2"), ("zero", "u1"), ("gc", "u1"), ("off", "u1"),
                            ("g_level", "u1"), ("disabled", "u1"), ("accum", "u1")])
assert JOB_DTYPE.itemsize == 128 and PLAN_DTYPE.itemsize == 8 and PLAN_WIDE_DTYPE.itemsize == 12
assert ASSIGN_DTYPE.itemsize == 40 and NODE_DTYPE.itemsize == 24


class Env(C.Structure):
    _fields_ = [("B_intra", C.c_double), ("B_inter", C.c_double), ("B_pcie", C.c_double),
                ("gpu_mem_bytes", C.c_int64), ("mem_per_node_bytes", C.c_int64), ("gpus_per_node", C.c_int32),
                ("cpus_per_node", C.c_int32), ("bytes_per_elem", C.c_int32), ("strict_zero_dp_only", C.c_int32),
                ("zero3_extra_volume", C.c_int32), ("reserved", C.c_int32)]


class Grid(C.Structure):
    _fields_ = [("nG", C.c_int32), ("nC", C.c_int32), ("nM", C.c_int32), ("reserved", C.c_int32),
                ("g_levels", C.POINTER(C.c_int32)), ("c_levels", C.POINTER(C.c_int32)),
                ("m_levels_bytes", C.POINTER(C.c_int64))]


class SpreadClass(C.Structure):
    _fields_ = [("d_curve_val", C.c_void_p), ("d_curve_plan", C.c_void_p), ("d_curve_g", C.c_void_p), ("d_feas", C.c_void_p),
                ("align", C.c_int32), ("reserved", C.c_int32)]


MAX_PIECES = 32


class Cluster(C.Structure):
    _fields_ = [("n_nodes", C.c_int32), ("n_tenants", C.c_int32), ("quota_gpus", C.POINTER(C.c_int32)),
                ("quota_cpus", C.POINTER(C.c_int32))]


def make_cluster(n_nodes, quota=None):
    """rubick_cluster for n_nodes nodes; quota = None or an [n_tenants, 2] array of (GPUs, cores).
    Returns (struct, keep-alive objects)."""
    if quota is None:
        return Cluster(int(n_nodes), 0, None, None), ()
    q = np.ascontiguousarray(quota, dtype=np.int32).reshape(-1, 2)
    qg, qc = np.ascontiguousarray(q[:, 0]), np.ascontiguousarray(q[:, 1])
    return Cluster(int(n_nodes), len(q), qg.ctypes.data_as(C.POINTER(C.c_int32)), qc.ctypes.data_as(C.POINTER(C.c_int32))), (qg, qc)


EXPORTS = ["rubick_create", "rubick_destroy", "rubick_sync", "rubick_last_error", "rubick_enumerate_plans",
           "rubick_set_space", "rubick_enumerate_plans_wide", "rubick_set_space_wide", "rubick_eval_candidates", "rubick_best_plan", "rubick_curves", "rubick_marginal_gain",
           "rubick_min_resources", "rubick_fit_models",
           "rubick_greedy_round", "rubick_incremental_round", "rubick_greedy_round_noalloc", "rubick_schedule_round",
           "rubick_schedule_round_host", "rubick_incremental_event_host", "rubick_probe", "rubick_kernel_launches",
           "rubick_set_placement", "rubick_greedy_round_spread"]

_lib = None


class RubickError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__(f"librubick error {code}: {msg}")
        self.code = code


def lib():
    """The loaded shared library.  Raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_2408_08586_b200.build` "
                              "(nvcc, sm_100a); this package has no CPU or PyTorch fallback")
        L = C.CDLL(LIB_PATH)
        vp, ip = C.c_void_p, C.c_int
        L.rubick_create.argtypes = [C.POINTER(vp), C.POINTER(Env), ip, vp]
        L.rubick_destroy.argtypes = [vp]
        L.rubick_destroy.restype = None
        L.rubick_sync.argtypes = [vp]
        L.rubick_last_error.argtypes = [vp]
        L.rubick_last_error.restype = C.c_char_p
        L.rubick_enumerate_plans.argtypes = [vp, ip, vp, ip, C.POINTER(ip), vp]
        L.rubick_set_space.argtypes = [vp, vp, ip, C.POINTER(Grid)]
        L.rubick_enumerate_plans_wide.argtypes = [vp, ip, ip, vp, ip, C.POINTER(ip), vp]
        L.rubick_set_space_wide.argtypes = [vp, vp, ip, C.POINTER(Grid)]
        L.rubick_eval_candidates.argtypes = [vp, vp, ip, vp, vp]
        L.rubick_best_plan.argtypes = [vp, vp, vp, ip, C.c_uint, vp, vp, vp]
        L.rubick_curves.argtypes = [vp, vp, ip, C.c_uint, vp, vp, vp, vp]
        L.rubick_marginal_gain.argtypes = [vp, vp, ip, vp, vp, vp, vp, vp, vp]
        L.rubick_min_resources.argtypes = [vp, vp, vp, vp, ip, vp, vp, vp, vp]
        L.rubick_fit_models.argtypes = [vp, vp, ip, vp, ip, ip, vp, vp]
        L.rubick_greedy_round.argtypes = [vp, vp, ip, vp, vp, vp, vp, C.POINTER(Cluster), ip, vp, vp, vp, C.POINTER(C.c_int32)]
        L.rubick_incremental_round.argtypes = [vp, vp, ip, vp, vp, vp, vp, C.POINTER(Cluster), vp, vp, vp, C.c_float, ip, vp, vp, vp,
                                               C.POINTER(C.c_int32)]
        L.rubick_greedy_round_noalloc.argtypes = [vp, vp, ip, vp, vp, vp, vp, C.POINTER(Cluster), ip, vp, vp, C.POINTER(C.c_int32)]
        L.rubick_schedule_round.argtypes = [vp, vp, ip, C.POINTER(Cluster), ip, vp, vp, C.POINTER(C.c_int32)]
        L.rubick_schedule_round_host.argtypes = [vp, vp, ip, C.POINTER(Cluster), ip, vp, vp, C.POINTER(C.c_int32)]
        L.rubick_incremental_event_host.argtypes = [vp, vp, ip, C.POINTER(Cluster), vp, ip, vp, C.c_float, ip, ip, vp, vp,
                                                    C.POINTER(C.c_int32)]
        L.rubick_set_placement.argtypes = [vp, ip]
        L.rubick_greedy_round_spread.argtypes = [vp, vp, ip, vp, vp, vp, vp, C.POINTER(SpreadClass), ip, C.POINTER(Cluster), ip, vp, vp, vp,
                                                 vp, vp, C.POINTER(C.c_int32)]
        L.rubick_probe.argtypes = [vp, ip, vp, C.c_size_t, ip, C.POINTER(C.c_double)]
        L.rubick_kernel_launches.argtypes = []
        L.rubick_kernel_launches.restype = C.c_ulonglong
        for name in EXPORTS:
            if name not in ("rubick_destroy", "rubick_last_error", "rubick_kernel_launches"):
                getattr(L, name).restype = ip
        _lib = L
    return _lib


def _ptr(x):
    """Address of a torch tensor, a numpy array or None."""
    if x is None:
        return None
    if hasattr(x, "data_ptr"):
        return C.c_void_p(x.data_ptr())
    return C.c_void_p(x.ctypes.data)


def enumerate_plans(g_levels):
    """rubick_enumerate_plans -> (plans as PLAN_DTYPE array, group offsets [nG + 1] int32)."""
    gl = np.ascontiguousarray(g_levels, dtype=np.int32)
    n = C.c_int(0)
    off = np.zeros(len(gl) + 1, dtype=np.int32)
    rc = lib().rubick_enumerate_plans(_ptr(gl), len(gl), None, 0, C.byref(n), _ptr(off))
    if rc:
        raise RubickError(rc, "rubick_enumerate_plans")
    plans = np.zeros(max(n.value, 1), dtype=PLAN_DTYPE)
    rc = lib().rubick_enumerate_plans(_ptr(gl), len(gl), _ptr(plans), n.value, C.byref(n), _ptr(off))
    if rc:
        raise RubickError(rc, "rubick_enumerate_plans")
    return plans[:n.value], off


def enumerate_plans_wide(g_levels, accumulation_levels=1):
    """rubick_enumerate_plans_wide -> (plans as PLAN_WIDE_DTYPE array, group offsets [nG + 1] int32)."""
    gl = np.ascontiguousarray(g_levels, dtype=np.int32)
    n = C.c_int(0)
    off = np.zeros(len(gl) + 1, dtype=np.int32)
    rc = lib().rubick_enumerate_plans_wide(_ptr(gl), len(gl), int(accumulation_levels), None, 0, C.byref(n), _ptr(off))
    if rc:
        raise RubickError(rc, "rubick_enumerate_plans_wide")
    plans = np.zeros(max(n.value, 1), dtype=PLAN_WIDE_DTYPE)
    rc = lib().rubick_enumerate_plans_wide(_ptr(gl), len(gl), int(accumulation_levels), _ptr(plans), n.value, C.byref(n), _ptr(off))
    if rc:
        raise RubickError(rc, "rubick_enumerate_plans_wide")
    return plans[:n.value], off


def pack_jobs(jobs):
    """dict of per-job arrays -> contiguous JOB_DTYPE records (the 128-byte rubick_job layout)."""
    J = len(np.atleast_1d(jobs["P"]))
    rec = np.zeros(J, dtype=JOB_DTYPE)
    for name in JOB_DTYPE.names:
        if name in ("flags", "pad") or (name == "tenant" and name not in jobs):
            continue
        rec[name] = np.asarray(jobs[name])
    return rec


def to_device(arr, device="cuda:0"):
    """numpy array (any dtype, also structured) -> torch uint8 CUDA tensor with the same bytes."""
    import torch
    flat = np.ascontiguousarray(arr).reshape(-1).view(np.uint8)
    return torch.from_numpy(flat.copy()).to(device)


def from_device(t, dtype, shape=None):
    """torch tensor (any dtype) -> numpy array of `dtype` over the same bytes."""
    a = t.detach().cpu().contiguous().view(-1).numpy().view(np.uint8).view(dtype)
    return a.reshape(shape) if shape is not None else a


PROBE_WRITE, PROBE_READ, PROBE_FMA, PROBE_XU = 0, 1, 2, 3


def kernel_launches():
    """rubick_kernel_launches: kernels the library has launched in this process so far."""
    return int(lib().rubick_kernel_launches())


class Context:
    """Owns one rubick_ctx.  Methods carry the names of the C entry points they call."""

    def probe(self, kind, d_buf, iters=1):
        """rubick_probe: one launch of a machine probe on the context's stream -> the work it does
        (bytes for the two streams, operations for the register probes)."""
        work = C.c_double(0.0)
        self._check(lib().rubick_probe(self._h, int(kind), _ptr(d_buf), int(d_buf.numel() * d_buf.element_size()), int(iters),
                                       C.byref(work)))
        return work.value

    def __init__(self, env, device=0, stream=None):
        e = Env(float(env["B_intra"]), float(env["B_inter"]), float(env["B_pcie"]), int(env["gpu_mem_bytes"]),
                int(env["mem_per_node_bytes"]), int(env["gpus_per_node"]), int(env["cpus_per_node"]),
                int(env["bytes_per_elem"]), int(env.get("strict_zero_dp_only", 0)),
                int(env.get("zero3_extra_volume", 0)), 0)
        self._h = C.c_void_p()
        self.device = device
        rc = lib().rubick_create(C.byref(self._h), C.byref(e), int(device), C.c_void_p(stream) if stream else None)
        if rc:
            self._h = C.c_void_p()
            raise RubickError(rc, "rubick_create failed (no CUDA device, or invalid environment)")
        self.P = self.nG = self.nC = self.nM = 0

    def close(self):
        if self._h:
            lib().rubick_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, rc, allow=()):
        if rc and rc not in allow:
            raise RubickError(rc, lib().rubick_last_error(self._h).decode())
        return rc

    def last_error(self):
        return lib().rubick_last_error(self._h).decode()

    def sync(self):
        return self._check(lib().rubick_sync(self._h))

    def set_space(self, plans, g_levels, c_levels, m_levels):
        """rubick_set_space, or rubick_set_space_wide when `plans` has PLAN_WIDE_DTYPE."""
        wide = getattr(plans, "dtype", None) == PLAN_WIDE_DTYPE
        plans = np.ascontiguousarray(plans, dtype=PLAN_WIDE_DTYPE if wide else PLAN_DTYPE)
        gl = np.ascontiguousarray(g_levels, dtype=np.int32)
        cl = np.ascontiguousarray(c_levels, dtype=np.int32)
        ml = np.ascontiguousarray(m_levels, dtype=np.int64)
        grid = Grid(len(gl), len(cl), len(ml), 0, gl.ctypes.data_as(C.POINTER(C.c_int32)),
                    cl.ctypes.data_as(C.POINTER(C.c_int32)), ml.ctypes.data_as(C.POINTER(C.c_int64)))
        fn = lib().rubick_set_space_wide if wide else lib().rubick_set_space
        self._check(fn(self._h, _ptr(plans), len(plans), C.byref(grid)))
        self.P, self.nG, self.nC, self.nM = len(plans), len(gl), len(cl), len(ml)

    def eval_candidates(self, d_jobs, J, d_thr, d_feas):
        return self._check(lib().rubick_eval_candidates(self._h, _ptr(d_jobs), int(J), _ptr(d_thr), _ptr(d_feas)))

    def best_plan(self, d_thr, d_feas, J, d_best_val, d_best_plan, d_best_g, flags=0):
        return self._check(lib().rubick_best_plan(self._h, _ptr(d_thr), _ptr(d_feas), int(J), int(flags),
                                                  _ptr(d_best_val), _ptr(d_best_plan), _ptr(d_best_g)))

    def curves(self, d_jobs, J, d_feas, d_best_val, d_best_plan, d_best_g, flags=0):
        return self._check(lib().rubick_curves(self._h, _ptr(d_jobs), int(J), int(flags), _ptr(d_feas), _ptr(d_best_val),
                                               _ptr(d_best_plan), _ptr(d_best_g)))

    def marginal_gain(self, d_jobs, J, d_curve_val, d_state, d_gain_gpu, d_gain_cpu, d_next_g, d_next_c):
        return self._check(lib().rubick_marginal_gain(self._h, _ptr(d_jobs), int(J), _ptr(d_curve_val), _ptr(d_state),
                                                      _ptr(d_gain_gpu), _ptr(d_gain_cpu), _ptr(d_next_g), _ptr(d_next_c)))

    def min_resources(self, d_thr, d_feas, d_curve_val, J, d_req, d_gmin_idx, d_cmin_idx, d_baseline):
        return self._check(lib().rubick_min_resources(self._h, _ptr(d_thr), _ptr(d_feas), _ptr(d_curve_val), int(J), _ptr(d_req),
                                                      _ptr(d_gmin_idx), _ptr(d_cmin_idx), _ptr(d_baseline)))

    def fit_models(self, d_jobs, J, d_samples, S, sweeps, d_theta, d_rmsle):
        return self._check(lib().rubick_fit_models(self._h, _ptr(d_jobs), int(J), _ptr(d_samples), int(S), int(sweeps),
                                                   _ptr(d_theta), _ptr(d_rmsle)))

    def greedy_round(self, d_jobs, J, d_curve_val, d_curve_plan, d_curve_g, d_feas, n_nodes, max_steps, d_out,
                     d_node_out=None, d_step_log=None, quota=None):
        """-> (steps, capped); quota: None or [n_tenants, 2] (GPUs, cores)"""
        steps = C.c_int32(0)
        cl, _keep = make_cluster(n_nodes, quota)
        rc = self._check(lib().rubick_greedy_round(self._h, _ptr(d_jobs), int(J), _ptr(d_curve_val), _ptr(d_curve_plan),
                                                   _ptr(d_curve_g), _ptr(d_feas), C.byref(cl), int(max_steps), _ptr(d_out),
                                                   _ptr(d_node_out), _ptr(d_step_log), C.byref(steps)), allow=(ESTEPS,))
        return steps.value, rc == ESTEPS

    def incremental_round(self, d_jobs, J, d_curve_val, d_curve_plan, d_curve_g, d_feas, n_nodes, max_steps, d_out,
                          d_node_out=None, d_step_log=None, d_prev=None, d_prev_nodes=None, d_reconf=None, theta=0.97,
                          quota=None):
        """rubick_incremental_round -> (steps, capped); d_prev / d_prev_nodes: the previous round's
        outputs (None: empty cluster); d_reconf: RECONF_DTYPE records (None: gate open)."""
        steps = C.c_int32(0)
        cl, _keep = make_cluster(n_nodes, quota)
        rc = self._check(lib().rubick_incremental_round(self._h, _ptr(d_jobs), int(J), _ptr(d_curve_val), _ptr(d_curve_plan),
                                                        _ptr(d_curve_g), _ptr(d_feas), C.byref(cl), _ptr(d_prev),
                                                        _ptr(d_prev_nodes), _ptr(d_reconf), C.c_float(theta), int(max_steps),
                                                        _ptr(d_out), _ptr(d_node_out), _ptr(d_step_log), C.byref(steps)),
                         allow=(ESTEPS,))
        return steps.value, rc == ESTEPS

    def greedy_round_noalloc(self, d_jobs, J, d_curve_val, d_curve_plan, d_curve_g, d_feas, n_nodes, max_steps, d_out,
                             d_node_out=None):
        """rubick_greedy_round_noalloc: the round with its job state in the library's fixed array,
        for callers that may not allocate device memory; at most NOALLOC_MAX_JOBS jobs.
        -> (steps, capped)"""
        steps = C.c_int32(0)
        cl, _keep = make_cluster(n_nodes)
        rc = self._check(lib().rubick_greedy_round_noalloc(self._h, _ptr(d_jobs), int(J), _ptr(d_curve_val),
                                                           _ptr(d_curve_plan), _ptr(d_curve_g), _ptr(d_feas), C.byref(cl),
                                                           int(max_steps), _ptr(d_out), _ptr(d_node_out), C.byref(steps)),
                         allow=(ESTEPS,))
        return steps.value, rc == ESTEPS

    def set_placement(self, align):
        """rubick_set_placement: 0 = packed, a > 0 = spread over several nodes in pieces of a GPUs."""
        return self._check(lib().rubick_set_placement(self._h, int(align)))

    def greedy_round_spread(self, d_jobs, J, d_curve_val, d_curve_plan, d_curve_g, d_feas, classes, n_nodes, max_steps, d_out,
                            d_pieces, d_class, d_node_out=None, d_step_log=None):
        """rubick_greedy_round_spread.  classes: list of (align, d_curve_val, d_curve_plan, d_curve_g, d_feas) device tensors,
        widest pieces first.  -> (steps, capped)"""
        steps = C.c_int32(0)
        cl, _keep = make_cluster(n_nodes)
        arr = (SpreadClass * max(len(classes), 1))()
        for i, (a, v, p, g, f) in enumerate(classes):
            arr[i] = SpreadClass(_ptr(v), _ptr(p), _ptr(g), _ptr(f), int(a), 0)
        rc = self._check(lib().rubick_greedy_round_spread(self._h, _ptr(d_jobs), int(J), _ptr(d_curve_val), _ptr(d_curve_plan),
                                                          _ptr(d_curve_g), _ptr(d_feas), arr if classes else None, len(classes), C.byref(cl),
                                                          int(max_steps), _ptr(d_out), _ptr(d_node_out), _ptr(d_step_log), _ptr(d_pieces),
                                                          _ptr(d_class), C.byref(steps)), allow=(ESTEPS,))
        return steps.value, rc == ESTEPS

    def schedule_round(self, d_jobs, J, n_nodes, max_steps, d_out, d_node_out=None, quota=None):
        steps = C.c_int32(0)
        cl, _keep = make_cluster(n_nodes, quota)
        rc = self._check(lib().rubick_schedule_round(self._h, _ptr(d_jobs), int(J), C.byref(cl), int(max_steps), _ptr(d_out),
                                                     _ptr(d_node_out), C.byref(steps)), allow=(ESTEPS,))
        return steps.value, rc == ESTEPS

    def schedule_round_host(self, h_jobs, J, n_nodes, max_steps, h_out, h_node_out=None, quota=None):
        """h_jobs: JOB_DTYPE array (or pinned torch uint8 tensor); h_out: ASSIGN_DTYPE array / tensor."""
        steps = C.c_int32(0)
        cl, _keep = make_cluster(n_nodes, quota)
        rc = self._check(lib().rubick_schedule_round_host(self._h, _ptr(h_jobs), int(J), C.byref(cl), int(max_steps),
                                                          _ptr(h_out), _ptr(h_node_out), C.byref(steps)), allow=(ESTEPS,))
        return steps.value, rc == ESTEPS

    def incremental_event_host(self, h_jobs, J, n_nodes, h_out, changed=None, h_reconf=None, theta=0.97, restart=False,
                               max_steps=1 << 30, h_node_out=None, quota=None):
        """rubick_incremental_event_host -> (steps, capped).  changed: slot indices whose records are new
        (None: all); h_reconf: RECONF_DTYPE array (None: all active, gate open)."""
        steps = C.c_int32(0)
        cl, _keep = make_cluster(n_nodes, quota)
        if changed is None:
            ch, n_ch = None, -1
        else:
            ch = np.ascontiguousarray(changed, dtype=np.int32)
            n_ch = len(ch)
        rc = self._check(lib().rubick_incremental_event_host(self._h, _ptr(h_jobs), int(J), C.byref(cl), _ptr(ch) if n_ch > 0 else None,
                                                             n_ch, _ptr(h_reconf), C.c_float(theta), int(bool(restart)),
                                                             int(min(max_steps, 0x7fffffff)), _ptr(h_out), _ptr(h_node_out),
                                                             C.byref(steps)), allow=(ESTEPS,))
        return steps.value, rc == ESTEPS
