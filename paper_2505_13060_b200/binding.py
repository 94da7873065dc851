"""Thin ctypes binding of the C-ABI library (``include/ampq.h``).

Argument marshalling only: every step of the scoring path runs in the CUDA
kernels of ``libampq.so``.  Tensors are passed as raw device (or host)
pointers; PyTorch is used by callers for device memory and streams.  The
library must have been built (``python -m paper_2505_13060_b200.build``);
there is no fallback of any kind, loading fails loudly if it is missing.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
# AMPQ_LIBRARY names another build of the same library (a debug or tuning build)
LIB_PATH = os.environ.get("AMPQ_LIBRARY") or os.path.join(_HERE, "libampq.so")

F32, BF16 = 0, 1
FMT_BASE, FMT_E4M3, FMT_E5M2 = 0, 1, 2
LINEAR, BGEMM = 0, 1
D_MODEL, D_MEASURED = 0, 1
MEM_DEVICE, MEM_HOST = 0, 1
SCALE_AMAX, SCALE_POW2 = 0, 1

OK = 0
ERR_INVALID, ERR_ALIGN, ERR_STATE, ERR_CUDA = -1, -2, -3, -4
ERR_NONFINITE, ERR_INFEASIBLE, ERR_TOO_LARGE, ERR_NOMEM, ERR_TIMEOUT = -5, -6, -7, -8, -9

# every symbol include/ampq.h declares
EXPORTS = [
    "ampq_strerror", "ampq_last_error", "ampq_create", "ampq_destroy", "ampq_set_formats",
    "ampq_register_layer", "ampq_bind_operand", "ampq_set_amax", "ampq_score",
    "ampq_last_launch_count", "ampq_set_timing", "ampq_get_timing", "ampq_get_layer", "ampq_get_operand", "ampq_export_codes",
    "ampq_define_group", "ampq_clear_groups", "ampq_group_costs", "ampq_budget_from_tau",
    "ampq_all_lowp_cost", "ampq_select", "ampq_select_tables", "ampq_score_segment_noalloc",
    "ampq_group_costs_table", "ampq_stream_begin", "ampq_stream_sample", "ampq_stream_end", "ampq_fake_quant",
    "ampq_partition", "ampq_gain_table", "ampq_select_in_order",
    "ampq_set_scale_mode", "ampq_measure_amax", "ampq_get_amax", "ampq_set_causal", "ampq_set_measured",
    "ampq_set_sharing", "ampq_get_pass_bytes", "ampq_merge_sample_tables", "ampq_get_layer_table", "ampq_last_tile_shift",
]
NOALLOC_MAX_NUMEL = 2147483648

_lib = None


class AmpqError(RuntimeError):
    def __init__(self, status: int, detail: str = ""):
        self.status = status
        msg = lib().ampq_strerror(status).decode()
        super().__init__("ampq status %d (%s)%s" % (status, msg, (": " + detail) if detail else ""))


def lib():
    """Loads ``libampq.so`` (once).  Raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(
            "%s is missing: build it with `python -m paper_2505_13060_b200.build` "
            "(nvcc, sm_100a); there is no fallback path" % LIB_PATH)
    L = C.CDLL(LIB_PATH)
    vp, i, ll, dp, fp, ip = C.c_void_p, C.c_int, C.c_longlong, C.POINTER(C.c_double), C.POINTER(C.c_float), C.POINTER(C.c_int)
    L.ampq_strerror.restype = C.c_char_p
    L.ampq_strerror.argtypes = [i]
    L.ampq_last_error.restype = C.c_char_p
    L.ampq_last_error.argtypes = [vp]
    L.ampq_create.argtypes = [C.POINTER(vp), i, vp]
    L.ampq_destroy.argtypes = [vp]
    L.ampq_set_formats.argtypes = [vp, ip, i]
    L.ampq_register_layer.argtypes = [vp, i, C.c_char_p, i, ip]
    L.ampq_bind_operand.argtypes = [vp, i, i, i, i, vp, ll, i, vp, ll]
    L.ampq_set_amax.argtypes = [vp, i, i, C.c_float]
    L.ampq_score.argtypes = [vp]
    L.ampq_last_launch_count.argtypes = [vp]
    L.ampq_last_tile_shift.argtypes = [vp]
    L.ampq_set_timing.argtypes = [vp, i]
    L.ampq_get_timing.argtypes = [vp, fp]
    L.ampq_get_layer.argtypes = [vp, i, vp, vp, vp, vp, vp, vp, vp, vp]
    L.ampq_get_operand.argtypes = [vp, i, i, vp]
    L.ampq_get_layer_table.argtypes = [vp, vp, i, vp]
    L.ampq_export_codes.argtypes = [vp, i, i, i, vp]
    L.ampq_define_group.argtypes = [vp, vp, i, vp, vp, i, ip]
    L.ampq_clear_groups.argtypes = [vp]
    L.ampq_group_costs.argtypes = [vp, i, i, vp]
    L.ampq_stream_begin.argtypes = [vp]
    L.ampq_stream_sample.argtypes = [vp, i, i, i, i, vp, vp, ll]
    L.ampq_stream_end.argtypes = [vp]
    L.ampq_fake_quant.argtypes = [vp, i, i, vp, ll, C.c_float, vp]
    L.ampq_set_causal.argtypes = [vp, i, i, ll]
    L.ampq_set_measured.argtypes = [vp, i]
    L.ampq_set_sharing.argtypes = [vp, i]
    L.ampq_get_pass_bytes.argtypes = [vp, vp]
    L.ampq_set_scale_mode.argtypes = [vp, i]
    L.ampq_measure_amax.argtypes = [vp]
    L.ampq_get_amax.argtypes = [vp, i, vp]
    L.ampq_partition.argtypes = [i, i, vp, vp, vp, vp, ip]
    L.ampq_gain_table.argtypes = [i, i, vp, vp, vp, vp, vp, i, vp, i, vp]
    L.ampq_select_in_order.argtypes = [i, vp, vp, vp, C.c_double, vp, dp, dp]
    L.ampq_group_costs_table.argtypes = [vp, i, vp, i, vp, i, i, vp]
    L.ampq_merge_sample_tables.argtypes = [vp, vp, i, i, i, vp]
    L.ampq_budget_from_tau.argtypes = [C.c_double, vp, i, dp]
    L.ampq_all_lowp_cost.argtypes = [vp, i, i, dp]
    L.ampq_select.argtypes = [vp, i, C.c_double, vp, dp, dp]
    L.ampq_select_tables.argtypes = [i, vp, vp, vp, vp, C.c_double, vp, dp, dp]
    L.ampq_score_segment_noalloc.argtypes = [i, vp, i, i, vp, vp, ll, C.c_float, vp]
    for name in EXPORTS:
        if name not in ("ampq_strerror", "ampq_last_error"):
            getattr(L, name).restype = i
    _lib = L
    return L


def _np_ptr(a: np.ndarray):
    return a.ctypes.data_as(C.c_void_p)


def budget_from_tau(tau: float, losses) -> float:
    g = np.ascontiguousarray(losses, dtype=np.float64)
    out = C.c_double()
    rc = lib().ampq_budget_from_tau(tau, _np_ptr(g), g.size, C.byref(out))
    if rc:
        raise AmpqError(rc)
    return out.value


GAIN_MAC, GAIN_MEMORY = 0, 1


def partition(n: int, edges, quantisable):
    """Sequential sub-graphs of a model DAG (Algorithm 2).  Returns (group_of[n], J)."""
    e = np.ascontiguousarray(np.asarray(edges, dtype=np.int32).reshape(-1, 2))
    src, dst = np.ascontiguousarray(e[:, 0]), np.ascontiguousarray(e[:, 1])
    q = np.ascontiguousarray(quantisable, dtype=np.uint8)
    out = np.zeros(n, dtype=np.int32)
    J = C.c_int()
    rc = lib().ampq_partition(n, len(e), _np_ptr(src), _np_ptr(dst), _np_ptr(q), _np_ptr(out), C.byref(J))
    if rc:
        raise AmpqError(rc, "ampq_partition")
    return out, J.value


def gain_table(kind: int, layers, Q, delta) -> np.ndarray:
    """layers: [(layer kind, N, C, K)] of one group; Q: [Lj, Pj]; delta: [F]."""
    lk = np.ascontiguousarray([l[0] for l in layers], dtype=np.int32)
    N, Cc, K = (np.ascontiguousarray([l[k] for l in layers], dtype=np.int64) for k in (1, 2, 3))
    Q = np.asarray(Q, dtype=np.uint8)
    Lj, Pj = Q.shape
    Qf = np.ascontiguousarray(Q.T).reshape(-1)
    dl = np.ascontiguousarray(delta, dtype=np.float64)
    out = np.zeros(Pj)
    rc = lib().ampq_gain_table(kind, Lj, _np_ptr(lk), _np_ptr(N), _np_ptr(Cc), _np_ptr(K), _np_ptr(Qf), Pj,
                               _np_ptr(dl), dl.size, _np_ptr(out))
    if rc:
        raise AmpqError(rc, "ampq_gain_table")
    return out


def select_in_order(order, d_low, c_low, budget: float):
    """Prefix / Random baselines: returns (chosen[L], c_total, d_total)."""
    o = np.ascontiguousarray(order, dtype=np.int32)
    d = np.ascontiguousarray(d_low, dtype=np.float64)
    c = np.ascontiguousarray(c_low, dtype=np.float64)
    ch = np.zeros(max(o.size, 1), dtype=np.uint8)
    co, do = C.c_double(), C.c_double()
    rc = lib().ampq_select_in_order(o.size, _np_ptr(o), _np_ptr(d), _np_ptr(c), budget, _np_ptr(ch), C.byref(co),
                                    C.byref(do))
    if rc:
        raise AmpqError(rc, "ampq_select_in_order")
    return ch[:o.size].copy(), co.value, do.value


def group_costs_table(layer_ids, Q, d_layer) -> np.ndarray:
    """d_{j,p} of one group from a per-layer table d_layer[L, F]; Q: [Lj, Pj]."""
    ids = np.ascontiguousarray(layer_ids, dtype=np.int32)
    Q = np.asarray(Q, dtype=np.uint8)
    Lj, Pj = Q.shape
    Qf = np.ascontiguousarray(Q.T).reshape(-1)  # Q[l + Lj*p]
    d_layer = np.ascontiguousarray(d_layer, dtype=np.float64)
    out = np.zeros(Pj)
    rc = lib().ampq_group_costs_table(_np_ptr(ids), Lj, _np_ptr(Qf), Pj, _np_ptr(d_layer), d_layer.shape[0],
                                      d_layer.shape[1], _np_ptr(out))
    if rc:
        raise AmpqError(rc, "ampq_group_costs_table")
    return out


def merge_sample_tables(tables, R_local) -> np.ndarray:
    """tables: [nranks, L, K] per-process tables of per-layer means over each
    process's own samples; R_local: [nranks] sample counts.  Returns the [L, K]
    table over all samples."""
    t = np.ascontiguousarray(tables, dtype=np.float64)
    R = np.ascontiguousarray(R_local, dtype=np.int32)
    assert t.ndim == 3 and R.size == t.shape[0]
    out = np.zeros(t.shape[1:])
    rc = lib().ampq_merge_sample_tables(_np_ptr(t), _np_ptr(R), t.shape[0], t.shape[1], t.shape[2], _np_ptr(out))
    if rc:
        raise AmpqError(rc, "ampq_merge_sample_tables")
    return out


def select_tables(c_tables, d_tables, budget: float):
    """Solves the integer program on explicit tables; returns (p, c, d) or None if infeasible."""
    P = np.asarray([len(x) for x in c_tables], dtype=np.int32)
    J = len(P)
    off = np.zeros(max(J, 1), dtype=np.int64)
    if J:
        off[1:J] = np.cumsum(P[:-1])
    c = np.concatenate([np.asarray(x, np.float64) for x in c_tables]) if J else np.zeros(1)
    d = np.concatenate([np.asarray(x, np.float64) for x in d_tables]) if J else np.zeros(1)
    p = np.zeros(max(J, 1), dtype=np.int32)
    co, do = C.c_double(), C.c_double()
    rc = lib().ampq_select_tables(J, _np_ptr(P) if J else None, _np_ptr(off), _np_ptr(c), _np_ptr(d),
                                  budget, _np_ptr(p), C.byref(co), C.byref(do))
    if rc == ERR_INFEASIBLE:
        return None
    if rc:
        raise AmpqError(rc)
    return p[:J].copy(), co.value, do.value


def score_segment_noalloc(device: int, stream: int, dtype: int, fmt: int, values_ptr: int, grads_ptr: int,
                          numel: int, amax: float, dev_out_ptr: int):
    """``ampq_score_segment_noalloc``: the pass over one segment for callers that
    must not allocate device memory (the library's own fixed device array holds
    the tables and partial sums).  ``dev_out_ptr`` receives {S, D, amax} as three
    doubles on the device; asynchronous on ``stream``."""
    rc = lib().ampq_score_segment_noalloc(device, C.c_void_p(stream), dtype, fmt, C.c_void_p(values_ptr),
                                          C.c_void_p(grads_ptr), numel, amax, C.c_void_p(dev_out_ptr))
    if rc == ERR_TOO_LARGE:
        raise AmpqError(rc, "numel %d exceeds the fixed scratch of the no-allocation call (at most %d elements)"
                        % (numel, NOALLOC_MAX_NUMEL))
    if rc:
        raise AmpqError(rc, "ampq_score_segment_noalloc")


class Context:
    """One scoring context on one CUDA device and stream (see ``ampq_create``)."""

    def __init__(self, device: int = 0, stream: int = 0):
        self._h = C.c_void_p()
        rc = lib().ampq_create(C.byref(self._h), device, C.c_void_p(stream))
        if rc:
            self._h = None
            raise AmpqError(rc, "ampq_create")
        self.F = 2
        self._R = {}
        self.device, self.stream = device, stream   # the cudaStream_t handle every call of this context runs on

    def _check(self, rc: int):
        if rc:
            raise AmpqError(rc, lib().ampq_last_error(self._h).decode())

    def destroy(self):
        if self._h is not None:
            lib().ampq_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    def set_formats(self, fmts):
        a = (C.c_int * len(fmts))(*fmts)
        self._check(lib().ampq_set_formats(self._h, a, len(fmts)))
        self.F = len(fmts)

    def register_layer(self, kind: int, name: str, R: int) -> int:
        out = C.c_int()
        self._check(lib().ampq_register_layer(self._h, kind, name.encode() if name else None, R, C.byref(out)))
        self._R[out.value] = R
        return out.value

    def bind_operand(self, layer_id: int, operand: int, dtype: int, values_ptr: int, numel: int,
                     per_sample_values: bool, grads_ptr: int, grad_stride: int, mem: int = MEM_DEVICE):
        self._check(lib().ampq_bind_operand(self._h, layer_id, operand, dtype, mem, C.c_void_p(values_ptr),
                                            numel, 1 if per_sample_values else 0, C.c_void_p(grads_ptr),
                                            grad_stride))

    def set_amax(self, layer_id: int, operand: int, amax: float):
        self._check(lib().ampq_set_amax(self._h, layer_id, operand, amax))

    def set_causal(self, layer_id: int, operand: int, T: int):
        self._check(lib().ampq_set_causal(self._h, layer_id, operand, T))

    def set_measured(self, on: bool):
        self._check(lib().ampq_set_measured(self._h, 1 if on else 0))

    def set_sharing(self, on: bool):
        self._check(lib().ampq_set_sharing(self._h, 1 if on else 0))

    def set_scale_mode(self, mode: int):
        self._check(lib().ampq_set_scale_mode(self._h, mode))

    def measure_amax(self):
        self._check(lib().ampq_measure_amax(self._h))

    def get_amax(self, layer_id: int) -> np.ndarray:
        out = np.zeros(2, np.float32)
        self._check(lib().ampq_get_amax(self._h, layer_id, _np_ptr(out)))
        return out

    def score(self):
        self._check(lib().ampq_score(self._h))

    def stream_begin(self):
        self._check(lib().ampq_stream_begin(self._h))

    def stream_sample(self, layer_id: int, operand: int, r: int, dtype: int, values_ptr: int, grads_ptr: int,
                      numel: int):
        self._check(lib().ampq_stream_sample(self._h, layer_id, operand, r, dtype, C.c_void_p(values_ptr),
                                             C.c_void_p(grads_ptr), numel))

    def stream_end(self):
        self._check(lib().ampq_stream_end(self._h))

    def fake_quant(self, dtype: int, fmt: int, values_ptr: int, numel: int, amax: float, out_ptr: int):
        self._check(lib().ampq_fake_quant(self._h, dtype, fmt, C.c_void_p(values_ptr), numel, amax,
                                          C.c_void_p(out_ptr)))

    def last_launch_count(self) -> int:
        return lib().ampq_last_launch_count(self._h)

    def last_tile_shift(self) -> int:
        return lib().ampq_last_tile_shift(self._h)

    def get_pass_bytes(self) -> dict:
        """Bytes of bound tensors the last pass reads: amax pass, scoring pass."""
        b = (C.c_longlong * 2)()
        self._check(lib().ampq_get_pass_bytes(self._h, b))
        return dict(amax=int(b[0]), score=int(b[1]))

    def set_timing(self, on: bool):
        self._check(lib().ampq_set_timing(self._h, 1 if on else 0))

    def get_timing(self) -> dict:
        """Device milliseconds of the last score: amax kernel, scoring kernel, whole call."""
        ms = (C.c_float * 3)()
        self._check(lib().ampq_get_timing(self._h, ms))
        return dict(amax_ms=ms[0], score_ms=ms[1], total_ms=ms[2])

    def get_layer(self, layer_id: int, allow_nonfinite: bool = False) -> dict:
        R, F = self._R[layer_id], self.F
        amax = np.zeros(2, np.float32)
        scale = np.zeros(2 * F, np.float32)
        inv = np.zeros(2 * F, np.float32)
        s_r = np.zeros(R)
        s_mean = np.zeros(1)
        d_meas_r = np.zeros(R * F)
        d_model = np.zeros(F)
        d_meas = np.zeros(F)
        rc = lib().ampq_get_layer(self._h, layer_id, _np_ptr(amax), _np_ptr(scale), _np_ptr(inv), _np_ptr(s_r),
                                  _np_ptr(s_mean), _np_ptr(d_meas_r), _np_ptr(d_model), _np_ptr(d_meas))
        if rc and not (allow_nonfinite and rc == ERR_NONFINITE):
            self._check(rc)
        return dict(amax=amax, scale=scale.reshape(2, F), inv_scale=inv.reshape(2, F), s_per_sample=s_r,
                    s_mean=float(s_mean[0]), d_meas_per_sample=d_meas_r.reshape(R, F), d_model=d_model,
                    d_meas=d_meas, status=rc)

    def get_layer_table(self, layer_ids) -> np.ndarray:
        """[n, 1 + 2F] rows {s_mean, d_model[F], d_meas[F]} of the given layers, one call."""
        ids = np.ascontiguousarray(layer_ids, dtype=np.int32)
        out = np.zeros((ids.size, 1 + 2 * self.F))
        self._check(lib().ampq_get_layer_table(self._h, _np_ptr(ids), ids.size, _np_ptr(out)))
        return out

    def get_operand(self, layer_id: int, operand: int) -> np.ndarray:
        out = np.zeros((self._R[layer_id], self.F))
        self._check(lib().ampq_get_operand(self._h, layer_id, operand, _np_ptr(out)))
        return out

    def export_codes(self, layer_id: int, operand: int, fmt: int, dev_out_ptr: int):
        self._check(lib().ampq_export_codes(self._h, layer_id, operand, fmt, C.c_void_p(dev_out_ptr)))

    def define_group(self, layer_ids, Q, c) -> int:
        """Q: [Lj, Pj] array of format indices (column p = configuration p); c: [Pj]."""
        ids = np.ascontiguousarray(layer_ids, dtype=np.int32)
        Q = np.asarray(Q, dtype=np.uint8)
        Lj, Pj = Q.shape
        Qf = np.ascontiguousarray(Q.T).reshape(-1)  # Q[l + Lj*p]
        cc = np.ascontiguousarray(c, dtype=np.float64)
        assert cc.size == Pj and ids.size == Lj
        out = C.c_int()
        self._check(lib().ampq_define_group(self._h, _np_ptr(ids), Lj, _np_ptr(Qf), _np_ptr(cc), Pj, C.byref(out)))
        if not hasattr(self, "_P"):
            self._P = {}
        self._P[out.value] = Pj
        return out.value

    def clear_groups(self):
        self._check(lib().ampq_clear_groups(self._h))
        self._P = {}

    def group_costs(self, group_id: int, d_mode: int = D_MODEL) -> np.ndarray:
        out = np.zeros(self._P[group_id])
        self._check(lib().ampq_group_costs(self._h, group_id, d_mode, _np_ptr(out)))
        return out

    def all_lowp_cost(self, d_mode: int, f: int) -> float:
        out = C.c_double()
        self._check(lib().ampq_all_lowp_cost(self._h, d_mode, f, C.byref(out)))
        return out.value

    def select(self, d_mode: int, budget: float):
        """Returns (p[J], c_total, d_total), or None when no assignment meets the budget."""
        J = len(getattr(self, "_P", {}))
        p = np.zeros(max(J, 1), dtype=np.int32)
        co, do = C.c_double(), C.c_double()
        rc = lib().ampq_select(self._h, d_mode, budget, _np_ptr(p), C.byref(co), C.byref(do))
        if rc == ERR_INFEASIBLE:
            return None
        self._check(rc)
        return p[:J].copy(), co.value, do.value


def torch_dtype_code(t) -> int:
    import torch

    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError("operands are float32 or bfloat16, got %s" % t.dtype)


def bind_layer_tensors(ctx: Context, layer_id: int, lt, mem: int = MEM_DEVICE):
    """Binds both operands of a ``synth.LayerTensors`` (or anything with
    ``spec``, ``values`` and ``grads`` laid out the same way)."""
    R = lt.spec.R
    for k, op in enumerate((lt.spec.op0, lt.spec.op1)):
        v, g = lt.values[k], lt.grads[k]
        assert v.is_contiguous() and g.is_contiguous()
        ext = v.numel() // R if op.per_sample else v.numel()
        ctx.bind_operand(layer_id, k, torch_dtype_code(v), v.data_ptr(), v.numel(), op.per_sample,
                         g.data_ptr(), ext, mem)
