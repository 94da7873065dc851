"""ctypes front end of the CPU oracle (``ampq_oracle.c``).

TEST INFRASTRUCTURE, NOT THE PRODUCT: only the tests, the smoke check and the
bench's CPU-baseline leg import this module.  It holds no arithmetic of its
own; every number comes out of the C file, which is written from the paper
(Sec. 2.1-2.2, Algorithm 1 steps 2 and 4) and shares nothing with the CUDA
path.  Arrays are numpy; bf16 tensors are passed as ``uint16`` bit patterns.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ampq_oracle.c")
_LIB = os.path.join(_HERE, "libampq_oracle.so")

F32, BF16 = 0, 1
FMT_BASE, FMT_E4M3, FMT_E5M2 = 0, 1, 2

_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (a second or so); returns the library path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fno-fast-math", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        build()
        L = C.CDLL(_LIB)
        L.orc_fmax.restype = C.c_double
        L.orc_fmax.argtypes = [C.c_int]
        L.orc_mantissa_bits.restype = C.c_int
        L.orc_mantissa_bits.argtypes = [C.c_int]
        L.orc_alpha.restype = C.c_double
        L.orc_alpha.argtypes = [C.c_int]
        L.orc_fp8_decode.restype = C.c_double
        L.orc_fp8_decode.argtypes = [C.c_int, C.c_uint]
        L.orc_fp8_encode.restype = C.c_uint
        L.orc_fp8_encode.argtypes = [C.c_int, C.c_float]
        L.orc_amax.restype = C.c_float
        L.orc_amax.argtypes = [C.c_int, C.c_void_p, C.c_longlong]
        L.orc_scales.restype = None
        L.orc_scales.argtypes = [C.c_int, C.c_float, C.POINTER(C.c_float), C.POINTER(C.c_float)]
        L.orc_scales_pow2.restype = None
        L.orc_scales_pow2.argtypes = [C.c_int, C.c_float, C.POINTER(C.c_float), C.POINTER(C.c_float)]
        L.orc_codes.restype = None
        L.orc_codes.argtypes = [C.c_int, C.c_void_p, C.c_longlong, C.c_int, C.c_float, C.c_void_p]
        L.orc_fake_quant.restype = None
        L.orc_fake_quant.argtypes = [C.c_int, C.c_void_p, C.c_longlong, C.c_int, C.c_float, C.c_float, C.c_void_p]
        L.orc_score_segment.restype = None
        L.orc_score_segment.argtypes = [C.c_int, C.c_void_p, C.c_void_p, C.c_longlong, C.c_int,
                                        C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.orc_layer_combine.restype = None
        L.orc_layer_combine.argtypes = [C.c_int, C.c_int] + [C.c_void_p] * 8
        L.orc_group_costs.restype = None
        L.orc_group_costs.argtypes = [C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_void_p,
                                      C.c_void_p, C.c_void_p]
        L.orc_budget_from_tau.restype = C.c_double
        L.orc_budget_from_tau.argtypes = [C.c_double, C.c_void_p, C.c_int]
        L.orc_select_bruteforce.restype = C.c_int
        L.orc_select_bruteforce.argtypes = [C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                            C.c_double, C.c_void_p, C.POINTER(C.c_double),
                                            C.POINTER(C.c_double)]
        L.orc_select_bnb.restype = C.c_int
        L.orc_select_bnb.argtypes = [C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                     C.c_double, C.c_longlong, C.c_void_p, C.POINTER(C.c_double),
                                     C.POINTER(C.c_double)]
        L.orc_select_dp_integer.restype = C.c_int
        L.orc_select_dp_integer.argtypes = [C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                            C.c_longlong, C.c_void_p, C.POINTER(C.c_double),
                                            C.POINTER(C.c_longlong)]
        _lib = L
    return _lib


def _dtype_of(a: np.ndarray) -> int:
    if a.dtype == np.float32:
        return F32
    if a.dtype == np.uint16:
        return BF16
    raise TypeError("oracle arrays are float32 or uint16 (bf16 bits), got %s" % a.dtype)


def _ptr(a: np.ndarray):
    assert a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(C.c_void_p)


# ---- format facts --------------------------------------------------------
def fmax(fmt: int) -> float:
    return lib().orc_fmax(fmt)


def mantissa_bits(fmt: int) -> int:
    return lib().orc_mantissa_bits(fmt)


def alpha(mbits: int) -> float:
    return lib().orc_alpha(mbits)


def fp8_decode(fmt: int, code: int) -> float:
    return lib().orc_fp8_decode(fmt, code)


def fp8_encode(fmt: int, y: float) -> int:
    return lib().orc_fp8_encode(fmt, C.c_float(y))


# ---- steps 1-4 -------------------------------------------------------------
def amax(values: np.ndarray) -> np.float32:
    v = np.ascontiguousarray(values).reshape(-1)
    return np.float32(lib().orc_amax(_dtype_of(v), _ptr(v), v.size))


def scales(fmt: int, amax_value, pow2: bool = False) -> tuple[np.float32, np.float32]:
    s, i = C.c_float(), C.c_float()
    fn = lib().orc_scales_pow2 if pow2 else lib().orc_scales
    fn(fmt, C.c_float(float(amax_value)), C.byref(s), C.byref(i))
    return np.float32(s.value), np.float32(i.value)


def codes(values: np.ndarray, fmt: int, inv_scale) -> np.ndarray:
    v = np.ascontiguousarray(values).reshape(-1)
    out = np.empty(v.size, dtype=np.uint8)
    lib().orc_codes(_dtype_of(v), _ptr(v), v.size, fmt, C.c_float(float(inv_scale)), _ptr(out))
    return out


def fake_quant(values: np.ndarray, fmt: int, scale, inv_scale) -> np.ndarray:
    """The quantised operand z^ = decode(q) * scale in the operand's own dtype."""
    v = np.ascontiguousarray(values).reshape(-1)
    out = np.empty_like(v)
    lib().orc_fake_quant(_dtype_of(v), _ptr(v), v.size, fmt, C.c_float(float(scale)),
                         C.c_float(float(inv_scale)), _ptr(out))
    return out.reshape(np.shape(values))


def score_segment(values: np.ndarray, grads: np.ndarray, fmts, scale_list, inv_list) -> np.ndarray:
    """[S, D_f...] of one segment (one tensor, one sample)."""
    v = np.ascontiguousarray(values).reshape(-1)
    g = np.ascontiguousarray(grads).reshape(-1)
    assert v.size == g.size and v.dtype == g.dtype
    fm = np.asarray(fmts, dtype=np.int32)
    sc = np.asarray(scale_list, dtype=np.float32)
    iv = np.asarray(inv_list, dtype=np.float32)
    out = np.zeros(1 + fm.size, dtype=np.float64)
    lib().orc_score_segment(_dtype_of(v), _ptr(v), _ptr(g), v.size, fm.size, _ptr(fm), _ptr(sc),
                            _ptr(iv), _ptr(out))
    return out


def score_operand(values: np.ndarray, grads: np.ndarray, R: int, per_sample_values: bool,
                  low_fmts, amax_preset=None, threads: int = 1, pow2: bool = False):
    """Steps 1-4 for one operand.

    values: per_sample_values -> [R, n] (sample r owns row r), else [n] shared by
    all samples (weights).  grads: [R, n].  Returns (amax, scales[nlow],
    inv_scales[nlow], seg[R, 1+nlow]).  ``threads`` only spreads independent
    segments over host threads (ctypes drops the GIL); each segment is still the
    plain sequential loop.
    """
    v = np.ascontiguousarray(values)
    g = np.ascontiguousarray(grads).reshape(R, -1)
    a = amax(v) if amax_preset is None else np.float32(amax_preset)
    sc, iv = [], []
    for f in low_fmts:
        s, i = scales(f, a, pow2)
        sc.append(s)
        iv.append(i)
    vv = v.reshape(R, -1) if per_sample_values else v.reshape(1, -1)

    def one(r):
        return score_segment(vv[r if per_sample_values else 0], g[r], low_fmts, sc, iv)

    if threads > 1 and R > 1:
        with ThreadPoolExecutor(max_workers=threads) as ex:
            seg = list(ex.map(one, range(R)))
    else:
        seg = [one(r) for r in range(R)]
    return a, np.asarray(sc, np.float32), np.asarray(iv, np.float32), np.stack(seg)


# ---- step 5 ---------------------------------------------------------------
def layer_combine(seg0: np.ndarray, seg1: np.ndarray, fmts):
    """fmts = [BASE, low...]; seg*: [R, F].  Returns dict of the layer's values."""
    seg0 = np.ascontiguousarray(seg0, dtype=np.float64)
    seg1 = np.ascontiguousarray(seg1, dtype=np.float64)
    R, F = seg0.shape
    assert len(fmts) == F and seg1.shape == seg0.shape
    mb = np.asarray([mantissa_bits(f) for f in fmts], dtype=np.int32)
    s_r = np.zeros(R)
    s_mean = np.zeros(1)
    d_meas_r = np.zeros((R, F))
    d_model = np.zeros(F)
    d_meas = np.zeros(F)
    lib().orc_layer_combine(R, F, _ptr(mb), _ptr(seg0), _ptr(seg1), _ptr(s_r), _ptr(s_mean),
                            _ptr(d_meas_r), _ptr(d_model), _ptr(d_meas))
    return dict(s_per_sample=s_r, s_mean=float(s_mean[0]), d_meas_per_sample=d_meas_r,
                d_model=d_model, d_meas=d_meas)


# ---- steps 6-7 --------------------------------------------------------------
def group_costs(layer_ids, Q: np.ndarray, d_layer: np.ndarray) -> np.ndarray:
    """Q: [Lj, Pj] (column p = one configuration); d_layer: [L, F]."""
    ids = np.asarray(layer_ids, dtype=np.int32)
    Q = np.asarray(Q, dtype=np.uint8)
    Lj, Pj = Q.shape
    Qf = np.ascontiguousarray(Q.T).reshape(-1)  # Q[l + Lj*p]
    d_layer = np.ascontiguousarray(d_layer, dtype=np.float64)
    out = np.zeros(Pj)
    lib().orc_group_costs(Lj, Pj, d_layer.shape[1], _ptr(ids), _ptr(Qf), _ptr(d_layer), _ptr(out))
    return out


def budget_from_tau(tau: float, losses) -> float:
    g = np.asarray(losses, dtype=np.float64)
    return lib().orc_budget_from_tau(tau, _ptr(g), g.size)


def _flatten(c_tables, d_tables):
    P = np.asarray([len(x) for x in c_tables], dtype=np.int32)
    off = np.zeros(len(P), dtype=np.int64)
    if len(P):
        off[1:] = np.cumsum(P[:-1])
    c = np.concatenate([np.asarray(x, dtype=np.float64) for x in c_tables]) if len(P) else np.zeros(0)
    d = np.concatenate([np.asarray(x, dtype=np.float64) for x in d_tables]) if len(P) else np.zeros(0)
    return P, off, c, d


def select_bruteforce(c_tables, d_tables, budget: float):
    """Exhaustive enumeration.  Returns (p[J], c, d) or None when infeasible."""
    P, off, c, d = _flatten(c_tables, d_tables)
    J = len(P)
    p = np.zeros(max(J, 1), dtype=np.int32)
    co, do = C.c_double(), C.c_double()
    rc = lib().orc_select_bruteforce(J, _ptr(P), _ptr(off), _ptr(c), _ptr(d), budget, _ptr(p),
                                     C.byref(co), C.byref(do))
    if rc:
        return None
    return p[:J].copy(), co.value, do.value


def select_dp_integer(c_tables, d_int_tables, budget: int):
    """The integer program with integer-valued d by the textbook dynamic
    program over the budget.  Returns (p[J], c, d) -- p is one optimal
    assignment, not necessarily the lexicographically smallest -- or None."""
    P, off, c, _ = _flatten(c_tables, d_int_tables)
    d = np.ascontiguousarray(np.concatenate([np.asarray(x) for x in d_int_tables]) if len(P) else np.zeros(1),
                             dtype=np.int64)
    J = len(P)
    p = np.zeros(max(J, 1), dtype=np.int32)
    co, do = C.c_double(), C.c_longlong()
    rc = lib().orc_select_dp_integer(J, _ptr(P), _ptr(off), _ptr(c), _ptr(d), int(budget), _ptr(p),
                                     C.byref(co), C.byref(do))
    if rc == 1:
        return None
    if rc:
        raise RuntimeError("integer budget too large for the oracle's dynamic program")
    return p[:J].copy(), co.value, int(do.value)


def select_bnb(c_tables, d_tables, budget: float, node_limit: int = 0):
    """Plain depth-first branch and bound with the same sums and ordering as the
    enumeration; slow when the budget admits many assignments."""
    P, off, c, d = _flatten(c_tables, d_tables)
    J = len(P)
    p = np.zeros(max(J, 1), dtype=np.int32)
    co, do = C.c_double(), C.c_double()
    rc = lib().orc_select_bnb(J, _ptr(P), _ptr(off), _ptr(c), _ptr(d), budget, node_limit, _ptr(p),
                              C.byref(co), C.byref(do))
    if rc == 1:
        return None
    if rc == 2:
        raise RuntimeError("oracle branch-and-bound hit its node limit")
    return p[:J].copy(), co.value, do.value
