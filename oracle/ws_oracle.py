"""ctypes front end of the CPU oracle (``ws_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
benchmark's CPU-baseline leg.  The product package never imports this module
and this module never imports the product's kernels or bindings.

Arrays are numpy; fp32 data are ``float32`` arrays, bf16 data are ``uint16``
arrays holding the raw bits.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ws_oracle.c")
_SO = os.path.join(_HERE, "libws_oracle.so")

SGDM, ADAM, LAMB, LARS, ADAFACTOR = 0, 1, 2, 3, 4
F32, BF16 = 0, 1
OPT_CODE = {"sgdm": SGDM, "adam": ADAM, "lamb": LAMB, "lars": LARS, "adafactor": ADAFACTOR}


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain C, -O2, IEEE arithmetic, OpenMP only
    for loops with independent iterations)."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
               "-o", _SO, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _SO


class Hyper(C.Structure):
    _fields_ = [("opt", C.c_int32), ("lr", C.c_double), ("beta1", C.c_double),
                ("beta2", C.c_double), ("eps", C.c_double), ("weight_decay", C.c_double),
                ("momentum", C.c_double), ("grad_scale", C.c_double), ("step", C.c_int64),
                ("trust_coeff", C.c_double), ("eps2", C.c_double), ("clip_threshold", C.c_double),
                ("decay_exponent", C.c_double)]


def make_hyper(opt, hyper: dict) -> Hyper:
    code = OPT_CODE[opt] if isinstance(opt, str) else int(opt)
    return Hyper(code, hyper["lr"], hyper["beta1"], hyper["beta2"], hyper["eps"],
                 hyper["weight_decay"], hyper["momentum"], hyper["grad_scale"],
                 int(hyper["step"]), float(hyper.get("trust_coeff", 0.001)),
                 float(hyper.get("eps2", 1e-3)), float(hyper.get("clip_threshold", 1.0)),
                 float(hyper.get("decay_exponent", 0.8)))


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        i64p, vpp = C.POINTER(C.c_int64), C.POINTER(C.c_void_p)
        L.wso_plan.restype = C.c_int64
        L.wso_plan.argtypes = [i64p, C.c_int32, C.c_int32, C.c_int32, i64p, i64p]
        L.wso_pack.restype = None
        L.wso_pack.argtypes = [vpp, i64p, i64p, i64p, C.c_int32, C.c_int32, C.c_int64,
                               C.c_int32, C.c_void_p]
        L.wso_unpack.restype = None
        L.wso_unpack.argtypes = [C.c_void_p, i64p, i64p, i64p, C.c_int32, C.c_int64,
                                 C.c_int32, vpp]
        L.wso_update_tensor.restype = None
        L.wso_update_tensor.argtypes = [C.POINTER(Hyper), C.c_int64, C.c_int32, vpp, C.c_int32,
                                        C.c_void_p, C.c_void_p, C.c_void_p,
                                        C.POINTER(C.c_double)]
        L.wso_sharded_update.restype = None
        L.wso_sharded_update.argtypes = [C.POINTER(Hyper), C.c_int32, i64p, i64p, i64p,
                                         C.c_int64, C.c_int32, C.c_int32, vpp, C.c_int32, C.c_void_p,
                                         C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32,
                                         C.POINTER(C.c_double), C.POINTER(C.c_double)]
        L.wso_lars_tensor.restype = None
        L.wso_lars_tensor.argtypes = [C.POINTER(Hyper), C.c_int64, C.c_int32, vpp, C.c_int32,
                                      C.c_void_p, C.c_void_p, C.POINTER(C.c_double)]
        L.wso_lars_sharded.restype = None
        L.wso_lars_sharded.argtypes = [C.POINTER(Hyper), C.c_int32, i64p, i64p, i64p, C.c_int64,
                                       C.c_int32, C.c_int32, vpp, C.c_int32, C.c_void_p, C.c_void_p,
                                       C.c_void_p, C.c_int32, C.POINTER(C.c_double)]
        L.wso_adafactor_tensor.restype = None
        L.wso_adafactor_tensor.argtypes = [C.POINTER(Hyper), C.c_int64, C.c_int64, C.c_int32, vpp, C.c_int32,
                                           C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(C.c_double)]
        L.wso_adafactor_sharded.restype = None
        L.wso_adafactor_sharded.argtypes = [C.POINTER(Hyper), C.c_int32, i64p, i64p, i64p, C.c_int64,
                                            C.c_int32, C.c_int32, vpp, C.c_int32, i64p, i64p, i64p,
                                            C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32,
                                            C.POINTER(C.c_double)]
        L.wso_plan_flat.restype = C.c_int64
        L.wso_plan_flat.argtypes = [i64p, C.c_int32, C.c_int32, C.c_int32, i64p]
        L.wso_sharded_update_map.restype = None
        L.wso_sharded_update_map.argtypes = [C.POINTER(Hyper), C.c_int32, C.POINTER(C.c_int32), C.c_int64,
                                             C.c_int32, C.c_int32, vpp, C.c_int32, C.c_void_p, C.c_void_p,
                                             C.c_void_p, C.c_void_p, C.c_int32, C.POINTER(C.c_double)]
        L.wso_shard_reduce.restype = None
        L.wso_shard_reduce.argtypes = [C.c_int32, i64p, i64p, i64p, C.c_int64, C.c_int32,
                                       C.c_int32, vpp, C.c_int32, C.c_double, C.c_void_p]
        dp = C.POINTER(C.c_double)
        L.wso_lamb_shard_partial.restype = None
        L.wso_lamb_shard_partial.argtypes = [C.POINTER(Hyper), C.c_int32, i64p, i64p, i64p, C.c_int32, C.c_void_p,
                                             C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, dp, dp]
        L.wso_lars_shard_partial.restype = None
        L.wso_lars_shard_partial.argtypes = [C.POINTER(Hyper), C.c_int32, i64p, i64p, i64p, C.c_int32, C.c_void_p,
                                             C.c_int32, C.c_void_p, dp, dp]
        L.wso_norm_ratio.restype = C.c_double
        L.wso_norm_ratio.argtypes = [C.POINTER(Hyper), C.c_double, C.c_double]
        L.wso_norm_shard_apply.restype = None
        L.wso_norm_shard_apply.argtypes = [C.POINTER(Hyper), C.c_int32, i64p, i64p, i64p, C.c_int64, C.c_int32, dp, dp,
                                           C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32]
        L.wso_af_shard_sums.restype = None
        L.wso_af_shard_sums.argtypes = [C.POINTER(Hyper), C.c_int32, i64p, i64p, i64p, C.c_int32, C.c_void_p, C.c_int32,
                                        C.c_void_p, i64p, i64p, i64p, dp, dp, dp]
        L.wso_af_moments.restype = None
        L.wso_af_moments.argtypes = [C.POINTER(Hyper), C.c_int32, i64p, i64p, i64p, dp, C.c_void_p, dp, dp]
        L.wso_af_shard_sumsq.restype = None
        L.wso_af_shard_sumsq.argtypes = [C.c_int32, i64p, i64p, i64p, C.c_int32, i64p, i64p, i64p, dp, dp, dp, dp, dp]
        L.wso_af_step.restype = None
        L.wso_af_step.argtypes = [C.POINTER(Hyper), C.c_int64, C.c_double, C.c_double, dp, dp]
        L.wso_af_shard_apply.restype = None
        L.wso_af_shard_apply.argtypes = [C.c_int32, i64p, i64p, i64p, C.c_int64, C.c_int32, dp, dp, dp, C.c_void_p,
                                         C.c_void_p, C.c_int32]
        L.wso_f32_to_bf16.restype = C.c_uint16
        L.wso_f32_to_bf16.argtypes = [C.c_float]
        L.wso_bf16_to_double.restype = C.c_double
        L.wso_bf16_to_double.argtypes = [C.c_uint16]
        L.wso_num_threads.restype = C.c_int32
        L.wso_set_num_threads.restype = C.c_int32
        L.wso_set_num_threads.argtypes = [C.c_int32]
        _lib = L
    return _lib


def _i64(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.int64))


def _p(a: np.ndarray):
    return a.ctypes.data_as(C.POINTER(C.c_int64))


def _ptrs(arrs: Sequence[np.ndarray]):
    out = (C.c_void_p * max(1, len(arrs)))()
    for i, a in enumerate(arrs):
        assert a.flags["C_CONTIGUOUS"]
        out[i] = a.ctypes.data
    return out


def _dtype_code(a: np.ndarray) -> int:
    if a.dtype == np.float32:
        return F32
    if a.dtype == np.uint16:
        return BF16
    raise TypeError(f"oracle takes float32 or uint16(bf16 bits) arrays, got {a.dtype}")


class Plan:
    """O1: piece sizes, in-shard offsets and the combined shard length."""

    def __init__(self, numel: Sequence[int], R: int, A: int):
        self.numel = _i64(numel)
        self.T, self.R, self.A = len(self.numel), int(R), int(A)
        self.piece = np.zeros(self.T, dtype=np.int64)
        self.off = np.zeros(self.T, dtype=np.int64)
        self.S = int(lib().wso_plan(_p(self.numel), self.T, self.R, self.A,
                                    _p(self.piece), _p(self.off)))
        self.G = self.R * self.S
        self.N = int(self.numel.sum())


def pack(plan: Plan, tensors: Sequence[np.ndarray]) -> np.ndarray:
    dt = tensors[0].dtype if len(tensors) else np.float32
    flat = np.empty(plan.G, dtype=dt)
    lib().wso_pack(_ptrs(tensors), _p(plan.numel), _p(plan.piece), _p(plan.off), plan.T,
                   plan.R, plan.S, np.dtype(dt).itemsize, flat.ctypes.data)
    return flat


def unpack(plan: Plan, flat: np.ndarray) -> List[np.ndarray]:
    outs = [np.empty(int(n), dtype=flat.dtype) for n in plan.numel]
    lib().wso_unpack(flat.ctypes.data, _p(plan.numel), _p(plan.piece), _p(plan.off), plan.T,
                     plan.S, flat.dtype.itemsize, _ptrs(outs))
    return outs


def update_tensor(h: Hyper, grads: Sequence[np.ndarray], w: np.ndarray, m: np.ndarray,
                  v: Optional[np.ndarray]) -> float:
    """Unsharded definition on one whole tensor, in place; returns rho (LAMB trust ratio,
    LARS local rate, 1 otherwise)."""
    rho = C.c_double(1.0)
    n = w.size
    if h.opt == LARS:
        lib().wso_lars_tensor(C.byref(h), n, len(grads), _ptrs(grads), _dtype_code(grads[0]),
                              w.ctypes.data, m.ctypes.data, C.byref(rho))
        return rho.value
    lib().wso_update_tensor(C.byref(h), n, len(grads), _ptrs(grads), _dtype_code(grads[0]),
                            w.ctypes.data, m.ctypes.data,
                            v.ctypes.data if v is not None else None, C.byref(rho))
    return rho.value


def update_unsharded(h: Hyper, grads: Sequence[Sequence[np.ndarray]], w, m, v):
    """All tensors of a model; grads[k][t].  In place.  Returns rho per tensor."""
    T = len(w)
    return [update_tensor(h, [g[t] for g in grads], w[t], m[t], v[t] if v is not None else None)
            for t in range(T)]


def sharded_update(h: Hyper, plan: Plan, gpacked: Sequence[np.ndarray], w: np.ndarray,
                   m: np.ndarray, v: Optional[np.ndarray], out_dtype: Optional[int] = None):
    """Sharded route on packed [R][S] buffers, in place.  Returns
    (gathered or None, rho[T], partials[R][T][2])."""
    rho = np.ones(plan.T, dtype=np.float64)
    partials = np.zeros((plan.R, plan.T, 2), dtype=np.float64)
    gathered = None
    if out_dtype is not None:
        gathered = np.empty(plan.G, dtype=np.uint16 if out_dtype == BF16 else np.float32)
    if h.opt == LARS:
        lib().wso_lars_sharded(
            C.byref(h), plan.T, _p(plan.numel), _p(plan.piece), _p(plan.off), plan.S, plan.R,
            len(gpacked), _ptrs(gpacked), _dtype_code(gpacked[0]), w.ctypes.data, m.ctypes.data,
            gathered.ctypes.data if gathered is not None else None,
            out_dtype if out_dtype is not None else F32, rho.ctypes.data_as(C.POINTER(C.c_double)))
        return gathered, rho, partials
    lib().wso_sharded_update(
        C.byref(h), plan.T, _p(plan.numel), _p(plan.piece), _p(plan.off), plan.S, plan.R,
        len(gpacked), _ptrs(gpacked), _dtype_code(gpacked[0]), w.ctypes.data, m.ctypes.data,
        v.ctypes.data if v is not None else None,
        gathered.ctypes.data if gathered is not None else None,
        out_dtype if out_dtype is not None else F32,
        rho.ctypes.data_as(C.POINTER(C.c_double)),
        partials.ctypes.data_as(C.POINTER(C.c_double)))
    return gathered, rho, partials


def _dp(a: np.ndarray):
    assert a.dtype == np.float64 and a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(C.POINTER(C.c_double))


def norm_shard_partial(h: Hyper, plan: Plan, r: int, gslice: np.ndarray, w: np.ndarray, m: np.ndarray,
                       v: Optional[np.ndarray]):
    """Phase 1 of LAMB / LARS as ONE replica runs it: shard r's S-element state and its reduced gradient
    slice.  LAMB updates m, v in place.  Returns (part[T][2], u[S]): the shard's partial sums and the
    per-element quantity phase 2 needs (LAMB: the step direction, LARS: the scaled gradient)."""
    part = np.zeros((plan.T, 2), dtype=np.float64)
    u = np.zeros(plan.S, dtype=np.float64)
    if h.opt == LARS:
        lib().wso_lars_shard_partial(C.byref(h), plan.T, _p(plan.numel), _p(plan.piece), _p(plan.off), r,
                                     gslice.ctypes.data, _dtype_code(gslice), w.ctypes.data, _dp(part), _dp(u))
    else:
        lib().wso_lamb_shard_partial(C.byref(h), plan.T, _p(plan.numel), _p(plan.piece), _p(plan.off), r,
                                     gslice.ctypes.data, _dtype_code(gslice), w.ctypes.data, m.ctypes.data,
                                     v.ctypes.data, _dp(part), _dp(u))
    return part, u


def norm_ratio(h: Hyper, a: float, b: float) -> float:
    """LAMB's trust ratio / LARS's local rate from a tensor's combined sums."""
    return float(lib().wso_norm_ratio(C.byref(h), float(a), float(b)))


def norm_shard_apply(h: Hyper, plan: Plan, r: int, ratio: np.ndarray, u: np.ndarray, w: np.ndarray,
                     m: Optional[np.ndarray], out_dtype: Optional[int] = None):
    """Phase 2 for shard r, in place; returns the shard's slot of the gathered layout (or None)."""
    ratio = np.ascontiguousarray(ratio, dtype=np.float64)
    slot = None
    if out_dtype is not None:
        slot = np.empty(plan.S, dtype=np.uint16 if out_dtype == BF16 else np.float32)
    lib().wso_norm_shard_apply(C.byref(h), plan.T, _p(plan.numel), _p(plan.piece), _p(plan.off), plan.S, r,
                               _dp(ratio), _dp(u), w.ctypes.data, m.ctypes.data if m is not None else None,
                               slot.ctypes.data if slot is not None else None,
                               out_dtype if out_dtype is not None else F32)
    return slot


def factor_shapes(shapes):
    """Adafactor's view of each tensor: (rows, cols) with cols the last dimension and rows all the
    leading ones together; a vector (or scalar) is (numel, 0) and keeps a full second moment.
    Returns int64 arrays rows, cols, foff (start of each tensor's factored state) and the total."""
    rows, cols, foff, tot = [], [], [], 0
    for s in shapes:
        s = tuple(int(d) for d in s)
        n = int(np.prod(s)) if len(s) else 1
        if len(s) >= 2 and n > 0:
            rows.append(n // s[-1]); cols.append(s[-1])
        else:
            rows.append(n); cols.append(0)
        foff.append(tot)
        tot += rows[-1] + cols[-1]
    return _i64(rows), _i64(cols), _i64(foff), tot


def adafactor_tensor(h: Hyper, grads: Sequence[np.ndarray], w: np.ndarray, vr: np.ndarray,
                     vc: Optional[np.ndarray]):
    """One whole tensor, unsharded.  w is (rows, cols) or 1-D; vr/vc fp32, in place.
    Returns (alpha, rms_u, sum_vr)."""
    if w.ndim >= 2:
        cols = w.shape[-1]; rows = w.size // cols
    else:
        rows, cols = w.size, 0
    info = (C.c_double * 3)()
    lib().wso_adafactor_tensor(C.byref(h), rows, cols, len(grads), _ptrs(grads), _dtype_code(grads[0]),
                               w.ctypes.data, vr.ctypes.data, vc.ctypes.data if vc is not None else None, info)
    return tuple(info)


def adafactor_sharded(h: Hyper, plan: Plan, shapes, gpacked: Sequence[np.ndarray], w: np.ndarray,
                      fstate: np.ndarray, out_dtype: Optional[int] = None):
    """Sharded route on packed [R][S] buffers; fstate is the concatenated factored state
    (factor_shapes).  In place.  Returns (gathered or None, info[T][3])."""
    rows, cols, foff, tot = factor_shapes(shapes)
    assert fstate.size == tot and fstate.dtype == np.float32
    info = np.zeros((plan.T, 3), dtype=np.float64)
    gathered = None
    if out_dtype is not None:
        gathered = np.empty(plan.G, dtype=np.uint16 if out_dtype == BF16 else np.float32)
    lib().wso_adafactor_sharded(
        C.byref(h), plan.T, _p(plan.numel), _p(plan.piece), _p(plan.off), plan.S, plan.R,
        len(gpacked), _ptrs(gpacked), _dtype_code(gpacked[0]), _p(rows), _p(cols), _p(foff),
        w.ctypes.data, fstate.ctypes.data, gathered.ctypes.data if gathered is not None else None,
        out_dtype if out_dtype is not None else F32, info.ctypes.data_as(C.POINTER(C.c_double)))
    return gathered, info


class AdafactorReplica:
    """Adafactor as ONE replica runs it (shard r of a plan), stage by stage; the caller moves the partial
    results between replicas.  ``acc`` (this replica's row / column sums, F doubles, to be added over the
    replicas), ``pw`` / ``pu`` (its per-tensor sums of w^2 and u^2)."""

    def __init__(self, h: Hyper, plan: Plan, shapes, r: int):
        self.h, self.plan, self.r = h, plan, r
        self.rows, self.cols, self.foff, self.F = factor_shapes(shapes)
        self.acc = np.zeros(self.F, dtype=np.float64)
        self.pw = np.zeros(plan.T, dtype=np.float64)
        self.pu = np.zeros(plan.T, dtype=np.float64)
        self.gk = np.zeros(plan.S, dtype=np.float64)
        self.u = np.zeros(plan.S, dtype=np.float64)
        self.st = np.zeros(self.F, dtype=np.float64)
        self.sum_r = np.zeros(plan.T, dtype=np.float64)

    def _plan(self):
        p = self.plan
        return p.T, _p(p.numel), _p(p.piece), _p(p.off)

    def sums(self, gslice: np.ndarray, w: np.ndarray):
        T, n, pc, off = self._plan()
        self.acc[:] = 0.0
        lib().wso_af_shard_sums(C.byref(self.h), T, n, pc, off, self.r, gslice.ctypes.data, _dtype_code(gslice),
                                w.ctypes.data, _p(self.rows), _p(self.cols), _p(self.foff), _dp(self.acc), _dp(self.pw),
                                _dp(self.gk))

    def moments(self, acc_total: np.ndarray, fstate: np.ndarray):
        acc_total = np.ascontiguousarray(acc_total, dtype=np.float64)
        lib().wso_af_moments(C.byref(self.h), self.plan.T, _p(self.rows), _p(self.cols), _p(self.foff), _dp(acc_total),
                             fstate.ctypes.data, _dp(self.st), _dp(self.sum_r))

    def sumsq(self):
        T, n, pc, off = self._plan()
        lib().wso_af_shard_sumsq(T, n, pc, off, self.r, _p(self.rows), _p(self.cols), _p(self.foff), _dp(self.st),
                                 _dp(self.sum_r), _dp(self.gk), _dp(self.u), _dp(self.pu))

    def step_sizes(self, sw_total: np.ndarray, su_total: np.ndarray):
        alpha, clip = np.zeros(self.plan.T), np.zeros(self.plan.T)
        a, c = C.c_double(), C.c_double()
        for t in range(self.plan.T):
            lib().wso_af_step(C.byref(self.h), int(self.plan.numel[t]), float(sw_total[t]), float(su_total[t]),
                              C.byref(a), C.byref(c))
            alpha[t], clip[t] = a.value, c.value
        return alpha, clip

    def apply(self, alpha: np.ndarray, clip: np.ndarray, w: np.ndarray, out_dtype: Optional[int] = None):
        T, n, pc, off = self._plan()
        slot = None
        if out_dtype is not None:
            slot = np.empty(self.plan.S, dtype=np.uint16 if out_dtype == BF16 else np.float32)
        lib().wso_af_shard_apply(T, n, pc, off, self.plan.S, self.r, _dp(np.ascontiguousarray(alpha)),
                                 _dp(np.ascontiguousarray(clip)), _dp(self.u), w.ctypes.data,
                                 slot.ctypes.data if slot is not None else None,
                                 out_dtype if out_dtype is not None else F32)
        return slot


def shard_reduce(plan: Plan, r: int, gpacked: Sequence[np.ndarray], grad_scale: float = 1.0):
    out = np.empty(plan.S, dtype=np.float32)
    lib().wso_shard_reduce(plan.T, _p(plan.numel), _p(plan.piece), _p(plan.off), plan.S,
                           len(gpacked), r, _ptrs(gpacked), _dtype_code(gpacked[0]),
                           float(grad_scale), out.ctypes.data)
    return out


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    f = lib().wso_f32_to_bf16
    flat = np.ascontiguousarray(x, dtype=np.float32).ravel()
    return np.array([f(float(a)) if not np.isnan(a) else f(C.c_float(float("nan")))
                     for a in flat], dtype=np.uint16).reshape(np.shape(x))


def bf16_bits_to_f64(x: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(x, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def num_threads() -> int:
    return int(lib().wso_num_threads())


def set_num_threads(n: int) -> int:
    """Threads for the loops with independent iterations (the results do not depend on it);
    returns the previous setting."""
    return int(lib().wso_set_num_threads(int(n)))


class FlatPlan:
    """Concatenated layout (Section 5.2): tensors back to back (starts rounded up to A), the
    concatenation cut into R equal shards wherever the boundaries fall."""

    def __init__(self, numel: Sequence[int], R: int, A: int):
        self.numel = _i64(numel)
        self.T, self.R, self.A = len(self.numel), int(R), int(A)
        self.cat = np.zeros(self.T + 1, dtype=np.int64)
        self.S = int(lib().wso_plan_flat(_p(self.numel), self.T, self.R, self.A, _p(self.cat)))
        self.G = self.R * self.S
        self.N = int(self.numel.sum())

    def tensor_map(self) -> np.ndarray:
        """Owner tensor of every position of the [R][S] layout, -1 for padding."""
        tmap = np.full(self.G, -1, dtype=np.int32)
        for t in range(self.T):
            tmap[self.cat[t]:self.cat[t] + self.numel[t]] = t
        return tmap


def pack_flat(plan: FlatPlan, tensors: Sequence[np.ndarray]) -> np.ndarray:
    dt = tensors[0].dtype if len(tensors) else np.float32
    flat = np.zeros(plan.G, dtype=dt)                      # pads are all-zero bits
    for t, x in enumerate(tensors):
        flat[plan.cat[t]:plan.cat[t] + plan.numel[t]] = x  # position = start of the tensor + index
    return flat


def unpack_flat(plan: FlatPlan, flat: np.ndarray) -> List[np.ndarray]:
    return [flat[plan.cat[t]:plan.cat[t] + plan.numel[t]].copy() for t in range(plan.T)]


def sharded_update_flat(h: Hyper, plan: FlatPlan, gpacked: Sequence[np.ndarray], w: np.ndarray, m: np.ndarray,
                        v: Optional[np.ndarray], out_dtype: Optional[int] = None):
    """Sharded route on the concatenated layout, in place.  Returns (gathered or None, rho[T])."""
    rho = np.ones(plan.T, dtype=np.float64)
    gathered = None
    if out_dtype is not None:
        gathered = np.empty(plan.G, dtype=np.uint16 if out_dtype == BF16 else np.float32)
    tmap = plan.tensor_map()
    lib().wso_sharded_update_map(
        C.byref(h), plan.T, tmap.ctypes.data_as(C.POINTER(C.c_int32)), plan.S, plan.R, len(gpacked),
        _ptrs(gpacked), _dtype_code(gpacked[0]), w.ctypes.data, m.ctypes.data,
        v.ctypes.data if v is not None else None, gathered.ctypes.data if gathered is not None else None,
        out_dtype if out_dtype is not None else F32, rho.ctypes.data_as(C.POINTER(C.c_double)))
    return gathered, rho
