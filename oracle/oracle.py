"""ctypes front end of the CPU oracle (``omni_oracle.c``).

TEST INFRASTRUCTURE: only the tests, the smoke check and the benchmark's CPU-baseline leg load
this module.  It shares nothing with the CUDA library and never imports it.

Arrays are numpy; gradients are a list of K one-dimensional arrays, ``float32`` or ``uint16``
(bfloat16 bit patterns).  State arrays are updated in place.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "omni_oracle.c"
_LIB = _HERE / "libomni_oracle.so"

MAX_K = 32
MODE_BSP, MODE_ASP = 0, 1
FLAG_UNSCALED_MEAN, FLAG_ASP_NO_LR_SCALE, FLAG_INPUT_IS_TIME, FLAG_CONSERVE_MULTIPLICATIVE = 1, 2, 4, 8
OK, ERR_ARG, ERR_INFEASIBLE, ERR_MEASUREMENT = 0, -1, -2, -3


def build(force: bool = False) -> Path:
    """Compile the oracle with the host compiler alone.  No FMA contraction, no fast-math."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".{os.getpid()}.tmp")
        subprocess.run(
            ["gcc", "-std=c11", "-O2", "-ffp-contract=off", "-fPIC", "-shared",
             "-o", str(tmp), str(_SRC), "-lm"],
            check=True,
        )
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        # OMNI_ORACLE_LIB: load this build of the oracle instead (used by the test that plants
        # mistakes in copies of the source to show that the pins catch them)
        L = C.CDLL(os.environ.get("OMNI_ORACLE_LIB") or str(build()))
        vp, i32, u32, u64, f64, f32 = C.c_void_p, C.c_int32, C.c_uint32, C.c_uint64, C.c_double, C.c_float
        L.oracle_ctl_sizeof.restype = C.c_size_t
        L.oracle_ctl_init.argtypes = [vp, i32, i32, i32, i32, f64, f64, i32, u32]
        L.oracle_ctl_set_batches.argtypes = [vp, vp]
        L.oracle_ctl_get_batches.argtypes = [vp, vp]
        L.oracle_ctl_get_batches.restype = None
        L.oracle_rebatch.argtypes = [vp, vp, vp, vp, vp, vp]
        L.oracle_asp_report.argtypes = [vp, i32, i32, f64, vp]
        L.oracle_rebatch_static.argtypes = [vp, vp, vp]
        L.oracle_bsp_weights.argtypes = [i32, vp, u32, vp, vp]
        L.oracle_bsp_weights.restype = None
        L.oracle_asp_lr.argtypes = [f64, i32, i32, u32]
        L.oracle_asp_lr.restype = f64
        L.oracle_float_to_bf16.argtypes = [vp, vp, u64]
        L.oracle_float_to_bf16.restype = None
        L.oracle_bf16_to_float.argtypes = [vp, vp, u64]
        L.oracle_bf16_to_float.restype = None
        L.oracle_bsp_step_f64.argtypes = [i32, u64, vp, C.c_int, vp, u32, vp, vp, f64, f64, f64, vp]
        L.oracle_bsp_step_f64.restype = None
        L.oracle_bsp_step_f32.argtypes = [i32, u64, vp, C.c_int, vp, u32, vp, vp, vp, f32, f32, f32, vp]
        L.oracle_bsp_step_f32.restype = None
        L.oracle_asp_apply_f64.argtypes = [u64, vp, C.c_int, i32, i32, u32, vp, vp, f64, f64, f64]
        L.oracle_asp_apply_f64.restype = None
        L.oracle_asp_apply_f32.argtypes = [u64, vp, C.c_int, i32, i32, u32, vp, vp, vp, f32, f32, f32]
        L.oracle_asp_apply_f32.restype = None
        L.oracle_asp_push_overwrite_f64.argtypes = [u64, vp, C.c_int, i32, i32, u32, vp, vp, f64, f64]
        L.oracle_asp_push_overwrite_f64.restype = None
        L.oracle_asp_push_overwrite_f32.argtypes = [u64, vp, C.c_int, i32, i32, u32, vp, vp, vp, f32, f32]
        L.oracle_asp_push_overwrite_f32.restype = None
        L.oracle_tau_record.argtypes = [vp, vp, i32]
        L.oracle_tau_record.restype = None
        _lib = L
    return _lib


class OracleError(RuntimeError):
    def __init__(self, code: int):
        super().__init__(f"oracle error {code}")
        self.code = code


def _ptr(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _chk(a: np.ndarray, dtype) -> np.ndarray:
    assert a.dtype == dtype and a.flags.c_contiguous and a.ndim == 1, (a.dtype, a.shape)
    return a


def _grad_table(g):
    """K one-dimensional arrays of one dtype -> (void*[K], is_bf16, n)."""
    K = len(g)
    dt = g[0].dtype
    assert dt in (np.float32, np.uint16)
    n = g[0].shape[0]
    tab = (C.c_void_p * K)()
    for k, a in enumerate(g):
        _chk(a, dt)
        assert a.shape[0] == n
        tab[k] = a.ctypes.data
    return tab, int(dt == np.uint16), n


class Controller:
    """The batch-size controller of Alg. 1 (``rebatch``) and Alg. 2 (``asp_report``)."""

    def __init__(self, K, B, b_min, b_max, deadband, alpha=1.0, mode=MODE_BSP, flags=0):
        L = lib()
        self._buf = C.create_string_buffer(L.oracle_ctl_sizeof())
        rc = L.oracle_ctl_init(self._buf, K, B, b_min, b_max, deadband, alpha, mode, flags)
        if rc != OK:
            raise OracleError(rc)
        self.K = K

    @property
    def batches(self) -> np.ndarray:
        b = np.zeros(self.K, np.int32)
        lib().oracle_ctl_get_batches(self._buf, _ptr(b))
        return b

    def set_batches(self, b) -> None:
        b = np.ascontiguousarray(b, np.int32)
        assert b.shape == (self.K,)
        rc = lib().oracle_ctl_set_batches(self._buf, _ptr(b))
        if rc != OK:
            raise OracleError(rc)

    def rebatch(self, measured, want_bstar=False, want_scaled=False):
        """(new batches, changed flags[, b* of Eq. 6b][, real-valued batches before rounding])."""
        m = np.ascontiguousarray(measured, np.float64)
        assert m.shape == (self.K,)
        nb = np.zeros(self.K, np.int32)
        ch = np.zeros(self.K, np.int32)
        bs = np.zeros(self.K, np.float64)
        sc = np.zeros(self.K, np.float64)
        rc = lib().oracle_rebatch(self._buf, _ptr(m), _ptr(nb), _ptr(ch), _ptr(bs), _ptr(sc))
        if rc != OK:
            raise OracleError(rc)
        out = (nb, ch)
        if want_bstar:
            out += (bs,)
        if want_scaled:
            out += (sc,)
        return out

    def rebatch_static(self, capacity) -> np.ndarray:
        c = np.ascontiguousarray(capacity, np.float64)
        assert c.shape == (self.K,)
        nb = np.zeros(self.K, np.int32)
        rc = lib().oracle_rebatch_static(self._buf, _ptr(c), _ptr(nb))
        if rc != OK:
            raise OracleError(rc)
        return nb

    def asp_report(self, worker, b_used, measured) -> int:
        out = C.c_int32(0)
        rc = lib().oracle_asp_report(self._buf, worker, b_used, float(measured), C.byref(out))
        if rc != OK:
            raise OracleError(rc)
        return out.value


def bsp_weights(b, flags=0):
    b = np.ascontiguousarray(b, np.int32)
    l64 = np.zeros(len(b), np.float64)
    l32 = np.zeros(len(b), np.float32)
    lib().oracle_bsp_weights(len(b), _ptr(b), flags, _ptr(l64), _ptr(l32))
    return l64, l32


def asp_lr(lr, b_used, B, flags=0) -> float:
    return lib().oracle_asp_lr(lr, b_used, B, flags)


def float_to_bf16(x: np.ndarray) -> np.ndarray:
    x = np.ascontiguousarray(x, np.float32).ravel()
    y = np.empty(x.shape, np.uint16)
    lib().oracle_float_to_bf16(_ptr(x), _ptr(y), x.size)
    return y


def bf16_to_float(x: np.ndarray) -> np.ndarray:
    x = np.ascontiguousarray(x, np.uint16).ravel()
    y = np.empty(x.shape, np.float32)
    lib().oracle_bf16_to_float(_ptr(x), _ptr(y), x.size)
    return y


def bsp_step_f64(g, b, theta, v, lr, mu, wd, flags=0) -> float:
    tab, bf, n = _grad_table(g)
    b = np.ascontiguousarray(b, np.int32)
    _chk(theta, np.float64)
    assert theta.shape[0] == n and (v is None or _chk(v, np.float64).shape[0] == n)
    assert v is not None or mu == 0
    sq = C.c_double(0)
    lib().oracle_bsp_step_f64(len(g), n, tab, bf, _ptr(b), flags, _ptr(theta), _ptr(v),
                              lr, mu, wd, C.byref(sq))
    return sq.value


def bsp_step_f32(g, b, theta, v, lr, mu, wd, flags=0, theta_lp=None) -> float:
    tab, bf, n = _grad_table(g)
    b = np.ascontiguousarray(b, np.int32)
    _chk(theta, np.float32)
    assert theta.shape[0] == n and (v is None or _chk(v, np.float32).shape[0] == n)
    assert v is not None or mu == 0
    assert theta_lp is None or _chk(theta_lp, np.uint16).shape[0] == n
    sq = C.c_double(0)
    lib().oracle_bsp_step_f32(len(g), n, tab, bf, _ptr(b), flags, _ptr(theta), _ptr(v),
                              _ptr(theta_lp), lr, mu, wd, C.byref(sq))
    return sq.value


def asp_apply_f64(g, b_used, B, theta, v, lr, mu, wd, flags=0) -> None:
    assert g.dtype in (np.float32, np.uint16) and g.flags.c_contiguous
    _chk(theta, np.float64)
    assert v is not None or mu == 0
    lib().oracle_asp_apply_f64(g.shape[0], _ptr(g), int(g.dtype == np.uint16), b_used, B, flags,
                               _ptr(theta), _ptr(v), lr, mu, wd)


def asp_apply_f32(g, b_used, B, theta, v, lr, mu, wd, flags=0, theta_lp=None) -> None:
    assert g.dtype in (np.float32, np.uint16) and g.flags.c_contiguous
    _chk(theta, np.float32)
    assert v is not None or mu == 0
    lib().oracle_asp_apply_f32(g.shape[0], _ptr(g), int(g.dtype == np.uint16), b_used, B, flags,
                               _ptr(theta), _ptr(v), _ptr(theta_lp), lr, mu, wd)


def asp_push_overwrite_f64(g, b_used, B, theta, snapshot, lr, wd=0.0, flags=0) -> None:
    """Algorithm 2 literally: theta (server, overwritten) <- snapshot - eta_k * g."""
    assert g.dtype in (np.float32, np.uint16) and g.flags.c_contiguous
    _chk(theta, np.float64), _chk(snapshot, np.float64)
    assert theta.shape == snapshot.shape == g.shape
    lib().oracle_asp_push_overwrite_f64(g.shape[0], _ptr(g), int(g.dtype == np.uint16), b_used, B, flags,
                                        _ptr(theta), _ptr(snapshot), lr, wd)


def asp_push_overwrite_f32(g, b_used, B, theta, snapshot, lr, wd=0.0, flags=0, theta_lp=None) -> None:
    assert g.dtype in (np.float32, np.uint16) and g.flags.c_contiguous
    _chk(theta, np.float32), _chk(snapshot, np.float32)
    assert theta.shape == snapshot.shape == g.shape
    lib().oracle_asp_push_overwrite_f32(g.shape[0], _ptr(g), int(g.dtype == np.uint16), b_used, B, flags,
                                        _ptr(theta), _ptr(snapshot), _ptr(theta_lp), lr, wd)


class TauStats:
    """Staleness tally of an arrival stream: 32 bins and an overflow bin, plus the maximum."""

    def __init__(self):
        self.hist = np.zeros(33, np.uint64)
        self._max = C.c_int32(0)

    def record(self, tau: int) -> None:
        lib().oracle_tau_record(_ptr(self.hist), C.byref(self._max), tau)

    @property
    def tau_max(self) -> int:
        return self._max.value
