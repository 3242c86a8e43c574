"""Python face of the C-ABI library (``include/omni.h``): argument marshalling only.

Every step of the path runs inside ``libomni.so``; this module turns torch tensors into the
plain pointers and sizes the C functions take.  There is no fallback: if the library cannot
be built or loaded, importing a symbol from it raises.
"""
from __future__ import annotations

import ctypes as C
from dataclasses import dataclass
from typing import List, Optional, Sequence

from . import build as _build

MAX_K = 32
TAU_BINS = 33
BSP, ASP = 0, 1
F32, BF16 = 0, 1
UNSCALED_MEAN, ASP_NO_LR_SCALE, INPUT_IS_TIME, BULK_COPY, NO_BULK_COPY = 1, 2, 4, 8, 16
CONSERVE_MULTIPLICATIVE = 32
DEFAULT_FLAGS = 0  # OR-ed into every new context's flags (the tests use it to force a kernel family)

OK = 0
ERR_NULL, ERR_BAD_K, ERR_BAD_WORKER, ERR_BAD_BATCH, ERR_INFEASIBLE, ERR_BAD_MEASUREMENT = -1, -2, -3, -4, -5, -6
ERR_ALIGN, ERR_BAD_TAU, ERR_CUDA, ERR_TIMEOUT, ERR_BAD_CONFIG, ERR_TOO_LARGE = -7, -8, -9, -10, -11, -12
ERR_NO_MEMORY = -13

EXPORTS = (
    "omni_strerror", "omni_create", "omni_destroy", "omni_get_batches", "omni_set_batches",
    "omni_rebatch", "omni_asp_report", "omni_rebatch_static", "omni_aggregate_bsp",
    "omni_apply_asp", "omni_aggregate_bsp_host", "omni_get_stats", "omni_last_cuda_error",
    "omni_query_launch", "omni_kernel_launches", "omni_aggregate_bsp_noalloc", "omni_apply_asp_batch", "omni_asp_pull", "omni_asp_push_overwrite", "omni_selftest_wait_expiry",
    "omni_ctl_to_device", "omni_ctl_from_device", "omni_rebatch_device", "omni_aggregate_bsp_device_batches",
    "omni_shard_range", "omni_asp_push_pull", "omni_ctl_export", "omni_ctl_import", "omni_step_bsp",
    "omni_asp_report_device",
)
MAX_ASP_BATCH = 16
NOALLOC_MAX_BUCKETS = 8
NOALLOC_MAX_ELEMENTS = 1 << 31


class omni_config(C.Structure):
    _fields_ = [("K", C.c_int32), ("global_batch", C.c_int32), ("b_min", C.c_int32), ("b_max", C.c_int32),
                ("deadband", C.c_double), ("ewma_alpha", C.c_double), ("mode", C.c_int32), ("flags", C.c_uint32)]


class omni_bucket(C.Structure):
    _fields_ = [("param", C.c_void_p), ("momentum", C.c_void_p), ("param_lp", C.c_void_p),
                ("grads", C.POINTER(C.c_void_p)), ("n", C.c_uint64)]


class omni_stats(C.Structure):
    _fields_ = [("grad_sqnorm", C.c_double), ("weight_sum", C.c_double), ("steps", C.c_uint64),
                ("arrivals", C.c_uint64), ("tau_hist", C.c_uint64 * TAU_BINS), ("tau_max", C.c_int32),
                ("tau_sum", C.c_uint64)]


_lib: Optional[C.CDLL] = None


def lib() -> C.CDLL:
    """Build (if stale) and load ``libomni.so``; declare the C signatures."""
    global _lib
    if _lib is not None:
        return _lib
    L = C.CDLL(str(_build.build()))
    vp, i32, f32 = C.c_void_p, C.c_int32, C.c_float
    L.omni_strerror.restype = C.c_char_p
    L.omni_strerror.argtypes = [C.c_int]
    L.omni_create.argtypes = [C.POINTER(omni_config), C.POINTER(vp)]
    L.omni_destroy.argtypes = [vp]
    L.omni_destroy.restype = None
    L.omni_get_batches.argtypes = [vp, C.POINTER(i32)]
    L.omni_set_batches.argtypes = [vp, C.POINTER(i32)]
    L.omni_rebatch.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(i32), C.POINTER(i32)]
    L.omni_asp_report.argtypes = [vp, i32, i32, C.c_double, C.POINTER(i32)]
    L.omni_rebatch_static.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(i32)]
    L.omni_aggregate_bsp.argtypes = [vp, C.POINTER(omni_bucket), i32, i32, C.POINTER(i32), f32, f32, f32, vp]
    L.omni_step_bsp.argtypes = [vp, C.POINTER(omni_bucket), i32, i32, C.POINTER(C.c_double), f32, f32, f32,
                                C.POINTER(i32), C.POINTER(i32), vp]
    L.omni_apply_asp.argtypes = [vp, C.POINTER(omni_bucket), i32, i32, i32, i32, i32, f32, f32, f32, vp]
    L.omni_apply_asp_batch.argtypes = [vp, C.POINTER(omni_bucket), i32, i32, i32, C.POINTER(i32), C.POINTER(i32),
                                       C.POINTER(i32), f32, f32, f32, vp]
    L.omni_asp_pull.argtypes = [vp, C.POINTER(omni_bucket), i32, C.POINTER(vp), vp]
    L.omni_asp_push_overwrite.argtypes = [vp, C.POINTER(omni_bucket), i32, i32, i32, i32, i32, C.POINTER(vp), f32, f32, vp]
    L.omni_asp_push_pull.argtypes = [vp, C.POINTER(omni_bucket), i32, i32, i32, i32, i32, C.POINTER(vp), f32, f32, vp]
    L.omni_aggregate_bsp_host.argtypes = [vp, C.POINTER(omni_bucket), i32, i32, C.POINTER(vp), C.POINTER(i32),
                                          f32, f32, f32, vp, C.POINTER(C.c_double)]
    L.omni_get_stats.argtypes = [vp, C.POINTER(omni_stats), vp]
    L.omni_ctl_to_device.argtypes = [vp, vp]
    L.omni_ctl_from_device.argtypes = [vp, vp]
    L.omni_rebatch_device.argtypes = [vp, vp, vp, vp]
    L.omni_asp_report_device.argtypes = [vp, i32, i32, vp, vp, vp]
    L.omni_aggregate_bsp_device_batches.argtypes = [vp, C.POINTER(omni_bucket), i32, i32, f32, f32, f32, vp]
    L.omni_shard_range.argtypes = [C.c_uint64, i32, i32, C.POINTER(C.c_uint64), C.POINTER(C.c_uint64)]
    L.omni_ctl_export.argtypes = [vp, vp, C.POINTER(C.c_uint64)]
    L.omni_ctl_import.argtypes = [vp, vp, C.c_uint64]
    L.omni_selftest_wait_expiry.argtypes = [vp, vp]
    L.omni_last_cuda_error.argtypes = [vp]
    L.omni_query_launch.argtypes = [vp, i32, i32, C.POINTER(i32), C.POINTER(i32)]
    L.omni_kernel_launches.argtypes = [vp]
    L.omni_kernel_launches.restype = C.c_uint64
    L.omni_aggregate_bsp_noalloc.argtypes = [i32, C.POINTER(omni_bucket), i32, i32, C.POINTER(i32), C.c_uint32,
                                             f32, f32, f32, vp, vp]
    _lib = L
    return L


def shard_range(n: int, world: int, rank: int):
    """(begin, count) of the elements of an n-element bucket that rank ``rank`` of ``world`` owns."""
    b, c = C.c_uint64(), C.c_uint64()
    rc = lib().omni_shard_range(n, world, rank, C.byref(b), C.byref(c))
    if rc != OK:
        raise OmniError(rc)
    return b.value, c.value


class OmniError(RuntimeError):
    def __init__(self, status: int, cuda: int = 0):
        msg = lib().omni_strerror(status).decode()
        super().__init__(f"omni status {status}: {msg}" + (f" (cudaError {cuda})" if cuda else ""))
        self.status = status
        self.cuda = cuda


def _dtype_code(t) -> int:
    import torch

    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError(f"gradient dtype {t.dtype} is not float32 or bfloat16")


@dataclass
class Stats:
    grad_sqnorm: float
    weight_sum: float
    steps: int
    arrivals: int
    tau_hist: List[int]
    tau_max: int
    tau_sum: int = 0

    @property
    def tau_mean(self) -> float:
        return self.tau_sum / self.arrivals if self.arrivals else 0.0


class BucketSet:
    """Marshalled bucket descriptors, built once and reused every step.

    ``params`` / ``momenta`` / ``params_lp``: one tensor per bucket (momentum and low-precision
    entries may be None); ``grads[i][k]``: worker k's gradient tensor for bucket i.  The tensors
    are kept alive by this object.
    """

    def __init__(self, params: Sequence, grads: Sequence[Sequence], momenta: Optional[Sequence] = None,
                 params_lp: Optional[Sequence] = None):
        nb = len(params)
        momenta = list(momenta) if momenta is not None else [None] * nb
        params_lp = list(params_lp) if params_lp is not None else [None] * nb
        assert len(grads) == nb and len(momenta) == nb and len(params_lp) == nb
        self._keep = (list(params), [list(g) for g in grads], momenta, params_lp)
        self.n_buckets = nb
        self.K = len(grads[0]) if nb else 0
        self.dtype = _dtype_code(grads[0][0]) if nb else F32
        self.array = (omni_bucket * max(nb, 1))()
        self._tables = []
        for i in range(nb):
            p, m, lp, gs = params[i], momenta[i], params_lp[i], grads[i]
            n = p.numel()
            assert p.is_contiguous() and p.dtype.is_floating_point and p.element_size() == 4
            assert len(gs) == self.K
            tab = (C.c_void_p * self.K)()
            for k, g in enumerate(gs):
                assert g.numel() == n and g.is_contiguous() and _dtype_code(g) == self.dtype
                tab[k] = g.data_ptr()
            self._tables.append(tab)
            if m is not None:
                assert m.numel() == n and m.is_contiguous() and m.element_size() == 4
            if lp is not None:
                assert lp.numel() == n and lp.is_contiguous() and lp.element_size() == 2
            self.array[i] = omni_bucket(p.data_ptr(), m.data_ptr() if m is not None else None,
                                        lp.data_ptr() if lp is not None else None,
                                        C.cast(tab, C.POINTER(C.c_void_p)), n)

    @classmethod
    def from_flat(cls, layout, theta, grads, v=None, theta_lp=None) -> "BucketSet":
        """Slice flat buffers (``workloads.Layout``) into per-bucket views."""
        sl = [slice(b.start, b.start + b.n) for b in layout.buckets]
        return cls([theta[s] for s in sl], [[g[s] for g in grads] for s in sl],
                   [v[s] for s in sl] if v is not None else None,
                   [theta_lp[s] for s in sl] if theta_lp is not None else None)


def aggregate_bsp_noalloc(buckets: "BucketSet", b: Sequence[int], lr: float, momentum: float = 0.0,
                          weight_decay: float = 0.0, flags: int = 0, grad_sqnorm_out=None, stream=None) -> None:
    """The fused synchronous step through ``omni_aggregate_bsp_noalloc``, the entry point for
    callers that may not allocate device memory while stepping (allocator callbacks, processes
    whose memory is all pooled, loops that ban device-synchronising calls).  No context: K is
    ``buckets.K``.  ``grad_sqnorm_out``: optional one-element float64 CUDA tensor that receives
    the squared norm.  Calls on one device share a fixed scratch array: keep them ordered on a
    stream, and make the first call on a device outside stream capture."""
    K = buckets.K
    ptr = None
    if grad_sqnorm_out is not None:
        assert grad_sqnorm_out.numel() == 1 and grad_sqnorm_out.element_size() == 8 and grad_sqnorm_out.is_cuda
        ptr = C.c_void_p(grad_sqnorm_out.data_ptr())
    rc = lib().omni_aggregate_bsp_noalloc(K, buckets.array, buckets.n_buckets, buckets.dtype, (C.c_int32 * K)(*b),
                                          flags, lr, momentum, weight_decay, ptr, Omni._stream(stream))
    if rc != OK:
        raise OmniError(rc)


class Omni:
    """One controller + aggregation context (``omni_ctx``)."""

    def __init__(self, K: int, global_batch: int, b_min: int, b_max: int, deadband: float = 0.10,
                 ewma_alpha: float = 1.0, mode: int = BSP, flags: int = 0):
        self._h = C.c_void_p()
        self.K = K
        self.global_batch = global_batch
        cfg = omni_config(K, global_batch, b_min, b_max, deadband, ewma_alpha, mode, flags | DEFAULT_FLAGS)
        self._check(lib().omni_create(C.byref(cfg), C.byref(self._h)))
        self._i32K = C.c_int32 * K
        self._f64K = C.c_double * K

    def _check(self, rc: int) -> None:
        if rc != OK:
            raise OmniError(rc, lib().omni_last_cuda_error(self._h) if self._h else 0)

    def close(self) -> None:
        if self._h:
            lib().omni_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- controller -------------------------------------------------------------------------
    @property
    def batches(self) -> List[int]:
        b = self._i32K()
        self._check(lib().omni_get_batches(self._h, b))
        return list(b)

    def set_batches(self, b: Sequence[int]) -> None:
        self._check(lib().omni_set_batches(self._h, self._i32K(*b)))

    def rebatch(self, measured: Sequence[float]):
        """Returns (new batches, changed flags)."""
        nb, ch = self._i32K(), self._i32K()
        self._check(lib().omni_rebatch(self._h, self._f64K(*measured), nb, ch))
        return list(nb), list(ch)

    def asp_report(self, worker: int, b_used: int, measured: float) -> int:
        out = C.c_int32()
        self._check(lib().omni_asp_report(self._h, worker, b_used, measured, C.byref(out)))
        return out.value

    def rebatch_static(self, capacity: Sequence[float]) -> List[int]:
        nb = self._i32K()
        self._check(lib().omni_rebatch_static(self._h, self._f64K(*capacity), nb))
        return list(nb)

    def export_state(self) -> bytes:
        """The controller state (batches, smoothed times) as bytes, for a checkpoint."""
        size = C.c_uint64(0)
        self._check(lib().omni_ctl_export(self._h, None, C.byref(size)))
        buf = C.create_string_buffer(size.value)
        self._check(lib().omni_ctl_export(self._h, buf, C.byref(size)))
        return buf.raw[:size.value]

    def import_state(self, record: bytes) -> None:
        self._check(lib().omni_ctl_import(self._h, record, len(record)))

    # ---- device path ------------------------------------------------------------------------
    @staticmethod
    def _stream(stream) -> C.c_void_p:
        """The raw cudaStream_t of ``stream`` (a torch stream), or of torch's current stream."""
        if stream is None:
            import torch

            raw = getattr(torch._C, "_cuda_getCurrentRawStream", None)     # no Stream object built: the call sits
            if raw is not None:                                            # on the path of every step
                return C.c_void_p(raw(torch.cuda.current_device()))
            stream = torch.cuda.current_stream()
        return C.c_void_p(stream.cuda_stream)

    def aggregate_bsp(self, buckets: BucketSet, b: Sequence[int], lr: float, momentum: float = 0.0,
                      weight_decay: float = 0.0, stream=None) -> None:
        self._check(lib().omni_aggregate_bsp(self._h, buckets.array, buckets.n_buckets, buckets.dtype,
                                             self._i32K(*b), lr, momentum, weight_decay, self._stream(stream)))

    def step_bsp(self, buckets: BucketSet, measured: Sequence[float], lr: float, momentum: float = 0.0,
                 weight_decay: float = 0.0, stream=None) -> List[int]:
        """One iteration of Algorithm 1 in one call: aggregate + update with the current batches,
        then re-batch from ``measured``; returns the batches for the next iteration."""
        nb = self._i32K()
        self._check(lib().omni_step_bsp(self._h, buckets.array, buckets.n_buckets, buckets.dtype,
                                        self._f64K(*measured), lr, momentum, weight_decay, nb, None,
                                        self._stream(stream)))
        return list(nb)

    def aggregate_bsp_host(self, buckets: BucketSet, host_grads: Sequence[Sequence], b: Sequence[int], lr: float,
                           momentum: float = 0.0, weight_decay: float = 0.0, stream=None) -> float:
        """``host_grads[i][k]``: pinned host tensor with worker k's gradient of bucket i."""
        flat = (C.c_void_p * max(1, buckets.n_buckets * self.K))()
        for i, row in enumerate(host_grads):
            for k, t in enumerate(row):
                flat[i * self.K + k] = t.data_ptr()
        sq = C.c_double()
        self._check(lib().omni_aggregate_bsp_host(self._h, buckets.array, buckets.n_buckets, buckets.dtype, flat,
                                                  self._i32K(*b), lr, momentum, weight_decay,
                                                  self._stream(stream), C.byref(sq)))
        return sq.value

    def apply_asp(self, buckets: BucketSet, worker: int, b_used: int, tau: int, lr: float, momentum: float = 0.0,
                  weight_decay: float = 0.0, stream=None) -> None:
        self._check(lib().omni_apply_asp(self._h, buckets.array, buckets.n_buckets, buckets.dtype, worker, b_used,
                                         tau, lr, momentum, weight_decay, self._stream(stream)))

    def apply_asp_batch(self, buckets: BucketSet, workers: Sequence[int], b_used: Sequence[int], tau: Sequence[int],
                        lr: float, momentum: float = 0.0, weight_decay: float = 0.0, stream=None) -> None:
        """m queued arrivals in one pass (same result as m ``apply_asp`` calls in that order)."""
        m = len(workers)
        arr = C.c_int32 * m
        self._check(lib().omni_apply_asp_batch(self._h, buckets.array, buckets.n_buckets, buckets.dtype, m,
                                               arr(*workers), arr(*b_used), arr(*tau), lr, momentum, weight_decay,
                                               self._stream(stream)))

    @staticmethod
    def _ptr_table(tensors):
        tab = (C.c_void_p * max(1, len(tensors)))()
        for i, t in enumerate(tensors):
            tab[i] = t.data_ptr()
        return tab

    def asp_pull(self, buckets: BucketSet, snapshots: Sequence, stream=None) -> None:
        """pullFromPS: ``snapshots[i]`` (float32 CUDA tensor per bucket) <- the server parameters."""
        self._check(lib().omni_asp_pull(self._h, buckets.array, buckets.n_buckets, self._ptr_table(snapshots),
                                        self._stream(stream)))

    def asp_push_overwrite(self, buckets: BucketSet, worker: int, b_used: int, tau: int, snapshots: Sequence,
                           lr: float, weight_decay: float = 0.0, stream=None) -> None:
        """Algorithm 2 literally: server parameters <- snapshot - eta_k * gradient (overwrite)."""
        self._check(lib().omni_asp_push_overwrite(self._h, buckets.array, buckets.n_buckets, buckets.dtype, worker,
                                                  b_used, tau, self._ptr_table(snapshots), lr, weight_decay,
                                                  self._stream(stream)))

    # ---- device-resident controller ---------------------------------------------------------
    def ctl_to_device(self, stream=None) -> None:
        """Copy the controller state and the weights to the device copy (allocated on first use)."""
        self._check(lib().omni_ctl_to_device(self._h, self._stream(stream)))

    def ctl_from_device(self, stream=None) -> List[int]:
        """Synchronise, copy the device copy back into the host controller; returns the batches.
        Raises the failure a device re-batch recorded (e.g. a non-positive measurement)."""
        self._check(lib().omni_ctl_from_device(self._h, self._stream(stream)))
        return self.batches

    def rebatch_device(self, measured, new_b=None, stream=None) -> None:
        """``measured``: float64 CUDA tensor of K values; ``new_b``: optional int32 CUDA tensor of K."""
        assert measured.is_cuda and measured.element_size() == 8 and measured.numel() >= self.K
        assert new_b is None or (new_b.is_cuda and new_b.element_size() == 4 and new_b.numel() >= self.K)
        self._check(lib().omni_rebatch_device(self._h, C.c_void_p(measured.data_ptr()),
                                              C.c_void_p(new_b.data_ptr()) if new_b is not None else None,
                                              self._stream(stream)))

    def asp_report_device(self, worker: int, b_used: int, measured, new_b=None, stream=None) -> None:
        """evalBsz on the device copy: ``measured`` is a one-element float64 CUDA tensor, ``new_b`` an
        optional one-element int32 CUDA tensor that receives the worker's new batch."""
        assert measured.is_cuda and measured.element_size() == 8 and measured.numel() >= 1
        assert new_b is None or (new_b.is_cuda and new_b.element_size() == 4 and new_b.numel() >= 1)
        self._check(lib().omni_asp_report_device(self._h, worker, b_used, C.c_void_p(measured.data_ptr()),
                                                 C.c_void_p(new_b.data_ptr()) if new_b is not None else None,
                                                 self._stream(stream)))

    def aggregate_bsp_device_batches(self, buckets: BucketSet, lr: float, momentum: float = 0.0,
                                     weight_decay: float = 0.0, stream=None) -> None:
        self._check(lib().omni_aggregate_bsp_device_batches(self._h, buckets.array, buckets.n_buckets, buckets.dtype,
                                                            lr, momentum, weight_decay, self._stream(stream)))

    def asp_push_pull(self, buckets: BucketSet, worker: int, b_used: int, tau: int, snapshots: Sequence,
                      lr: float, weight_decay: float = 0.0, stream=None) -> None:
        """Push with overwrite and the same worker's next pull in one launch: the server parameters
        and ``snapshots`` both receive snapshot - eta_k * gradient."""
        self._check(lib().omni_asp_push_pull(self._h, buckets.array, buckets.n_buckets, buckets.dtype, worker,
                                             b_used, tau, self._ptr_table(snapshots), lr, weight_decay,
                                             self._stream(stream)))

    def stats(self, stream=None) -> Stats:
        s = omni_stats()
        st = C.c_void_p(0) if stream is None and not self._device_used() else self._stream(stream)
        self._check(lib().omni_get_stats(self._h, C.byref(s), st))
        return Stats(s.grad_sqnorm, s.weight_sum, s.steps, s.arrivals, list(s.tau_hist), s.tau_max, s.tau_sum)

    def selftest_wait_expiry(self, stream=None) -> None:
        """Enqueue the diagnostic kernel whose bounded wait runs out (next ``stats()`` raises TIMEOUT)."""
        self._check(lib().omni_selftest_wait_expiry(self._h, self._stream(stream)))

    def _device_used(self) -> bool:
        return lib().omni_kernel_launches(self._h) > 0

    def query_launch(self, K: int, dtype: int):
        g, b = C.c_int32(), C.c_int32()
        self._check(lib().omni_query_launch(self._h, K, dtype, C.byref(g), C.byref(b)))
        return g.value, b.value

    @property
    def kernel_launches(self) -> int:
        return lib().omni_kernel_launches(self._h)
