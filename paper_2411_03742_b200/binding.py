"""ctypes binding of the C ABI in include/adacons.h.

Argument marshalling only: every step of the aggregation runs in the library's CUDA kernels.
torch is used for device memory and streams.  If the shared library has not been built the
import of this module's `load_library()` raises -- there is no fallback implementation.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np

_LIB = None
LIB_NAME = "libadacons_b200.so"

# enum adacons_dtype
F32, BF16 = 0, 1
# enum adacons_option
(OPT_BETA, OPT_MOMENTUM, OPT_SORTED, OPT_NORMALIZE, OPT_PER_SEGMENT, OPT_PROFILE, OPT_OVERLAP_LAUNCH,
 OPT_FUSED_SMALL, OPT_ROW_PITCH, OPT_ONE_LAUNCH, OPT_CLUSTER_PASS1, OPT_TALL_TILES, OPT_ALIGNED_BODY,
 OPT_GRAM_PASS1, OPT_SHIFTED_LOADS) = range(15)
# enum adacons_coeff
COEFF_A, COEFF_A_TILDE, COEFF_GAMMA, COEFF_P, COEFF_Q = range(5)
# enum adacons_info
(INFO_NUM_SEGMENTS, INFO_COEFF_SETS, INFO_PASS1_BLOCKS, INFO_SCRATCH_BYTES, INFO_LAUNCHES_PER_CALL,
 INFO_LAST_PATH, INFO_TOTAL_LAUNCHES, INFO_LAST_PASS2, INFO_STATS_DOUBLES) = range(9)
# enum adacons_flag
FLAG_ZERO_ROW, FLAG_DEGENERATE_Z, FLAG_NONFINITE, FLAG_NEG_Z, FLAG_TIMEOUT = 1, 2, 4, 8, 0x100
# enum adacons_error
OK, EINVAL, EALIGN, ENOMEM, ECUDA, EARCH, ETIMEOUT, ELIMIT = range(8)
NOALLOC_MAX_N = 64


class AdaConsError(RuntimeError):
    def __init__(self, code: int, what: str):
        self.code = code
        super().__init__(f"{what}: {strerror(code)} (code {code})")


def library_path() -> str:
    return os.path.join(os.path.dirname(os.path.abspath(__file__)), LIB_NAME)


def load_library() -> ctypes.CDLL:
    """Load the in-tree shared library and declare its prototypes."""
    global _LIB
    if _LIB is not None:
        return _LIB
    path = library_path()
    if not os.path.exists(path):
        raise ImportError(
            f"{path} is missing: build it with `python -m paper_2411_03742_b200.build` "
            "(nvcc, sm_100a).  There is no CPU fallback.")
    lib = ctypes.CDLL(path)
    vp, i32, i64, dbl = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_double
    P = ctypes.POINTER
    protos = {
        "adacons_create": [P(vp), i32, i64, i32, P(i64), i32],
        "adacons_aggregate": [vp, vp, vp, vp],
        "adacons_aggregate_host": [vp, vp, vp, vp],
        "adacons_pass1": [vp, vp, vp, vp],
        "adacons_finish": [vp, vp, vp, vp, i32, vp],
        "adacons_reset": [vp, vp],
        "adacons_destroy": [vp],
        "adacons_set_option": [vp, i32, dbl],
        "adacons_get_option": [vp, i32, P(dbl)],
        "adacons_get_coeffs": [vp, i32, P(dbl), vp],
        "adacons_get_normaliser": [vp, P(dbl), vp],
        "adacons_get_state": [vp, P(dbl), P(i64), vp],
        "adacons_set_state": [vp, P(dbl), i64, vp],
        "adacons_get_status": [vp, P(ctypes.c_uint32), vp],
        "adacons_get_info": [vp, i32, P(i64)],
        "adacons_selftest_bounded_wait": [vp, i32, vp],
        "adacons_get_profile": [vp, P(dbl), P(i64), vp],
        "adacons_stats_noalloc": [vp, i32, i64, i32, vp, vp],
        "adacons_version": [],
    }
    for name, args in protos.items():
        fn = getattr(lib, name)
        fn.argtypes = args
        fn.restype = i32
    lib.adacons_strerror.argtypes = [i32]
    lib.adacons_strerror.restype = ctypes.c_char_p
    _LIB = lib
    return lib


def strerror(code: int) -> str:
    return load_library().adacons_strerror(int(code)).decode()


def _check(code: int, what: str) -> None:
    if code != OK:
        raise AdaConsError(code, what)


def _stream_handle(stream) -> int:
    import torch
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream)


def stats_noalloc(grads, pq_out, stream=None) -> None:
    """p_i = <g_i, gbar> and q_i = ||g_i||^2 of an N x d CUDA tensor into `pq_out` (CUDA tensor of
    2N float64), through the entry point that allocates no device memory (N <= NOALLOC_MAX_N).
    For callers that cannot allocate: e.g. a gradient hook inside a framework whose caching
    allocator already owns the device's memory."""
    import torch
    if grads.dim() != 2 or grads.dtype not in (torch.float32, torch.bfloat16):
        raise ValueError("grads must be an N x d matrix of float32 or bfloat16")
    N, d = grads.shape
    if (N > 1 and grads.stride(0) != d) or (d > 1 and grads.stride(1) != 1):
        raise ValueError("grads must be contiguous (rows d elements apart, unit column stride)")
    if pq_out.dtype != torch.float64 or pq_out.dim() != 1 or pq_out.numel() < 2 * N or not pq_out.is_contiguous():
        raise ValueError("pq_out must be a contiguous float64 vector of at least 2N elements")
    if not (grads.is_cuda and pq_out.is_cuda) or grads.device != pq_out.device:
        raise ValueError("grads and pq_out must live on the same CUDA device")
    if grads.device.index != torch.cuda.current_device():
        raise ValueError("grads must live on the current CUDA device")
    dt = F32 if grads.dtype == torch.float32 else BF16
    _check(load_library().adacons_stats_noalloc(grads.data_ptr(), N, d, dt, pq_out.data_ptr(), _stream_handle(stream)),
           "adacons_stats_noalloc")


def check_tensors(N: int, d: int, dtype: str, pitch: int, grads, out, want_cuda: bool = True) -> None:
    """Raise ValueError unless `grads` is an N x d matrix of `dtype` whose rows are `pitch` elements
    apart with unit column stride and `out` is a contiguous d-vector of the same type (and, with
    want_cuda, both live on one CUDA device).  The library trusts its pointers; this is the guard."""
    import torch
    tdt = {"f32": torch.float32, "bf16": torch.bfloat16}[dtype]
    if grads.dtype != tdt or out.dtype != tdt:
        raise ValueError(f"expected {tdt} tensors, got grads {grads.dtype} and out {out.dtype}")
    if grads.dim() != 2 or tuple(grads.shape) != (N, d):
        raise ValueError(f"grads must have shape ({N}, {d}), got {tuple(grads.shape)}")
    if out.dim() != 1 or out.shape[0] != d:
        raise ValueError(f"out must have shape ({d},), got {tuple(out.shape)}")
    if d > 1 and grads.stride(1) != 1:
        raise ValueError("grads must have unit stride along the gradient dimension")
    if N > 1 and grads.stride(0) != pitch:
        raise ValueError(f"rows of grads are {grads.stride(0)} elements apart, the context expects {pitch} "
                         "(set OPT_ROW_PITCH or pass a contiguous matrix)")
    if d > 1 and out.stride(0) != 1:
        raise ValueError("out must be contiguous")
    if want_cuda:
        if not (grads.is_cuda and out.is_cuda):
            raise ValueError("grads and out must be CUDA tensors (use aggregate_host for host memory)")
        if grads.device != out.device:
            raise ValueError("grads and out must be on the same device")
    elif grads.is_cuda or out.is_cuda:
        raise ValueError("aggregate_host takes host tensors")


class AdaCons:
    """One aggregation context: N workers, gradients of d elements of `dtype` ("f32"/"bf16").

    aggregate(grads, out) takes torch CUDA tensors (grads: N x d contiguous, out: d) and
    enqueues the three kernels on the current (or given) torch stream.
    """

    def __init__(self, N: int, d: int, dtype: str = "f32", seg_offsets=None):
        self._lib = load_library()
        self._ctx = ctypes.c_void_p()
        self.N, self.d, self.dtype = int(N), int(d), dtype
        dt = {"f32": F32, "bf16": BF16}[dtype]
        if seg_offsets is not None:
            off = (ctypes.c_int64 * len(seg_offsets))(*[int(o) for o in seg_offsets])
            rc = self._lib.adacons_create(ctypes.byref(self._ctx), N, d, dt, off, len(seg_offsets) - 1)
        else:
            rc = self._lib.adacons_create(ctypes.byref(self._ctx), N, d, dt, None, 0)
        _check(rc, "adacons_create")
        self._pitch = self.d          # mirrors OPT_ROW_PITCH
        self._checked = None          # signature of the last tensor layout that passed check_tensors

    # -- lifetime ---------------------------------------------------------------------------
    def close(self) -> None:
        if getattr(self, "_ctx", None) is not None and self._ctx.value:
            self._lib.adacons_destroy(self._ctx)
            self._ctx = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    # -- hot path ---------------------------------------------------------------------------
    def aggregate(self, grads, out, stream=None) -> None:
        # the full check runs once per distinct layout; repeats are recognised by their signature
        sig = (grads.dtype, grads.shape, grads.stride(), grads.device, out.dtype, out.shape, out.stride(), out.device)
        if sig != self._checked:
            check_tensors(self.N, self.d, self.dtype, self._pitch, grads, out)
            self._checked = sig
        self.aggregate_ptr(grads.data_ptr(), out.data_ptr(), _stream_handle(stream))

    def aggregate_ptr(self, grads_ptr: int, out_ptr: int, stream_handle: int) -> None:
        _check(self._lib.adacons_aggregate(self._ctx, grads_ptr, out_ptr, stream_handle), "adacons_aggregate")

    def aggregate_host(self, host_grads, host_out, stream=None) -> None:
        """host_grads / host_out: CPU tensors (checked) or numpy arrays (contiguous, unchecked)."""
        if hasattr(host_grads, "data_ptr") and hasattr(host_out, "data_ptr"):
            check_tensors(self.N, self.d, self.dtype, self._pitch, host_grads, host_out, want_cuda=False)
        gp = host_grads.data_ptr() if hasattr(host_grads, "data_ptr") else host_grads.ctypes.data
        op = host_out.data_ptr() if hasattr(host_out, "data_ptr") else host_out.ctypes.data
        _check(self._lib.adacons_aggregate_host(self._ctx, gp, op, _stream_handle(stream)), "adacons_aggregate_host")

    # -- the step in two halves, for a matrix whose columns are spread over devices ----------------
    @property
    def stats_doubles(self) -> int:
        """Doubles in one shard's statistics record: sets * (2 N + 1)."""
        return self.info(INFO_STATS_DOUBLES)

    def _check_stats(self, stats, least: int, what: str) -> None:
        import torch
        if not (stats.is_cuda and stats.dtype == torch.float64 and stats.is_contiguous() and stats.numel() >= least):
            raise ValueError(f"{what} must be a contiguous float64 CUDA tensor of at least {least} elements")

    def pass1(self, grads, stats, stream=None) -> None:
        """Pass 1 on this shard's columns; `stats` (float64 CUDA, stats_doubles elements) receives the
        shard's statistics.  No state change."""
        if grads.device != stats.device:
            raise ValueError("grads and stats must be on the same device")
        self._check_stats(stats, self.stats_doubles, "stats")
        check_tensors(self.N, self.d, self.dtype, self._pitch, grads, grads[0], want_cuda=True)
        _check(self._lib.adacons_pass1(self._ctx, grads.data_ptr(), stats.data_ptr(), _stream_handle(stream)), "adacons_pass1")

    def finish(self, grads, out, stats_all, shards: int, stream=None) -> None:
        """Coefficients from the statistics of all `shards` shards (stats_all: shards x stats_doubles,
        the same order on every device), then pass 2 on this shard's columns."""
        if int(shards) < 1:
            raise ValueError("shards must be at least 1")
        if grads.device != stats_all.device:
            raise ValueError("grads and stats_all must be on the same device")
        self._check_stats(stats_all, int(shards) * self.stats_doubles, "stats_all")
        check_tensors(self.N, self.d, self.dtype, self._pitch, grads, out)
        _check(self._lib.adacons_finish(self._ctx, grads.data_ptr(), out.data_ptr(), stats_all.data_ptr(), int(shards),
                                        _stream_handle(stream)), "adacons_finish")

    def reset(self, stream=None) -> None:
        _check(self._lib.adacons_reset(self._ctx, _stream_handle(stream)), "adacons_reset")

    # -- options, state, diagnostics -----------------------------------------------------------
    def set_option(self, key: int, value: float) -> None:
        _check(self._lib.adacons_set_option(self._ctx, key, float(value)), "adacons_set_option")
        if key == OPT_ROW_PITCH:
            self._pitch = int(value)
            self._checked = None

    def get_option(self, key: int) -> float:
        v = ctypes.c_double()
        _check(self._lib.adacons_get_option(self._ctx, key, ctypes.byref(v)), "adacons_get_option")
        return v.value

    def info(self, key: int) -> int:
        v = ctypes.c_int64()
        _check(self._lib.adacons_get_info(self._ctx, key, ctypes.byref(v)), "adacons_get_info")
        return v.value

    def coeffs(self, which: int = COEFF_GAMMA, stream=None) -> np.ndarray:
        sets = self.info(INFO_COEFF_SETS)
        buf = np.empty((sets, self.N), dtype=np.float64)
        _check(self._lib.adacons_get_coeffs(self._ctx, which, buf.ctypes.data_as(ctypes.POINTER(ctypes.c_double)),
                                            _stream_handle(stream)), "adacons_get_coeffs")
        return buf

    def normaliser(self, stream=None) -> np.ndarray:
        """Z = sum_i u_i of the last call, one value per coefficient set."""
        buf = np.empty(self.info(INFO_COEFF_SETS), dtype=np.float64)
        _check(self._lib.adacons_get_normaliser(self._ctx, buf.ctypes.data_as(ctypes.POINTER(ctypes.c_double)),
                                                _stream_handle(stream)), "adacons_get_normaliser")
        return buf

    def state(self, stream=None):
        sets = self.info(INFO_COEFF_SETS)
        buf = np.empty((sets, self.N), dtype=np.float64)
        step = ctypes.c_int64()
        _check(self._lib.adacons_get_state(self._ctx, buf.ctypes.data_as(ctypes.POINTER(ctypes.c_double)),
                                           ctypes.byref(step), _stream_handle(stream)), "adacons_get_state")
        return buf, step.value

    def set_state(self, m: np.ndarray, step: int, stream=None) -> None:
        m = np.ascontiguousarray(m, dtype=np.float64)
        assert m.size == self.info(INFO_COEFF_SETS) * self.N
        _check(self._lib.adacons_set_state(self._ctx, m.ctypes.data_as(ctypes.POINTER(ctypes.c_double)), int(step),
                                           _stream_handle(stream)), "adacons_set_state")

    def profile(self, stream=None):
        """Mean device time in ms of (pass 1, coefficient step, pass 2) and the number of calls."""
        ms = (ctypes.c_double * 3)()
        n = ctypes.c_int64()
        _check(self._lib.adacons_get_profile(self._ctx, ms, ctypes.byref(n), _stream_handle(stream)), "adacons_get_profile")
        return [ms[0], ms[1], ms[2]], n.value

    def selftest_bounded_wait(self, which: int, stream=None) -> None:
        _check(self._lib.adacons_selftest_bounded_wait(self._ctx, int(which), _stream_handle(stream)),
               "adacons_selftest_bounded_wait")

    def status(self, stream=None) -> int:
        v = ctypes.c_uint32()
        _check(self._lib.adacons_get_status(self._ctx, ctypes.byref(v), _stream_handle(stream)), "adacons_get_status")
        return v.value
