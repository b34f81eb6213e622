"""ctypes binding of ``libleapfrog.so``: argument marshalling only.

Every function has the name and meaning of the C entry point declared in
``include/leapfrog.h``; tensors are passed as raw device (or, for ``lf_backward_host``, host)
addresses.  There is no fallback of any kind: if the shared library has not been built the
import fails with an error that says how to build it.
"""
from __future__ import annotations

import ctypes
import os

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libleapfrog.so")

LF_OK, LF_EINVAL, LF_ENULL, LF_EALIGN, LF_ERESOURCE, LF_ECUDA, LF_ETIMEOUT, LF_ENOMEM = (
    0, -1, -2, -3, -4, -5, -6, -7)
LF_ECAPACITY = -8
LF_VARIANT_AUTO, LF_VARIANT_STREAMS, LF_VARIANT_PERSISTENT, LF_VARIANT_FUSED = 0, 1, 2, 3
LF_GW_MATH_AUTO, LF_GW_MATH_FP32, LF_GW_MATH_TF32 = 0, 1, 2
LF_OPT_VARIANT, LF_OPT_GW_MATH, LF_OPT_WAIT_BUDGET_US, LF_OPT_USE_GRAPH, LF_OPT_WITHHOLD = 1, 2, 3, 4, 5
LF_OPT_DELTA_MATH = 6
LF_OPT_TC_TILING = 7
LF_OPT_COST = 8
LF_OPT_ACTIVATION = 9
LF_OPT_SHARD_COUNT, LF_OPT_SHARD_RANK = 10, 11
LF_OPT_FUSED_TILING = 12
LF_OPT_TIME_CALLS = 13
LF_FUSED_TILING_AUTO, LF_FUSED_TILING_CLUSTERS, LF_FUSED_TILING_COLUMNS = 0, 1, 2
LF_ACT_SIGMOID, LF_ACT_TANH, LF_ACT_RELU = 0, 1, 2
LF_COST_QUADRATIC, LF_COST_CROSS_ENTROPY = 0, 1
LF_TC_TILING_AUTO, LF_TC_TILING_ONE_SM, LF_TC_TILING_TWO_SM = 0, 1, 2
LF_DELTA_MATH_AUTO, LF_DELTA_MATH_FP32, LF_DELTA_MATH_3XTF32, LF_DELTA_MATH_TF32_BF16 = 0, 1, 2, 3

EXPORTS = ("lf_create", "lf_create_widths", "lf_set_stream", "lf_set_option", "lf_forward", "lf_backward",
           "lf_backward_sgd", "lf_grad_w", "lf_backward_host", "lf_sync", "lf_owner", "lf_get_stats", "lf_last_cuda_error",
           "lf_strerror", "lf_version", "lf_destroy", "lf_delta_step_static")


class lf_stats(ctypes.Structure):
    _fields_ = [("L", ctypes.c_int), ("N", ctypes.c_int), ("B", ctypes.c_int),
                ("k", ctypes.c_int), ("k_effective", ctypes.c_int), ("variant", ctypes.c_int),
                ("gw_math", ctypes.c_int), ("sm_count", ctypes.c_int),
                ("chain_ctas", ctypes.c_int), ("worker_ctas", ctypes.c_int),
                ("launches_forward", ctypes.c_int), ("launches_backward", ctypes.c_int),
                ("device_status", ctypes.c_uint), ("workspace_bytes", ctypes.c_longlong),
                ("delta_math", ctypes.c_int), ("gw_tiling", ctypes.c_int), ("delta_tiling", ctypes.c_int), ("cost", ctypes.c_int), ("activation", ctypes.c_int),
                ("shard_rank", ctypes.c_int), ("shard_count", ctypes.c_int),
                ("fused_tiling", ctypes.c_int), ("last_backward_ms", ctypes.c_float)]


def _load() -> ctypes.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_1801_04928_b200.build` "
            "(needs nvcc). There is no CPU or PyTorch fallback.")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i, ll = ctypes.c_void_p, ctypes.c_int, ctypes.c_longlong
    lib.lf_create.argtypes = [ctypes.POINTER(vp), i, i, i, i]
    lib.lf_create_widths.argtypes = [ctypes.POINTER(vp), i, ctypes.POINTER(ctypes.c_int), i, i]
    lib.lf_set_stream.argtypes = [vp, vp]
    lib.lf_set_option.argtypes = [vp, i, ll]
    lib.lf_forward.argtypes = [vp] * 6
    lib.lf_backward.argtypes = [vp] * 8
    lib.lf_backward_host.argtypes = [vp] * 8
    lib.lf_grad_w.argtypes = [vp] * 4
    lib.lf_backward_sgd.argtypes = [vp] * 5 + [ctypes.c_float] + [vp] * 3
    lib.lf_sync.argtypes = [vp]
    lib.lf_owner.argtypes = [vp, i]
    lib.lf_get_stats.argtypes = [vp, ctypes.POINTER(lf_stats)]
    lib.lf_last_cuda_error.argtypes = [vp]
    lib.lf_strerror.argtypes = [i]
    lib.lf_strerror.restype = ctypes.c_char_p
    lib.lf_version.argtypes = []
    lib.lf_destroy.argtypes = [vp]
    lib.lf_delta_step_static.argtypes = [vp, vp, vp, vp, i, vp]
    for name in EXPORTS:
        if name != "lf_strerror":
            getattr(lib, name).restype = i
    return lib


_lib = _load()


class LeapfrogError(RuntimeError):
    def __init__(self, status: int, where: str, cuda_error: int = 0):
        self.status = status
        self.cuda_error = cuda_error
        msg = f"{where}: {lf_strerror(status)} (status {status}"
        msg += f", cudaError {cuda_error})" if cuda_error else ")"
        super().__init__(msg)


def _check_tensor(t, need: int, name: str, where: str, on_device: bool = True) -> None:
    """Marshalling-side guard: a tensor handed to the library must be float32, contiguous, on the
    right side of the bus and hold at least `need` elements -- the kernels trust the context's sizes
    and would write past a buffer that is too small.  Raw addresses (ints) and None are passed on
    unchecked (None is rejected by the library itself)."""
    if t is None or isinstance(t, int):
        return
    global _FLOAT32
    dt = t.dtype
    if dt is not _FLOAT32:                   # (the dtype object is remembered: the check costs no string work)
        if str(dt) == "torch.float32":
            _FLOAT32 = dt
    if dt is _FLOAT32 and t.is_cuda == on_device and t.numel() >= need and t.is_contiguous():
        return
    problems = []
    if dt is not _FLOAT32:
        problems.append(f"dtype {dt} (float32 needed)")
    if not t.is_contiguous():
        problems.append("not contiguous")
    if bool(t.is_cuda) != on_device:
        problems.append("must be a CUDA tensor" if on_device else "must be a host tensor")
    if t.numel() < need:
        problems.append(f"{t.numel()} elements, {need} needed")
    raise LeapfrogError(LF_EINVAL, f"{where}: argument {name}: " + "; ".join(problems))


_FLOAT32 = None


def _ptr(t) -> ctypes.c_void_p:
    """Address of a tensor-like object (``data_ptr()``), an int, or None."""
    if t is None:
        return ctypes.c_void_p(None)
    if isinstance(t, int):
        return ctypes.c_void_p(t)
    return ctypes.c_void_p(t.data_ptr())


# ---- the C entry points, one to one -----------------------------------------------------------

def lf_version() -> int:
    return _lib.lf_version()


def lf_strerror(status: int) -> str:
    return _lib.lf_strerror(int(status)).decode()


def lf_create(L: int, N: int, B: int, k: int):
    """Returns (status, handle)."""
    h = ctypes.c_void_p(None)
    rc = _lib.lf_create(ctypes.byref(h), int(L), int(N), int(B), int(k))
    return rc, h


def lf_create_widths(widths, B: int, k: int):
    """``widths`` = [n_0, ..., n_L] (host ints).  Returns (status, handle)."""
    h = ctypes.c_void_p(None)
    n = [int(v) for v in widths]
    arr = (ctypes.c_int * len(n))(*n)
    rc = _lib.lf_create_widths(ctypes.byref(h), len(n) - 1, arr, int(B), int(k))
    return rc, h


def lf_set_stream(ctx, cuda_stream: int | None) -> int:
    return _lib.lf_set_stream(ctx, ctypes.c_void_p(cuda_stream or None))


def lf_set_option(ctx, key: int, value: int) -> int:
    return _lib.lf_set_option(ctx, int(key), int(value))


def lf_forward(ctx, w, b, x, z, a) -> int:
    return _lib.lf_forward(ctx, _ptr(w), _ptr(b), _ptr(x), _ptr(z), _ptr(a))


def lf_backward(ctx, w, z, a, y, delta, gw, gb) -> int:
    return _lib.lf_backward(ctx, _ptr(w), _ptr(z), _ptr(a), _ptr(y), _ptr(delta), _ptr(gw),
                            _ptr(gb))


def lf_grad_w(ctx, delta_l, a_prev, gw_l) -> int:
    return _lib.lf_grad_w(ctx, _ptr(delta_l), _ptr(a_prev), _ptr(gw_l))


def lf_backward_sgd(ctx, w, z, a, y, eta: float, delta, w_new, gb) -> int:
    return _lib.lf_backward_sgd(ctx, _ptr(w), _ptr(z), _ptr(a), _ptr(y), ctypes.c_float(eta), _ptr(delta),
                                _ptr(w_new), _ptr(gb))


def lf_backward_host(ctx, w, z, a, y, delta, gw, gb) -> int:
    return _lib.lf_backward_host(ctx, _ptr(w), _ptr(z), _ptr(a), _ptr(y), _ptr(delta),
                                 _ptr(gw), _ptr(gb))


def lf_sync(ctx) -> int:
    return _lib.lf_sync(ctx)


def lf_owner(ctx, l: int) -> int:
    return _lib.lf_owner(ctx, int(l))


def lf_get_stats(ctx):
    """Returns (status, dict)."""
    st = lf_stats()
    rc = _lib.lf_get_stats(ctx, ctypes.byref(st))
    return rc, {f: getattr(st, f) for f, _ in lf_stats._fields_}


def lf_last_cuda_error(ctx) -> int:
    return _lib.lf_last_cuda_error(ctx)


def lf_destroy(ctx) -> int:
    return _lib.lf_destroy(ctx)


def lf_delta_step_static(w_up, delta_up, a_l, delta_l, N: int, cuda_stream: int | None = None) -> int:
    """One Eq. bp2 step without a context and without any allocation (see the header).

    For processes that own all device memory through their own pool, or that cannot take the
    device-wide stall of a cudaMalloc: the kernel's scratch is a fixed array inside the
    library (N <= 4096, else LF_ECAPACITY).  Calls share that array, so do not let two of
    them overlap on the GPU.  The first call on a device loads that part of the library onto it:
    make it early, before memory is handed to a pool.  Returns the status code; the work is only
    enqueued.  Tensors (as opposed to raw addresses) are checked for dtype, device, contiguity and
    size first; a mismatch raises LeapfrogError(LF_EINVAL).
    """
    n = int(N)
    if 1 <= n <= 4096 and n % 4 == 0:
        _check_tensor(w_up, n * n, "w_up", "lf_delta_step_static")
        for name, t in (("delta_up", delta_up), ("a_l", a_l), ("delta_l", delta_l)):
            _check_tensor(t, n, name, "lf_delta_step_static")
    return _lib.lf_delta_step_static(_ptr(w_up), _ptr(delta_up), _ptr(a_l), _ptr(delta_l), int(N),
                                     ctypes.c_void_p(cuda_stream or None))


# ---- a small convenience wrapper (still marshalling only) -------------------------------------

class Leapfrog:
    """Owns one ``lf_ctx``; raises :class:`LeapfrogError` on any non-zero status."""

    def __init__(self, L: int, N: int, B: int = 1, k: int = 1, stream: int | None = None, widths=None):
        """``widths`` = [n_0, ..., n_L] selects lf_create_widths (L and N are then taken from it)."""
        if widths is not None:
            rc, self._h = lf_create_widths(widths, B, k)
            L, N = len(widths) - 1, max(int(v) for v in widths)
        else:
            rc, self._h = lf_create(L, N, B, k)
        if rc != LF_OK:
            self._h = None
            raise LeapfrogError(rc, "lf_create_widths" if widths is not None else "lf_create")
        self.L, self.N, self.B, self.k = L, N, B, k
        n = [int(v) for v in widths] if widths is not None else [int(N)] * (int(L) + 1)
        n_w = sum(n[l] * n[l - 1] for l in range(1, len(n)))
        n_h = sum(n[1:])
        # elements every argument must hold (w, gw | b, gb | z, delta | a | x | y)
        self._need = dict(w=n_w, gw=n_w, w_new=n_w, b=n_h, gb=n_h, z=B * n_h, delta=B * n_h,
                          a=B * sum(n), x=B * n[0], y=B * n[-1], layer_w=int(N) * int(N), layer_v=B * int(N))
        if stream is not None:
            self.set_stream(stream)

    def _args(self, where: str, on_device: bool = True, **tensors):
        for name, t in tensors.items():
            _check_tensor(t, self._need[name], name, where, on_device)

    def _check(self, rc: int, where: str):
        if rc != LF_OK:
            raise LeapfrogError(rc, where, lf_last_cuda_error(self._h))

    def set_stream(self, cuda_stream: int | None):
        self._check(lf_set_stream(self._h, cuda_stream), "lf_set_stream")

    def set_option(self, key: int, value: int):
        self._check(lf_set_option(self._h, key, value), "lf_set_option")

    def forward(self, w, b, x, z, a):
        self._args("lf_forward", w=w, b=b, x=x, z=z, a=a)
        self._check(lf_forward(self._h, w, b, x, z, a), "lf_forward")

    def backward(self, w, z, a, y, delta, gw, gb):
        self._args("lf_backward", w=w, z=z, a=a, y=y, delta=delta, gw=gw, gb=gb)
        self._check(lf_backward(self._h, w, z, a, y, delta, gw, gb), "lf_backward")

    def grad_w(self, delta_l, a_prev, gw_l):
        for name, t, need in (("delta_l", delta_l, "layer_v"), ("a_prev", a_prev, "layer_v"), ("gw_l", gw_l, "layer_w")):
            _check_tensor(t, self._need[need], name, "lf_grad_w")
        self._check(lf_grad_w(self._h, delta_l, a_prev, gw_l), "lf_grad_w")

    def backward_sgd(self, w, z, a, y, eta, delta, w_new, gb):
        self._args("lf_backward_sgd", w=w, z=z, a=a, y=y, delta=delta, w_new=w_new, gb=gb)
        self._check(lf_backward_sgd(self._h, w, z, a, y, eta, delta, w_new, gb), "lf_backward_sgd")

    def backward_host(self, w, z, a, y, delta, gw, gb):
        self._args("lf_backward_host", on_device=False, w=w, z=z, a=a, y=y, delta=delta, gw=gw, gb=gb)
        self._check(lf_backward_host(self._h, w, z, a, y, delta, gw, gb), "lf_backward_host")

    def sync(self):
        self._check(lf_sync(self._h), "lf_sync")

    def owner(self, l: int) -> int:
        return lf_owner(self._h, l)

    def stats(self) -> dict:
        rc, d = lf_get_stats(self._h)
        self._check(rc, "lf_get_stats")
        return d

    def close(self):
        if self._h is not None:
            lf_destroy(self._h)
            self._h = None

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
