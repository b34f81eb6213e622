"""ctypes loader for the float64 CPU oracle in ``lf_oracle.c``.

TEST INFRASTRUCTURE, NOT THE PRODUCT: only the tests, the smoke check and the benchmark's
CPU-baseline leg may import this module.  It holds no arithmetic of its own -- every number
it returns is computed by the C file beside it (arXiv 1801.04928, Section 2 Eq. x, z, a,
bp1-bp4 and Section 3 Algorithm 1; the readings of the paper are listed in that file's
header).  It does not import, and is not imported by, the CUDA package.

The C file is compiled twice: ``liblfo_f64.so`` takes double weights (finite-difference
pins), ``liblfo_f32.so`` takes float weights and promotes them element by element (large
networks).  The flavour is chosen from ``w.dtype``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "lf_oracle.c")
_LOCK = threading.Lock()
_LIBS: dict[str, ctypes.CDLL] = {}

_c_dp = ctypes.POINTER(ctypes.c_double)
_c_ip = ctypes.POINTER(ctypes.c_int)


def build(force: bool = False) -> dict[str, str]:
    """Compile both flavours of the oracle with gcc (no fast-math, no FMA contraction)."""
    out = {}
    for tag, ctype in (("f64", "double"), ("f32", "float")):
        so = os.path.join(_HERE, f"liblfo_{tag}.so")
        stale = (not os.path.exists(so)) or os.path.getmtime(so) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = so + f".tmp{os.getpid()}"
            cmd = ["gcc", "-std=c99", "-O2", "-fPIC", "-shared", "-pthread",
                   "-ffp-contract=off", "-fno-fast-math", f"-DLFO_W_T={ctype}",
                   "-o", tmp, _SRC, "-lm"]
            subprocess.run(cmd, check=True)
            os.replace(tmp, so)
        out[tag] = so
    return out


def _lib(tag: str) -> ctypes.CDLL:
    with _LOCK:
        if tag not in _LIBS:
            paths = build()
            lib = ctypes.CDLL(paths[tag])
            wp = ctypes.c_void_p
            i = ctypes.c_int
            lib.lfo_weight_bytes.restype = i
            lib.lfo_sigma.restype = ctypes.c_double
            lib.lfo_sigma.argtypes = [ctypes.c_double]
            lib.lfo_sigma_prime.restype = ctypes.c_double
            lib.lfo_sigma_prime.argtypes = [ctypes.c_double]
            lib.lfo_forward.restype = None
            lib.lfo_forward.argtypes = [i, i, i, wp, _c_dp, _c_dp, _c_dp, _c_dp]
            lib.lfo_cost.restype = ctypes.c_double
            lib.lfo_cost.argtypes = [i, i, i, _c_dp, _c_dp]
            lib.lfo_output_error.restype = None
            lib.lfo_output_error.argtypes = [i, i, _c_dp, _c_dp, _c_dp, _c_dp]
            lib.lfo_delta_step.restype = None
            lib.lfo_delta_step.argtypes = [i, i, wp, _c_dp, _c_dp, _c_dp]
            lib.lfo_grad_b.restype = None
            lib.lfo_grad_b.argtypes = [i, i, _c_dp, _c_dp]
            lib.lfo_grad_w.restype = None
            lib.lfo_grad_w.argtypes = [i, i, _c_dp, _c_dp, _c_dp]
            lib.lfo_grad_w_entry.restype = ctypes.c_double
            lib.lfo_grad_w_entry.argtypes = [i, i, _c_dp, _c_dp, i, i]
            lib.lfo_backward_sequential.restype = None
            lib.lfo_backward_sequential.argtypes = [i, i, i, wp, _c_dp, _c_dp, _c_dp, _c_dp,
                                                    _c_dp, _c_dp]
            lib.lfo_backward_leapfrog.restype = i
            lib.lfo_backward_leapfrog.argtypes = [i, i, i, i, wp, _c_dp, _c_dp, _c_dp, _c_dp,
                                                  _c_dp, _c_dp, _c_ip, _c_ip,
                                                  ctypes.POINTER(ctypes.c_longlong), i]
            lib.lfo_cost_cross_entropy.restype = ctypes.c_double
            lib.lfo_cost_cross_entropy.argtypes = [i, i, i, _c_dp, _c_dp]
            lib.lfo_output_error_cross_entropy.restype = None
            lib.lfo_output_error_cross_entropy.argtypes = [i, i, _c_dp, _c_dp, _c_dp, _c_dp]
            lib.lfo_backward_sequential_cross_entropy.restype = None
            lib.lfo_backward_sequential_cross_entropy.argtypes = [i, i, i, wp, _c_dp, _c_dp, _c_dp, _c_dp,
                                                                  _c_dp, _c_dp]
            lib.lfo_set_activation.restype = i
            lib.lfo_set_activation.argtypes = [i]
            lib.lfo_set_activation(_ACTIVATION)
            lib.lfo_forward_widths.restype = None
            lib.lfo_forward_widths.argtypes = [i, _c_ip, i, wp, _c_dp, _c_dp, _c_dp, _c_dp]
            lib.lfo_backward_widths.restype = None
            lib.lfo_backward_widths.argtypes = [i, _c_ip, i, i, wp, _c_dp, _c_dp, _c_dp, _c_dp, _c_dp, _c_dp]
            lib.lfo_backward_shard.restype = i
            lib.lfo_backward_shard.argtypes = [i, i, i, i, i, wp, _c_dp, _c_dp, _c_dp, _c_dp, _c_dp, _c_dp, _c_ip]
            lib.lfo_sgd_step.restype = None
            lib.lfo_sgd_step.argtypes = [i, i, wp, _c_dp, ctypes.c_double, _c_dp]
            assert lib.lfo_weight_bytes() == (8 if tag == "f64" else 4)
            _LIBS[tag] = lib
        return _LIBS[tag]


ACTIVATIONS = {"sigmoid": 0, "tanh": 1, "relu": 2}
_ACTIVATION = 0


def set_activation(name: str) -> None:
    """Choose the activation function of every later pass (both compiled flavours)."""
    global _ACTIVATION
    _ACTIVATION = ACTIVATIONS[name]
    for tag in ("f64", "f32"):
        if _lib(tag).lfo_set_activation(_ACTIVATION) != 0:
            raise ValueError(name)


class activation:
    """``with activation("tanh"): ...`` -- the sigmoid is restored afterwards."""

    def __init__(self, name: str):
        self.name = name

    def __enter__(self):
        set_activation(self.name)
        return self

    def __exit__(self, *exc):
        set_activation("sigmoid")


def _w(w: np.ndarray):
    """Weights stay in their own dtype (float32 or float64); returns (lib, array, pointer)."""
    if w.dtype == np.float32:
        tag = "f32"
    elif w.dtype == np.float64:
        tag = "f64"
    else:
        raise TypeError("weights must be float32 or float64")
    w = np.ascontiguousarray(w)
    return _lib(tag), w, ctypes.c_void_p(w.ctypes.data)


def _d(x) -> np.ndarray:
    return np.ascontiguousarray(x, dtype=np.float64)


def _p(x: np.ndarray):
    return x.ctypes.data_as(_c_dp)


def sigma(t: float) -> float:
    return _lib("f64").lfo_sigma(float(t))


def sigma_prime(t: float) -> float:
    return _lib("f64").lfo_sigma_prime(float(t))


def forward(w, b, x):
    """Eq. x, z, a.  w[L,N,N], b[L,N], x[B,N] -> z[L,B,N], a[L+1,B,N] (float64)."""
    lib, w, wp = _w(w)
    L, N, _ = w.shape
    b = _d(b)
    x = _d(x).reshape(-1, N)
    B = x.shape[0]
    z = np.empty((L, B, N), dtype=np.float64)
    a = np.empty((L + 1, B, N), dtype=np.float64)
    lib.lfo_forward(L, N, B, wp, _p(b), _p(x), _p(z), _p(a))
    return z, a


def cost(a, y, cross_entropy: bool = False) -> float:
    """C from the activations of a forward pass: 1/2 sum_b ||a^L_b - y_b||^2, or the
    cross-entropy of the sigmoid outputs."""
    a = _d(a)
    Lp1, B, N = a.shape
    y = _d(y).reshape(B, N)
    fn = _lib("f64").lfo_cost_cross_entropy if cross_entropy else _lib("f64").lfo_cost
    return fn(Lp1 - 1, N, B, _p(a), _p(y))


def output_error(aL, y, zL, cross_entropy: bool = False):
    """Eq. bp1 under either cost."""
    aL, y, zL = _d(aL), _d(y), _d(zL)
    B, N = aL.shape
    out = np.empty((B, N), dtype=np.float64)
    fn = _lib("f64").lfo_output_error_cross_entropy if cross_entropy else _lib("f64").lfo_output_error
    fn(N, B, _p(aL), _p(y), _p(zL), _p(out))
    return out


def delta_step(w_up, delta_up, z_l):
    """Eq. bp2 at one layer.  w_up = w^{l+1} [N,N]; delta_up, z_l: [B,N]."""
    lib, w_up, wp = _w(w_up)
    delta_up, z_l = _d(delta_up), _d(z_l)
    B, N = delta_up.shape
    out = np.empty((B, N), dtype=np.float64)
    lib.lfo_delta_step(N, B, wp, _p(delta_up), _p(z_l), _p(out))
    return out


def grad_b(delta_l):
    """Eq. bp3 summed over the samples."""
    delta_l = _d(delta_l)
    B, N = delta_l.shape
    out = np.empty((N,), dtype=np.float64)
    _lib("f64").lfo_grad_b(N, B, _p(delta_l), _p(out))
    return out


def grad_w(delta_l, a_prev):
    """Eq. bp4 summed over the samples: one full N x N layer."""
    delta_l, a_prev = _d(delta_l), _d(a_prev)
    B, N = delta_l.shape
    out = np.empty((N, N), dtype=np.float64)
    _lib("f64").lfo_grad_w(N, B, _p(delta_l), _p(a_prev), _p(out))
    return out


def grad_w_entry(delta_l, a_prev, j: int, k: int) -> float:
    """One entry of Eq. bp4."""
    delta_l, a_prev = _d(delta_l), _d(a_prev)
    B, N = delta_l.shape
    return _lib("f64").lfo_grad_w_entry(N, B, _p(delta_l), _p(a_prev), int(j), int(k))


def backward_sequential(w, z, a, y, want_gw: bool = True, cross_entropy: bool = False):
    """Plain backpropagation under the quadratic (default) or the cross-entropy cost.
    Returns delta[L,B,N], gw[L,N,N] (or None), gb[L,N]."""
    lib, w, wp = _w(w)
    L, N, _ = w.shape
    z, a = _d(z), _d(a)
    B = z.shape[1]
    y = _d(y).reshape(B, N)
    delta = np.empty((L, B, N), dtype=np.float64)
    gb = np.empty((L, N), dtype=np.float64)
    gw = np.empty((L, N, N), dtype=np.float64) if want_gw else None
    fn = lib.lfo_backward_sequential_cross_entropy if cross_entropy else lib.lfo_backward_sequential
    fn(L, N, B, wp, _p(z), _p(a), _p(y), _p(delta), _p(gw) if want_gw else None, _p(gb))
    return delta, gw, gb


def sgd_step(w, gw, eta: float):
    """w - eta * gw for all L weight matrices (float64); not in the paper, see the C file."""
    lib, w, wp = _w(w)
    L, N, _ = w.shape
    gw = _d(gw)
    out = np.empty((L, N, N), dtype=np.float64)
    lib.lfo_sgd_step(L, N, wp, _p(gw), float(eta), _p(out))
    return out


def backward_leapfrog(w, z, a, y, k: int, want_gw: bool = True, threads: bool = True):
    """Algorithm 1 taken literally with k threads.

    Returns (delta, gw or None, gb, writer[L], writes[L], bp2_total): ``writer`` names the
    thread that saved each layer (-1 = the parent), ``writes`` counts the saves per layer.
    """
    lib, w, wp = _w(w)
    L, N, _ = w.shape
    z, a = _d(z), _d(a)
    B = z.shape[1]
    y = _d(y).reshape(B, N)
    delta = np.full((L, B, N), np.nan, dtype=np.float64)
    gb = np.full((L, N), np.nan, dtype=np.float64)
    gw = np.full((L, N, N), np.nan, dtype=np.float64) if want_gw else None
    writer = np.zeros((L,), dtype=np.int32)
    writes = np.zeros((L,), dtype=np.int32)
    total = ctypes.c_longlong(0)
    rc = lib.lfo_backward_leapfrog(L, N, B, int(k), wp, _p(z), _p(a), _p(y), _p(delta),
                                   _p(gw) if want_gw else None, _p(gb),
                                   writer.ctypes.data_as(_c_ip), writes.ctypes.data_as(_c_ip),
                                   ctypes.byref(total), 1 if threads else 0)
    if rc != 0:
        raise ValueError("lfo_backward_leapfrog: invalid sizes")
    return delta, gw, gb, writer, writes, total.value


# ---- layers of different widths -----------------------------------------------------------------
# Arrays are flat: each is the concatenation of its per-layer blocks (see the C file).  `widths`
# is [n_0, ..., n_L]; `split` cuts a flat array back into per-layer views.

def _widths(widths):
    n = np.ascontiguousarray(widths, dtype=np.int32)
    if n.ndim != 1 or n.size < 2 or (n < 1).any():
        raise ValueError("widths must be [n_0, ..., n_L], all >= 1")
    return n, n.ctypes.data_as(_c_ip)


def sizes_widths(widths, B: int) -> dict[str, int]:
    """Element counts of the flat arrays of a network with these widths."""
    n = [int(v) for v in widths]
    hidden = sum(n[1:])
    return {"w": sum(n[l] * n[l - 1] for l in range(1, len(n))), "b": hidden, "z": B * hidden,
            "a": B * sum(n), "x": B * n[0], "y": B * n[-1]}


def split(flat, widths, kind: str, B: int = 1):
    """Per-layer views of a flat array: kind 'w' -> [n_l, n_{l-1}], 'b' -> [n_l], 'z' -> [B, n_l]
    (l = 1..L), 'a' -> [B, n_l] (l = 0..L)."""
    n = [int(v) for v in widths]
    out, pos = [], 0
    for l in range(0 if kind == "a" else 1, len(n)):
        shape = {"w": (n[l], n[l - 1]) if l else None, "b": (n[l],), "z": (B, n[l]), "a": (B, n[l])}[kind]
        cnt = int(np.prod(shape))
        out.append(flat[pos:pos + cnt].reshape(shape))
        pos += cnt
    assert pos == flat.size
    return out


def forward_widths(widths, w, b, x):
    """Eq. x, z, a for layer widths n_0..n_L; flat w, b, x in, flat float64 z, a out."""
    n, npnt = _widths(widths)
    lib, w, wp = _w(w)
    B = np.asarray(x).size // int(n[0])
    sz = sizes_widths(n, B)
    assert w.size == sz["w"] and np.asarray(b).size == sz["b"] and np.asarray(x).size == sz["x"]
    b, x = _d(b).ravel(), _d(x).ravel()
    z = np.empty(sz["z"], dtype=np.float64)
    a = np.empty(sz["a"], dtype=np.float64)
    lib.lfo_forward_widths(n.size - 1, npnt, B, wp, _p(b), _p(x), _p(z), _p(a))
    return z, a


def backward_widths(widths, w, z, a, y, want_gw: bool = True, cross_entropy: bool = False):
    """Eq. bp1-bp4 for layer widths n_0..n_L; flat arrays; returns flat delta, gw (or None), gb."""
    n, npnt = _widths(widths)
    lib, w, wp = _w(w)
    B = np.asarray(y).size // int(n[-1])
    sz = sizes_widths(n, B)
    z, a, y = _d(z).ravel(), _d(a).ravel(), _d(y).ravel()
    assert w.size == sz["w"] and z.size == sz["z"] and a.size == sz["a"] and y.size == sz["y"]
    delta = np.empty(sz["z"], dtype=np.float64)
    gb = np.empty(sz["b"], dtype=np.float64)
    gw = np.empty(sz["w"], dtype=np.float64) if want_gw else None
    lib.lfo_backward_widths(n.size - 1, npnt, B, 1 if cross_entropy else 0, wp, _p(z), _p(a), _p(y),
                            _p(delta), _p(gw) if want_gw else None, _p(gb))
    return delta, gw, gb


def backward_shard(w, z, a, y, S: int, r: int, want_gw: bool = True):
    """GPU r's pass of the schedule on S GPUs: the whole delta chain, Eq. bp3/bp4 only at the layers
    with (L - l) mod S = r.  Returns (delta, gw or None, gb, wrote[L]); layers of other shards hold NaN
    in gw and gb."""
    lib, w, wp = _w(w)
    L, N, _ = w.shape
    z, a = _d(z), _d(a)
    B = z.shape[1]
    y = _d(y).reshape(B, N)
    delta = np.full((L, B, N), np.nan, dtype=np.float64)
    gb = np.full((L, N), np.nan, dtype=np.float64)
    gw = np.full((L, N, N), np.nan, dtype=np.float64) if want_gw else None
    wrote = np.zeros((L,), dtype=np.int32)
    rc = lib.lfo_backward_shard(L, N, B, int(S), int(r), wp, _p(z), _p(a), _p(y), _p(delta),
                                _p(gw) if want_gw else None, _p(gb), wrote.ctypes.data_as(_c_ip))
    if rc != 0:
        raise ValueError("lfo_backward_shard: invalid sizes")
    return delta, gw, gb, wrote
