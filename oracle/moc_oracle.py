"""ctypes front end of the CPU oracle (test infrastructure, not the product).

Only the tests, the smoke check and the benchmark's CPU-baseline leg import this
module.  It compiles ``moc_oracle.c`` with gcc on first use and marshals numpy
float64 arrays; every piece of arithmetic lives in the C file (the functions here only compose
the C routines: a selection rule applied to the gate projection, then the layer's remaining steps).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "moc_oracle.c")
_LIB = os.path.join(_HERE, "libmoc_oracle.so")
_lock = threading.Lock()
_lib = None

_c_double_p = ctypes.POINTER(ctypes.c_double)
_c_float_p = ctypes.POINTER(ctypes.c_float)
_c_i32_p = ctypes.POINTER(ctypes.c_int32)


def build(force: bool = False) -> str:
    """Compile the oracle into a shared object next to its source; returns the path."""
    with _lock:
        stale = force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if stale:
            tmp = _LIB + ".tmp.%d" % os.getpid()
            cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
                   "-Wall", "-Wextra", "-o", tmp, _SRC, "-lm"]
            subprocess.run(cmd, check=True)
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        lib.moc_oracle_silu.restype = ctypes.c_double
        lib.moc_oracle_silu.argtypes = [ctypes.c_double]
        lib.moc_oracle_dsilu.restype = ctypes.c_double
        lib.moc_oracle_dsilu.argtypes = [ctypes.c_double]
        for name in ("moc_oracle_macs_dense", "moc_oracle_saved_elems_ffn", "moc_oracle_saved_elems_ffn_gcp",
                     "moc_oracle_saved_elems_moc", "moc_oracle_saved_elems_moc_gcp"):
            getattr(lib, name).restype = ctypes.c_int64
            getattr(lib, name).argtypes = [ctypes.c_int64, ctypes.c_int64]
        lib.moc_oracle_macs_moc.restype = ctypes.c_int64
        lib.moc_oracle_macs_moc.argtypes = [ctypes.c_int64] * 3
        lib.moc_oracle_num_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def _f64(a, shape=None):
    a = np.ascontiguousarray(np.asarray(a, dtype=np.float64))
    if shape is not None and tuple(a.shape) != tuple(shape):
        raise ValueError(f"expected shape {tuple(shape)}, got {tuple(a.shape)}")
    return a


def _i32(a, shape=None):
    a = np.ascontiguousarray(np.asarray(a, dtype=np.int32))
    if shape is not None and tuple(a.shape) != tuple(shape):
        raise ValueError(f"expected shape {tuple(shape)}, got {tuple(a.shape)}")
    return a


def _p(a):
    if a is None:
        return None
    if a.dtype == np.float64:
        return a.ctypes.data_as(_c_double_p)
    if a.dtype == np.float32:
        return a.ctypes.data_as(_c_float_p)
    if a.dtype == np.int32:
        return a.ctypes.data_as(_c_i32_p)
    raise TypeError(a.dtype)


def _check(rc, what):
    if rc != 0:
        raise RuntimeError(f"{what} failed with code {rc}")


def num_threads() -> int:
    return int(_load().moc_oracle_num_threads())


def silu(g: float) -> float:
    return float(_load().moc_oracle_silu(float(g)))


def dsilu(g: float) -> float:
    return float(_load().moc_oracle_dsilu(float(g)))


def macs_dense(d, F):
    return int(_load().moc_oracle_macs_dense(d, F))


def macs_moc(d, F, K):
    return int(_load().moc_oracle_macs_moc(d, F, K))


def saved_elems(kind: str, d: int, n: int) -> int:
    """kind in {'ffn','ffn_gcp'} with n = d_ff, or {'moc','moc_gcp'} with n = K."""
    return int(getattr(_load(), "moc_oracle_saved_elems_" + kind)(d, n))


def topk(gate, K: int, F: int | None = None):
    """Row-wise Top-K channel sets (ascending) of a [rows, ld] array; fp32 input is compared as fp32."""
    gate = np.ascontiguousarray(gate)
    if gate.ndim != 2:
        raise ValueError("gate must be 2-D")
    rows, ld = gate.shape
    F = ld if F is None else F
    idx = np.empty((rows, K), dtype=np.int32)
    lib = _load()
    if gate.dtype == np.float32:
        rc = lib.moc_oracle_topk_f32(ctypes.c_int64(rows), ctypes.c_int32(F), ctypes.c_int64(ld),
                                     ctypes.c_int32(K), _p(gate), _p(idx))
    else:
        gate = _f64(gate)
        rc = lib.moc_oracle_topk(ctypes.c_int64(rows), ctypes.c_int32(F), ctypes.c_int64(ld),
                                 ctypes.c_int32(K), _p(gate), _p(idx))
    _check(rc, "moc_oracle_topk")
    return idx


def topk_grouped(gate, group: int = 8, keep: int = 2, F: int | None = None):
    """Grouped selection (the a:b form, keep of every `group` consecutive channels; Section 4 and Theorem 1):
    [rows, keep * F / group] channel indices, ascending."""
    gate = _f64(np.ascontiguousarray(gate))
    if gate.ndim != 2:
        raise ValueError("gate must be 2-D")
    rows, ld = gate.shape
    F = ld if F is None else F
    if F % group:
        raise ValueError("F must be a multiple of the group size")
    idx = np.empty((rows, F // group * keep), dtype=np.int32)
    rc = _load().moc_oracle_topk_grouped(ctypes.c_int64(rows), ctypes.c_int32(F), ctypes.c_int64(ld),
                                         ctypes.c_int32(group), ctypes.c_int32(keep), _p(gate), _p(idx))
    _check(rc, "moc_oracle_topk_grouped")
    return idx


def gate_projection(x, w_gate, F: int | None = None):
    """G = X W_gate (Eq. (Moc-1)) for the first F channels, [T, F] float64."""
    x, w_gate = _f64(x), _f64(w_gate)
    F = w_gate.shape[0] if F is None else F
    T, d = x.shape
    if w_gate.ndim != 2 or w_gate.shape[1] != d or w_gate.shape[0] < F:
        raise ValueError("weight shape")
    g = np.empty((T, F))
    _check(_load().moc_oracle_gate_projection(ctypes.c_int64(T), ctypes.c_int32(d), ctypes.c_int32(F), _p(x),
                                              _p(w_gate), _p(g)), "moc_oracle_gate_projection")
    return g


def silu_rows(g):
    """SiLU (Eq. (silu)) of every element, float64."""
    g = _f64(g)
    s = np.empty_like(g)
    _check(_load().moc_oracle_silu_rows(ctypes.c_int64(g.size), _p(g), _p(s)), "moc_oracle_silu_rows")
    return s


def forward_post_silu(x, w_gate, w_up, w_down, K: int, F: int | None = None):
    """The layer with the Top-K operator placed after the activation (Section 6.5, "Effect of top-K position"): the
    mask keeps the K largest SiLU(g) of a token (equal values: the lower channel); everything else as in `forward`.
    Returns forward_given_idx's dictionary plus idx, g (gate values) and s (their SiLU: the selection keys)."""
    G = gate_projection(x, w_gate, F)
    S = silu_rows(G)
    idx = topk(S, K)
    res = forward_given_idx(x, w_gate, w_up, w_down, idx, F)
    res.update(idx=idx, g=G, s=S)
    return res


def rmsnorm(x, weight, eps: float):
    """y = x / RMS(x) . g per row, RMS(x) = sqrt(mean(x^2) + eps) (Section 2, item "RMSNorm"); [T, d] float64."""
    x, weight = _f64(x), _f64(weight)
    T, d = x.shape
    assert weight.shape == (d,)
    y = np.empty_like(x)
    _check(_load().moc_oracle_rmsnorm(ctypes.c_int64(T), ctypes.c_int32(d), _p(x), _p(weight), ctypes.c_double(eps),
                                      _p(y)), "moc_oracle_rmsnorm")
    return y


def residual(x, y):
    """Z = X + Y (Section 2, item "Residual connections")."""
    x, y = _f64(x), _f64(y)
    assert x.shape == y.shape
    z = np.empty_like(x)
    _check(_load().moc_oracle_residual(ctypes.c_int64(x.size), _p(x), _p(y), _p(z)), "moc_oracle_residual")
    return z


def decode_block(h, rms_weight, eps: float, w_gate, w_up, w_down, K: int, F: int | None = None, store=None):
    """The FFN half of a pre-norm Transformer layer (Section 2, "LLM structure"): out = h + MoC_FFN(RMSNorm(h)).

    `store`: what writing the normalised activations in the storage type does to them (the paper runs in BF16:
    the rounding to bf16), a callable on float64 arrays; None keeps them in float64.  Returns (out, x, picks) with x
    the activations the layer saw and picks the layer's forward dictionary.
    """
    x = rmsnorm(h, rms_weight, eps)
    if store is not None:
        x = _f64(store(x))
    f = forward(x, w_gate, w_up, w_down, K, F, want_g=True)
    return residual(h, f["out"]), x, f


def forward_grouped(x, w_gate, w_up, w_down, group: int = 8, keep: int = 2, F: int | None = None):
    """The layer with the grouped mask: gate projection, grouped selection, then the steps of the layer on the
    selected channels.  Returns dict(out, idx, gval, uval, g)."""
    g = gate_projection(x, w_gate, F)
    idx = topk_grouped(g, group, keep)
    res = forward_given_idx(x, w_gate, w_up, w_down, idx, F=F)
    res["idx"], res["g"] = idx, g
    return res


def forward(x, w_gate, w_up, w_down, K: int, F: int | None = None, want_g: bool = False):
    """Returns dict(out, idx, gval, uval[, g]); weights are [>=F, d] channel-major."""
    x = _f64(x)
    T, d = x.shape
    w_gate, w_up, w_down = _f64(w_gate), _f64(w_up), _f64(w_down)
    F = w_gate.shape[0] if F is None else F
    for w in (w_gate, w_up, w_down):
        if w.ndim != 2 or w.shape[1] != d or w.shape[0] < F:
            raise ValueError("weight shape")
    out = np.empty((T, d))
    idx = np.empty((T, K), dtype=np.int32)
    gval = np.empty((T, K))
    uval = np.empty((T, K))
    g = np.empty((T, F)) if want_g else None
    rc = _load().moc_oracle_forward(ctypes.c_int64(T), ctypes.c_int32(d), ctypes.c_int32(F), ctypes.c_int32(K),
                                    _p(x), _p(w_gate), _p(w_up), _p(w_down), _p(out), _p(idx), _p(gval),
                                    _p(uval), _p(g))
    _check(rc, "moc_oracle_forward")
    res = dict(out=out, idx=idx, gval=gval, uval=uval)
    if want_g:
        res["g"] = g
    return res


def forward_given_idx(x, w_gate, w_up, w_down, idx, F: int | None = None):
    x = _f64(x)
    T, d = x.shape
    w_gate, w_up, w_down = _f64(w_gate), _f64(w_up), _f64(w_down)
    F = w_gate.shape[0] if F is None else F
    idx = _i32(idx)
    if idx.ndim != 2 or idx.shape[0] != T:
        raise ValueError("idx shape")
    K = idx.shape[1]
    out = np.empty((T, d))
    gval = np.empty((T, K))
    uval = np.empty((T, K))
    rc = _load().moc_oracle_forward_given_idx(ctypes.c_int64(T), ctypes.c_int32(d), ctypes.c_int32(F),
                                              ctypes.c_int32(K), _p(x), _p(w_gate), _p(w_up), _p(w_down),
                                              _p(idx), _p(out), _p(gval), _p(uval))
    _check(rc, "moc_oracle_forward_given_idx")
    return dict(out=out, idx=idx, gval=gval, uval=uval)


def backward(x, w_gate, w_up, w_down, idx, gval, uval, grad_out, F: int | None = None,
             want=("x", "w_gate", "w_up", "w_down")):
    x = _f64(x)
    T, d = x.shape
    w_gate, w_up, w_down = _f64(w_gate), _f64(w_up), _f64(w_down)
    F = w_gate.shape[0] if F is None else F
    idx = _i32(idx)
    K = idx.shape[1]
    gval, uval = _f64(gval, (T, K)), _f64(uval, (T, K))
    grad_out = _f64(grad_out, (T, d))
    gx = np.empty((T, d)) if "x" in want else None
    gwg = np.empty((F, d)) if "w_gate" in want else None
    gwu = np.empty((F, d)) if "w_up" in want else None
    gwd = np.empty((F, d)) if "w_down" in want else None
    rc = _load().moc_oracle_backward(ctypes.c_int64(T), ctypes.c_int32(d), ctypes.c_int32(F), ctypes.c_int32(K),
                                     _p(x), _p(w_gate), _p(w_up), _p(w_down), _p(idx), _p(gval), _p(uval),
                                     _p(grad_out), _p(gx), _p(gwg), _p(gwu), _p(gwd))
    _check(rc, "moc_oracle_backward")
    return dict(grad_x=gx, grad_w_gate=gwg, grad_w_up=gwu, grad_w_down=gwd)


def backward_weight_rows(x, w_down, idx, gval, uval, grad_out, rows, F: int):
    """Rows `rows` of (grad_w_gate, grad_w_up, grad_w_down), each [len(rows), d]."""
    x = _f64(x)
    T, d = x.shape
    w_down = _f64(w_down)
    idx = _i32(idx)
    K = idx.shape[1]
    gval, uval = _f64(gval, (T, K)), _f64(uval, (T, K))
    grad_out = _f64(grad_out, (T, d))
    rows = _i32(rows)
    n = rows.shape[0]
    a, b, c = np.empty((n, d)), np.empty((n, d)), np.empty((n, d))
    rc = _load().moc_oracle_backward_weight_rows(ctypes.c_int64(T), ctypes.c_int32(d), ctypes.c_int32(F),
                                                 ctypes.c_int32(K), _p(x), _p(w_down), _p(idx), _p(gval),
                                                 _p(uval), _p(grad_out), ctypes.c_int32(n), _p(rows), _p(a),
                                                 _p(b), _p(c))
    _check(rc, "moc_oracle_backward_weight_rows")
    return dict(grad_w_gate=a, grad_w_up=b, grad_w_down=c)
