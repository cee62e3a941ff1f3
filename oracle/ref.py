"""ctypes front end of the fp64 CPU oracle in ``linattn_ref.c``.

TEST INFRASTRUCTURE ONLY: the tests, the smoke check and the benchmark's CPU
baseline may import this; the CUDA library and its Python binding never do.
It holds no arithmetic of its own: arguments are marshalled to the C routines,
which restate Eq. 5 (both forms) and Eq. 6 in double precision.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "linattn_ref.c")
_LIB = os.path.join(_HERE, "liblinattn_ref.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc if the shared object is missing or stale."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.run(
            ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"],
            check=True,
        )
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        fp = ctypes.POINTER(ctypes.c_float)
        dp = ctypes.POINTER(ctypes.c_double)
        lp = ctypes.POINTER(ctypes.c_long)
        lib.linattn_ref_threads.restype = ctypes.c_int
        lib.linattn_ref_phi.argtypes = [fp, fp, ctypes.c_long, ctypes.c_int, dp]
        lib.linattn_ref_quadratic.argtypes = [fp, fp, fp, fp, fp, ctypes.c_long, ctypes.c_int,
                                              ctypes.c_long, ctypes.c_int, ctypes.c_int,
                                              lp, ctypes.c_long, dp]
        lib.linattn_ref_linear.argtypes = [fp, fp, fp, fp, fp, ctypes.c_long, ctypes.c_int,
                                           ctypes.c_long, ctypes.c_int, ctypes.c_int,
                                           lp, ctypes.c_long, dp, dp, dp]
        lib.linattn_ref_softmax.argtypes = [fp, fp, fp, ctypes.c_long, ctypes.c_long, ctypes.c_int, ctypes.c_double,
                                            lp, ctypes.c_long, dp]
        lib.linattn_ref_mix.argtypes = [dp, dp, ctypes.c_long, ctypes.c_double, dp]
        lib.linattn_ref_backward.argtypes = [fp, fp, fp, fp, fp, fp, ctypes.c_long, ctypes.c_int, ctypes.c_long,
                                             ctypes.c_int, ctypes.c_int, dp, dp, dp, dp, dp]
        lib.linattn_ref_backward_mixed.argtypes = [fp, fp, fp, fp, fp, fp, ctypes.c_double, fp, ctypes.c_long, ctypes.c_int,
                                                   ctypes.c_long, ctypes.c_int, ctypes.c_int, dp, dp, dp, dp, dp, dp, dp]
        lib.linattn_ref_relu_backward.argtypes = [fp, fp, fp, fp, ctypes.c_long, ctypes.c_long, ctypes.c_int, dp, dp, dp]
        lib.linattn_ref_relu_quadratic.argtypes = [fp, fp, fp, ctypes.c_long, ctypes.c_long, ctypes.c_int, lp, ctypes.c_long, dp]
        lib.linattn_ref_relu_linear.argtypes = [fp, fp, fp, ctypes.c_long, ctypes.c_long, ctypes.c_int, lp, ctypes.c_long,
                                                dp, dp, dp]
        _lib = lib
    return _lib


def threads() -> int:
    """Threads the oracle's parallel loops use on this host."""
    return int(_load().linattn_ref_threads())


def _f32(a) -> np.ndarray:
    """Widen any array-like (numpy, or a CPU torch tensor of any float type) to contiguous float32.

    Every fp32 and bf16 value is exactly representable in float32, so nothing is rounded here."""
    if hasattr(a, "detach"):
        a = a.detach().cpu().float().numpy()
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a


def _ptr(a, ty):
    return a.ctypes.data_as(ctypes.POINTER(ty)) if a is not None else None


def phi(x, W) -> np.ndarray:
    """Eq. 6 on rows of ``x`` [n, d] with ``W`` [d, d/2]; returns float64 [n, d]."""
    x, W = _f32(x), _f32(W)
    n, d = x.shape
    assert W.shape == (d, d // 2)
    out = np.empty((n, d), dtype=np.float64)
    rc = _load().linattn_ref_phi(_ptr(x, ctypes.c_float), _ptr(W, ctypes.c_float), n, d,
                                 _ptr(out, ctypes.c_double))
    if rc:
        raise ValueError("oracle rejected the arguments")
    return out


def _prep(q, k, v, Wq, Wk):
    q, k, v, Wq, Wk = (_f32(t) for t in (q, k, v, Wq, Wk))
    assert q.ndim == 4 and q.shape == k.shape == v.shape, "q, k, v must be [B, H, n, d]"
    B, H, n, d = q.shape
    if Wq.ndim == 3:
        assert Wq.shape == (H, d, d // 2) and Wk.shape == (H, d, d // 2)
        per_head = 1
    else:
        assert Wq.shape == (d, d // 2) and Wk.shape == (d, d // 2)
        per_head = 0
    return q, k, v, Wq, Wk, B, H, n, d, per_head


def _rows(rows, n):
    if rows is None:
        return None, n
    r = np.ascontiguousarray(rows, dtype=np.int64)
    assert r.ndim == 1 and (r >= 0).all() and (r < n).all()
    return r, r.shape[0]


def ref_quadratic(q, k, v, Wq, Wk, rows=None) -> np.ndarray:
    """Left form of Eq. 5 (the O(n^2) definition). Returns float64 [B, H, len(rows) or n, d]."""
    q, k, v, Wq, Wk, B, H, n, d, per_head = _prep(q, k, v, Wq, Wk)
    r, nr = _rows(rows, n)
    out = np.empty((B, H, nr, d), dtype=np.float64)
    F = ctypes.c_float
    rc = _load().linattn_ref_quadratic(_ptr(q, F), _ptr(k, F), _ptr(v, F), _ptr(Wq, F), _ptr(Wk, F),
                                       B * H, H, n, d, per_head,
                                       _ptr(r, ctypes.c_long), nr, _ptr(out, ctypes.c_double))
    if rc:
        raise ValueError("oracle rejected the arguments or ran out of memory")
    return out


def ref_linear(q, k, v, Wq, Wk, rows=None, return_state: bool = False):
    """Right form of Eq. 5: S, z, then o_i = phi(q_i) S / (phi(q_i) . z).

    Returns float64 [B, H, len(rows) or n, d]; with ``return_state`` also S [B,H,d,d] and z [B,H,d]."""
    q, k, v, Wq, Wk, B, H, n, d, per_head = _prep(q, k, v, Wq, Wk)
    r, nr = _rows(rows, n)
    out = np.empty((B, H, nr, d), dtype=np.float64)
    S = np.empty((B, H, d, d), dtype=np.float64) if return_state else None
    z = np.empty((B, H, d), dtype=np.float64) if return_state else None
    F, D = ctypes.c_float, ctypes.c_double
    rc = _load().linattn_ref_linear(_ptr(q, F), _ptr(k, F), _ptr(v, F), _ptr(Wq, F), _ptr(Wk, F),
                                    B * H, H, n, d, per_head,
                                    _ptr(r, ctypes.c_long), nr, _ptr(out, D), _ptr(S, D), _ptr(z, D))
    if rc:
        raise ValueError("oracle rejected the arguments or ran out of memory")
    return (out, S, z) if return_state else out


def ref_softmax(q, k, v, scale: float, rows=None) -> np.ndarray:
    """Softmax attention, the first term of Eq. 8, with an explicit scale on q.k. float64 [B, H, len(rows) or n, d]."""
    q, k, v = (_f32(t) for t in (q, k, v))
    assert q.ndim == 4 and q.shape == k.shape == v.shape
    B, H, n, d = q.shape
    r, nr = _rows(rows, n)
    out = np.empty((B, H, nr, d), dtype=np.float64)
    F = ctypes.c_float
    rc = _load().linattn_ref_softmax(_ptr(q, F), _ptr(k, F), _ptr(v, F), B * H, n, d, float(scale),
                                     _ptr(r, ctypes.c_long), nr, _ptr(out, ctypes.c_double))
    if rc:
        raise ValueError("oracle rejected the arguments or ran out of memory")
    return out


def ref_mix(o_softmax, o_linear, r: float) -> np.ndarray:
    """Eq. 8: clip(r, 0, 1) * o_softmax + (1 - clip(r, 0, 1)) * o_linear, in float64."""
    a = np.ascontiguousarray(o_softmax, dtype=np.float64)
    b = np.ascontiguousarray(o_linear, dtype=np.float64)
    assert a.shape == b.shape
    out = np.empty_like(a)
    D = ctypes.c_double
    if _load().linattn_ref_mix(_ptr(a, D), _ptr(b, D), a.size, float(r), _ptr(out, D)):
        raise ValueError("oracle rejected the arguments")
    return out


def ref_backward(q, k, v, Wq, Wk, dout):
    """Gradients of sum(dout * o) with respect to q, k, v, Wq, Wk (o = right form of Eq. 5 with the phi of Eq. 6).
    Returns float64 (dq, dk, dv, dWq, dWk); the weight gradients have the shape of the weights."""
    q, k, v, Wq, Wk, B, H, n, d, per_head = _prep(q, k, v, Wq, Wk)
    g = _f32(dout)
    assert g.shape == q.shape
    dq, dk, dv = (np.empty(q.shape, dtype=np.float64) for _ in range(3))
    dWq, dWk = (np.empty(Wq.shape, dtype=np.float64) for _ in range(2))
    F, D = ctypes.c_float, ctypes.c_double
    rc = _load().linattn_ref_backward(_ptr(q, F), _ptr(k, F), _ptr(v, F), _ptr(Wq, F), _ptr(Wk, F), _ptr(g, F),
                                      B * H, H, n, d, per_head, _ptr(dq, D), _ptr(dk, D), _ptr(dv, D),
                                      _ptr(dWq, D), _ptr(dWk, D))
    if rc:
        raise ValueError("oracle rejected the arguments or ran out of memory")
    return dq, dk, dv, dWq, dWk


def ref_backward_mixed(q, k, v, Wq, Wk, o_softmax, r: float, dout):
    """Gradients of sum(dout * out) through Eq. 8, out = clip(r) * o_softmax + (1 - clip(r)) * linear attention.
    Returns float64 (dq, dk, dv, dWq, dWk, d_o_softmax, dr); dr is a Python float."""
    q, k, v, Wq, Wk, B, H, n, d, per_head = _prep(q, k, v, Wq, Wk)
    g, a = _f32(dout), _f32(o_softmax)
    assert g.shape == q.shape and a.shape == q.shape
    dq, dk, dv, da = (np.empty(q.shape, dtype=np.float64) for _ in range(4))
    dWq, dWk = (np.empty(Wq.shape, dtype=np.float64) for _ in range(2))
    dr = ctypes.c_double(0.0)
    F, D = ctypes.c_float, ctypes.c_double
    rc = _load().linattn_ref_backward_mixed(_ptr(q, F), _ptr(k, F), _ptr(v, F), _ptr(Wq, F), _ptr(Wk, F), _ptr(a, F), float(r),
                                            _ptr(g, F), B * H, H, n, d, per_head, _ptr(dq, D), _ptr(dk, D), _ptr(dv, D),
                                            _ptr(dWq, D), _ptr(dWk, D), _ptr(da, D), ctypes.byref(dr))
    if rc:
        raise ValueError("oracle rejected the arguments or ran out of memory")
    return dq, dk, dv, dWq, dWk, da, float(dr.value)


def ref_relu_backward(q, k, v, dout):
    """Gradients of sum(dout * o) with the ReLU kernel function: float64 (dq, dk, dv)."""
    q, k, v, g = (_f32(t) for t in (q, k, v, dout))
    assert q.ndim == 4 and q.shape == k.shape == v.shape == g.shape
    B, H, n, d = q.shape
    dq, dk, dv = (np.empty(q.shape, dtype=np.float64) for _ in range(3))
    F, D = ctypes.c_float, ctypes.c_double
    rc = _load().linattn_ref_relu_backward(_ptr(q, F), _ptr(k, F), _ptr(v, F), _ptr(g, F), B * H, n, d,
                                           _ptr(dq, D), _ptr(dk, D), _ptr(dv, D))
    if rc:
        raise ValueError("oracle rejected the arguments or ran out of memory")
    return dq, dk, dv


def ref_relu_quadratic(q, k, v, rows=None) -> np.ndarray:
    """Left form of Eq. 5 with the ReLU kernel function phi(x) = max(x, 0). float64 [B, H, len(rows) or n, d]."""
    q, k, v = (_f32(t) for t in (q, k, v))
    assert q.ndim == 4 and q.shape == k.shape == v.shape
    B, H, n, d = q.shape
    r, nr = _rows(rows, n)
    out = np.empty((B, H, nr, d), dtype=np.float64)
    F = ctypes.c_float
    rc = _load().linattn_ref_relu_quadratic(_ptr(q, F), _ptr(k, F), _ptr(v, F), B * H, n, d, _ptr(r, ctypes.c_long), nr,
                                            _ptr(out, ctypes.c_double))
    if rc:
        raise ValueError("oracle rejected the arguments or ran out of memory")
    return out


def ref_relu_linear(q, k, v, rows=None, return_state: bool = False):
    """Right form of Eq. 5 with the ReLU kernel function; as ``ref_linear``."""
    q, k, v = (_f32(t) for t in (q, k, v))
    assert q.ndim == 4 and q.shape == k.shape == v.shape
    B, H, n, d = q.shape
    r, nr = _rows(rows, n)
    out = np.empty((B, H, nr, d), dtype=np.float64)
    S = np.empty((B, H, d, d), dtype=np.float64) if return_state else None
    z = np.empty((B, H, d), dtype=np.float64) if return_state else None
    F, D = ctypes.c_float, ctypes.c_double
    rc = _load().linattn_ref_relu_linear(_ptr(q, F), _ptr(k, F), _ptr(v, F), B * H, n, d, _ptr(r, ctypes.c_long), nr,
                                         _ptr(out, D), _ptr(S, D), _ptr(z, D))
    if rc:
        raise ValueError("oracle rejected the arguments or ran out of memory")
    return (out, S, z) if return_state else out
