"""Thin ctypes binding of the C-ABI library declared in ``include/linattn.h``.

Only argument marshalling happens here: every step of the operator runs in the CUDA
kernels of ``liblinattn.so``.  PyTorch supplies device memory and streams.  There is no
fallback: if the shared library has not been built, importing the symbols raises.
"""
from __future__ import annotations

import ctypes
import os

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "liblinattn.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_NO_FEATURE_MAP, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT = range(7)
F32, BF16 = 0, 1
OPT_SPLITS, OPT_PATH, OPT_PROFILE, OPT_FUSE, OPT_LAYOUT, OPT_KERNEL_FUNCTION, OPT_REUSE_STATE = 0, 1, 2, 3, 4, 5, 6
OPT_WAIT_LIMIT_US, OPT_TEST_UNMET_ARRIVAL = 7, 8
PHI_HEDGEHOG, PHI_RELU = 0, 1
LAYOUT_BHND, LAYOUT_BNHD = 0, 1
PATH_AUTO, PATH_SIMT, PATH_TENSOR = 0, 1, 2

_DTYPES = {torch.float32: F32, torch.bfloat16: BF16}

# name -> (restype, argtypes); mirrors include/linattn.h
_vp, _ll, _i = ctypes.c_void_p, ctypes.c_longlong, ctypes.c_int
SIGNATURES = {
    "linattn_create": (_i, [ctypes.POINTER(_vp), _i, _i, _i, _ll, _ll]),
    "linattn_set_feature_map": (_i, [_vp, _vp, _vp, _i, _i, _vp]),
    "linattn_forward": (_i, [_vp, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _vp]),
    "linattn_forward_mixed": (_i, [_vp, _vp, _vp, _vp, _vp, ctypes.c_float, _vp, _i, _i, _i, _i, _i, _vp]),
    "linattn_backward": (_i, [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _i, _vp]),
    "linattn_backward_mixed": (_i, [_vp, _vp, _vp, _vp, _vp, ctypes.c_float, _vp, _vp, _vp, _vp, _vp, _vp, _i, _vp, _vp,
                                    _i, _i, _i, _i, _i, _vp]),
    "linattn_forward_host": (_i, [_vp, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _vp]),
    "linattn_forward_noalloc": (_i, [_vp, _vp, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _i, _vp]),
    "linattn_read_state": (_i, [_vp, _vp, _vp, _i, _vp]),
    "linattn_set_option": (_i, [_vp, _i, _ll]),
    "linattn_check": (_i, [_vp, _vp]),
    "linattn_profile_get": (_i, [_vp, _i, ctypes.POINTER(ctypes.c_char_p), ctypes.POINTER(ctypes.c_double),
                                ctypes.POINTER(_ll), ctypes.POINTER(ctypes.c_double)]),
    "linattn_last_launch_count": (_i, [_vp]),
    "linattn_last_error": (ctypes.c_char_p, [_vp]),
    "linattn_destroy": (_i, [_vp]),
    "linattn_status_string": (ctypes.c_char_p, [_i]),
}

_lib = None


class LinAttnError(RuntimeError):
    def __init__(self, status: int, text: str):
        super().__init__(f"linattn status {status}: {text}")
        self.status = status


def load_library() -> ctypes.CDLL:
    """Load ``liblinattn.so`` and attach the prototypes.  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2510_08318_b200.build` "
                              "(there is no fallback implementation)")
        lib = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(lib, name)
            fn.restype = res
            fn.argtypes = args
        _lib = lib
    return _lib


def status_string(status: int) -> str:
    return load_library().linattn_status_string(status).decode()


def _stream_ptr(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream


def forward_noalloc(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, Wq: torch.Tensor, Wk: torch.Tensor,
                    out: torch.Tensor, stream=None) -> torch.Tensor:
    """``linattn_forward_noalloc``: the forward for callers that may not allocate device memory.

    No context and no allocation inside the library: q, k, v, out are contiguous CUDA tensors
    [B, H, n, d] (the caller provides ``out``), Wq and Wk are fp32 CUDA tensors [H, d, d/2] or
    [d, d/2], and the scratch lives in a fixed device array of the library (B * H <= 16).
    Runs on the current device; calls on one device must be stream-ordered."""
    lib = load_library()
    for t in (q, k, v, out, Wq, Wk):
        assert t.is_cuda and t.is_contiguous()
    assert q.shape == k.shape == v.shape == out.shape and q.dtype == k.dtype == v.dtype == out.dtype
    assert Wq.dtype == torch.float32 and Wk.dtype == torch.float32 and Wq.shape == Wk.shape
    B, H, n, d = q.shape
    st = lib.linattn_forward_noalloc(q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), Wq.data_ptr(),
                                     Wk.data_ptr(), 1 if Wq.dim() == 3 else 0, B, H, n, d, _DTYPES[q.dtype],
                                     _stream_ptr(stream))
    if st != OK:
        raise LinAttnError(st, status_string(st))
    return out


class LinAttn:
    """One attention layer's context: ``linattn_create`` ... ``linattn_destroy``."""

    def __init__(self, H: int, d: int, max_B: int, max_n: int, device: int = 0):
        self._lib = load_library()
        self._h = _vp()
        self.H, self.d, self.device = H, d, device
        st = self._lib.linattn_create(ctypes.byref(self._h), device, H, d, max_B, max_n)
        if st != OK:
            self._h = _vp()
            raise LinAttnError(st, status_string(st))

    # -- helpers -----------------------------------------------------------------------------
    def _raise(self, st: int):
        detail = self._lib.linattn_last_error(self._h).decode() if self._h else ""
        raise LinAttnError(st, status_string(st) + (f" ({detail})" if detail else ""))

    def _call(self, fn, *args) -> None:
        st = fn(self._h, *args)
        if st != OK:
            self._raise(st)

    # -- the C-ABI, one method per entry point --------------------------------------------------
    def set_feature_map(self, Wq: torch.Tensor, Wk: torch.Tensor, stream=None) -> None:
        """Wq, Wk: CUDA tensors [H, d, d/2] (per head) or [d, d/2] (shared), fp32 or bf16."""
        assert Wq.is_cuda and Wk.is_cuda and Wq.dtype == Wk.dtype and Wq.shape == Wk.shape
        assert Wq.is_contiguous() and Wk.is_contiguous()
        per_head = 1 if Wq.dim() == 3 else 0
        assert tuple(Wq.shape[-2:]) == (self.d, self.d // 2) and (not per_head or Wq.shape[0] == self.H)
        self._call(self._lib.linattn_set_feature_map, Wq.data_ptr(), Wk.data_ptr(), per_head,
                   _DTYPES[Wq.dtype], _stream_ptr(stream))

    def forward(self, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, out: torch.Tensor | None = None,
                stream=None) -> torch.Tensor:
        """q, k, v: contiguous CUDA tensors [B, H, n, d]; returns out (allocated by torch if not given)."""
        assert q.is_cuda and q.is_contiguous() and k.is_contiguous() and v.is_contiguous()
        assert q.shape == k.shape == v.shape and q.dtype == k.dtype == v.dtype and q.dim() == 4
        if out is None:
            out = torch.empty_like(q)
        assert out.is_contiguous() and out.shape == q.shape and out.dtype == q.dtype
        B, H, n, d = q.shape
        self._call(self._lib.linattn_forward, q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(),
                   B, H, n, d, _DTYPES[q.dtype], _stream_ptr(stream))
        return out

    def forward_mixed(self, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, o_softmax: torch.Tensor, r: float,
                      out: torch.Tensor | None = None, stream=None) -> torch.Tensor:
        """Eq. 8: clip(r, 0, 1) * o_softmax + (1 - clip(r, 0, 1)) * linear attention.  ``o_softmax`` is the output of
        the layer's softmax-attention branch, [B, H, n, d]; ``out`` may be ``o_softmax`` itself (in place)."""
        assert q.is_cuda and q.is_contiguous() and k.is_contiguous() and v.is_contiguous() and o_softmax.is_contiguous()
        assert q.shape == k.shape == v.shape == o_softmax.shape and q.dtype == k.dtype == v.dtype == o_softmax.dtype
        if out is None:
            out = torch.empty_like(q)
        assert out.is_contiguous() and out.shape == q.shape and out.dtype == q.dtype
        B, H, n, d = q.shape
        self._call(self._lib.linattn_forward_mixed, q.data_ptr(), k.data_ptr(), v.data_ptr(), o_softmax.data_ptr(),
                   float(r), out.data_ptr(), B, H, n, d, _DTYPES[q.dtype], _stream_ptr(stream))
        return out

    def backward(self, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, dout: torch.Tensor, per_head: bool = True,
                 stream=None):
        """Gradients of ``forward``: returns (dq, dk, dv, dWq, dWk); dq, dk, dv like q, the weight gradients fp32
        [H, d, d/2] (``per_head``) or [d, d/2] (one shared matrix)."""
        for t in (q, k, v, dout):
            assert t.is_cuda and t.is_contiguous()
        assert q.shape == k.shape == v.shape == dout.shape and q.dtype == k.dtype == v.dtype == dout.dtype
        dq, dk, dv = torch.empty_like(q), torch.empty_like(q), torch.empty_like(q)
        wshape = (self.H, self.d, self.d // 2) if per_head else (self.d, self.d // 2)
        dWq = torch.empty(wshape, dtype=torch.float32, device=q.device)
        dWk = torch.empty(wshape, dtype=torch.float32, device=q.device)
        B, H, n, d = q.shape
        self._call(self._lib.linattn_backward, q.data_ptr(), k.data_ptr(), v.data_ptr(), dout.data_ptr(), dq.data_ptr(),
                   dk.data_ptr(), dv.data_ptr(), dWq.data_ptr(), dWk.data_ptr(), 1 if per_head else 0, B, H, n, d,
                   _DTYPES[q.dtype], _stream_ptr(stream))
        return dq, dk, dv, dWq, dWk

    def backward_mixed(self, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, o_softmax: torch.Tensor, r: float,
                       dout: torch.Tensor, per_head: bool = True, want_d_o_softmax: bool = True, stream=None):
        """Gradients through Eq. 8: returns (dq, dk, dv, dWq, dWk, d_o_softmax or None, dr); dr is a CUDA tensor of one float."""
        for t in (q, k, v, o_softmax, dout):
            assert t.is_cuda and t.is_contiguous()
        assert q.shape == k.shape == v.shape == dout.shape == o_softmax.shape
        assert q.dtype == k.dtype == v.dtype == dout.dtype == o_softmax.dtype
        dq, dk, dv = torch.empty_like(q), torch.empty_like(q), torch.empty_like(q)
        da = torch.empty_like(q) if want_d_o_softmax else None
        wshape = (self.H, self.d, self.d // 2) if per_head else (self.d, self.d // 2)
        dWq = torch.empty(wshape, dtype=torch.float32, device=q.device)
        dWk = torch.empty(wshape, dtype=torch.float32, device=q.device)
        dr = torch.empty(1, dtype=torch.float32, device=q.device)
        B, H, n, d = q.shape
        self._call(self._lib.linattn_backward_mixed, q.data_ptr(), k.data_ptr(), v.data_ptr(), o_softmax.data_ptr(), float(r),
                   dout.data_ptr(), dq.data_ptr(), dk.data_ptr(), dv.data_ptr(), dWq.data_ptr(), dWk.data_ptr(),
                   1 if per_head else 0, da.data_ptr() if da is not None else None, dr.data_ptr(), B, H, n, d,
                   _DTYPES[q.dtype], _stream_ptr(stream))
        return dq, dk, dv, dWq, dWk, da, dr

    def forward_host(self, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, out: torch.Tensor,
                     stream=None) -> torch.Tensor:
        """The same on CPU tensors (pinned or pageable); copies in, computes on the GPU, copies out, waits."""
        for t in (q, k, v, out):
            assert (not t.is_cuda) and t.is_contiguous()
        assert q.shape == k.shape == v.shape == out.shape and q.dtype == k.dtype == v.dtype == out.dtype
        B, H, n, d = q.shape
        self._call(self._lib.linattn_forward_host, q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(),
                   B, H, n, d, _DTYPES[q.dtype], _stream_ptr(stream))
        return out

    def read_state(self, B: int, stream=None):
        """(S [B,H,d,d], z [B,H,d]) fp32 CPU tensors left by the most recent forward."""
        S = torch.empty(B, self.H, self.d, self.d, dtype=torch.float32)
        z = torch.empty(B, self.H, self.d, dtype=torch.float32)
        self._call(self._lib.linattn_read_state, S.data_ptr(), z.data_ptr(), B, _stream_ptr(stream))
        return S, z

    def set_option(self, opt: int, value: int) -> None:
        self._call(self._lib.linattn_set_option, opt, value)

    def check(self, stream=None) -> None:
        self._call(self._lib.linattn_check, _stream_ptr(stream))

    def kernel_times(self):
        """Per-kernel figures gathered while OPT_PROFILE was on: [{name, ms, launches, bytes}] in launch order."""
        res, i = [], 0
        while True:
            name, ms, cnt, nb = ctypes.c_char_p(), ctypes.c_double(), _ll(), ctypes.c_double()
            if not self._lib.linattn_profile_get(self._h, i, ctypes.byref(name), ctypes.byref(ms), ctypes.byref(cnt),
                                                 ctypes.byref(nb)):
                return res
            res.append({"name": name.value.decode(), "ms": ms.value, "launches": cnt.value, "bytes": nb.value})
            i += 1

    def last_launch_count(self) -> int:
        return int(self._lib.linattn_last_launch_count(self._h))

    def destroy(self) -> None:
        if self._h:
            self._lib.linattn_destroy(self._h)
            self._h = _vp()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass
