"""ctypes binding of ``include/gsi.h`` (same names, argument marshalling only).

``Layer`` and ``Stack`` wrap a handle together with the torch tensors that back
its workspace; they add no computation.  If the CUDA library cannot be loaded
the import fails loudly: there is no fallback.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

from . import build as _build

GSI_BF16, GSI_F32 = 0, 1
GSI_FLAG_NONE, GSI_FLAG_STATIC_PROJECTION, GSI_FLAG_DENSE, GSI_FLAG_FP8_IMAGE = 0, 1, 2, 4
GSI_MAX_MAPS, GSI_MAX_TOKENS = 8, 64

EXPORTED = [
    "gsi_status_string", "gsi_build_image", "gsi_workspace_bytes", "gsi_create",
    "gsi_forward", "gsi_forward_n", "gsi_forward_host", "gsi_forward_static", "gsi_extend_basis", "gsi_get_image", "gsi_get_image_fp8", "gsi_get_status",
    "gsi_destroy", "gsi_stack_workspace_bytes", "gsi_stack_create", "gsi_stack_bind",
    "gsi_stack_set_mode", "gsi_stack_set_concurrent", "gsi_stack_is_persistent", "gsi_stack_set_trace", "gsi_stack_set_spin_limit", "gsi_stack_seek", "gsi_stack_step", "gsi_stack_launches_per_step",
    "gsi_stack_step_host", "gsi_stack_get_status", "gsi_stack_destroy",
]


class GsiDesc(C.Structure):
    _fields_ = [("d", C.c_int), ("k", C.c_int), ("n_maps", C.c_int),
                ("d_out", C.POINTER(C.c_int)), ("eps", C.c_float), ("max_tokens", C.c_int),
                ("p_dtype", C.c_int), ("flags", C.c_uint)]


class GsiStackIo(C.Structure):
    _fields_ = [("x", C.c_void_p), ("y", C.c_void_p)]


class GsiError(RuntimeError):
    def __init__(self, code, where):
        self.code = int(code)
        super().__init__(f"{where}: {gsi_status_string(code)} ({int(code)})")


def lib_path() -> str:
    return _build.LIB


def _load():
    path = _build.build()   # no-op when the library matches the sources
    l = C.CDLL(path)
    vp, i, sz = C.c_void_p, C.c_int, C.c_size_t
    l.gsi_status_string.restype = C.c_char_p
    l.gsi_status_string.argtypes = [i]
    l.gsi_build_image.argtypes = [vp, vp, i, i, i, i, vp, vp]
    l.gsi_workspace_bytes.restype = sz
    l.gsi_workspace_bytes.argtypes = [C.POINTER(GsiDesc)]
    l.gsi_create.argtypes = [C.POINTER(GsiDesc), C.POINTER(vp), vp, vp, sz, vp, C.POINTER(vp)]
    l.gsi_forward.argtypes = [vp, vp, vp, vp, vp]
    l.gsi_forward_n.argtypes = [vp, vp, i, vp, vp, vp, vp]
    l.gsi_forward_host.argtypes = [vp, vp, i, vp, vp, vp, vp]
    l.gsi_forward_static.argtypes = [C.POINTER(vp), C.POINTER(i), i, vp, i, vp, i, i, C.c_float,
                                     vp, i, vp, vp, vp, vp]
    l.gsi_get_image.argtypes = [vp, i, C.POINTER(vp)]
    l.gsi_get_image_fp8.argtypes = [vp, C.POINTER(vp), C.POINTER(C.c_size_t)]
    l.gsi_extend_basis.argtypes = [vp, vp, C.c_float, vp, vp, vp, vp]
    l.gsi_get_status.argtypes = [vp, C.POINTER(i)]
    l.gsi_destroy.argtypes = [vp]
    l.gsi_stack_workspace_bytes.restype = sz
    l.gsi_stack_workspace_bytes.argtypes = [i]
    l.gsi_stack_create.argtypes = [i, C.POINTER(vp), vp, sz, vp, C.POINTER(vp)]
    l.gsi_stack_bind.argtypes = [vp, C.POINTER(GsiStackIo), i, vp, vp, vp]
    l.gsi_stack_set_mode.argtypes = [vp, i]
    l.gsi_stack_set_concurrent.argtypes = [vp, i, i]
    l.gsi_stack_is_persistent.argtypes = [vp, C.POINTER(i)]
    l.gsi_stack_set_trace.argtypes = [vp, vp]
    l.gsi_stack_set_spin_limit.argtypes = [vp, C.c_uint]
    l.gsi_stack_seek.argtypes = [vp, i, vp]
    l.gsi_stack_step.argtypes = [vp, vp]
    l.gsi_stack_launches_per_step.argtypes = [vp, C.POINTER(i)]
    l.gsi_stack_step_host.argtypes = [vp, C.POINTER(vp), C.POINTER(vp), vp, vp]
    l.gsi_stack_get_status.argtypes = [vp, C.POINTER(i)]
    l.gsi_stack_destroy.argtypes = [vp]
    for name in EXPORTED:
        if name not in ("gsi_status_string", "gsi_workspace_bytes", "gsi_stack_workspace_bytes"):
            getattr(l, name).restype = i
    return l


lib = _load()


def gsi_status_string(code) -> str:
    return lib.gsi_status_string(int(code)).decode()


def _check(code, where):
    if code != 0:
        raise GsiError(code, where)


def _stream_ptr(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream) if hasattr(stream, "cuda_stream") else int(stream)


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return GSI_BF16
    if t.dtype == torch.float32:
        return GSI_F32
    raise TypeError("basis must be bfloat16 or float32")


def make_desc(d, k, d_out, eps, max_tokens, p_dtype=GSI_BF16, flags=0):
    arr = (C.c_int * len(d_out))(*[int(v) for v in d_out])
    desc = GsiDesc(int(d), int(k), len(d_out), C.cast(arr, C.POINTER(C.c_int)), float(eps),
                   int(max_tokens), int(p_dtype), int(flags))
    desc._keep = arr
    return desc


def gsi_workspace_bytes(d, k, d_out, eps, max_tokens, p_dtype=GSI_BF16, flags=0) -> int:
    return int(lib.gsi_workspace_bytes(C.byref(make_desc(d, k, d_out, eps, max_tokens, p_dtype, flags))))


def gsi_build_image(W: torch.Tensor, P: torch.Tensor, out: torch.Tensor | None = None,
                    stream=None) -> torch.Tensor:
    """W_P = bf16(W P) on the device (Section 4.2 of the paper)."""
    assert W.is_cuda and P.is_cuda and W.dtype == torch.bfloat16
    assert W.is_contiguous() and P.is_contiguous()
    o, d = W.shape
    d2, k = P.shape
    assert d == d2
    if out is None:
        out = torch.empty((o, k), dtype=torch.bfloat16, device=W.device)
    _check(lib.gsi_build_image(W.data_ptr(), P.data_ptr(), o, d, k, _dtype_code(P),
                               out.data_ptr(), _stream_ptr(stream)), "gsi_build_image")
    return out


def gsi_forward_static(Ws, P, W_P, eps, x, y=None, gate=None, rho=None, stream=None):
    """Algorithm 1 through the entry point that allocates nothing inside the
    library: scratch comes from an array built into ``libgsi_b200.so``.  For
    callers that may not call cudaMalloc (see ``include/gsi.h``).  ``W_P`` is the
    concatenation of ``gsi_build_image(W_j, P)`` over the maps.  The output
    tensors are allocated HERE, by torch, only when the caller passes none."""
    Ws = list(Ws)
    n = int(x.shape[0])
    d, k = int(P.shape[0]), int(P.shape[1])
    d_out = [int(W.shape[0]) for W in Ws]
    if y is None:
        y = torch.empty((n, sum(d_out)), dtype=torch.float32, device=x.device)
    if gate is None:
        gate = torch.empty(n, dtype=torch.uint8, device=x.device)
    if rho is None:
        rho = torch.empty(n, dtype=torch.float32, device=x.device)
    warr = (C.c_void_p * len(Ws))(*[W.data_ptr() for W in Ws])
    darr = (C.c_int * len(Ws))(*d_out)
    _check(lib.gsi_forward_static(warr, darr, len(Ws), P.data_ptr(), _dtype_code(P),
                                  W_P.data_ptr(), d, k, float(eps), x.data_ptr(), n,
                                  y.data_ptr(), gate.data_ptr(), rho.data_ptr(),
                                  _stream_ptr(stream)), "gsi_forward_static")
    return y, gate, rho


class Layer:
    """One group: maps ``Ws`` (list of [d_out_j][d] bf16) sharing basis ``P``."""

    def __init__(self, Ws, P, eps: float, max_tokens: int = 1, flags: int = 0, stream=None):
        Ws = list(Ws)
        dense = bool(flags & GSI_FLAG_DENSE)
        dev = Ws[0].device
        assert dev.type == "cuda", "the gated subspace layer runs on a CUDA device only"
        for W in Ws:
            assert W.dtype == torch.bfloat16 and W.is_contiguous() and W.device == dev
        self.d = int(Ws[0].shape[1])
        self.d_out = [int(W.shape[0]) for W in Ws]
        self.O = sum(self.d_out)
        self.k = 8 if (dense and P is None) else int(P.shape[1])
        self.max_tokens = int(max_tokens)
        self.eps = float(eps)
        self.flags = int(flags)
        assert P is None or (P.is_contiguous() and P.device == dev and tuple(P.shape) == (self.d, self.k))
        self._Ws, self._P = Ws, P
        pd = GSI_BF16 if P is None else _dtype_code(P)
        self._desc = make_desc(self.d, self.k, self.d_out, eps, max_tokens, pd, flags)
        nbytes = int(lib.gsi_workspace_bytes(C.byref(self._desc)))
        if nbytes == 0:
            raise GsiError(2, "gsi_workspace_bytes (descriptor rejected)")
        self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=dev)
        warr = (C.c_void_p * len(Ws))(*[W.data_ptr() for W in Ws])
        h = C.c_void_p()
        _check(lib.gsi_create(C.byref(self._desc), warr, None if P is None else P.data_ptr(),
                              self.workspace.data_ptr(), nbytes, _stream_ptr(stream),
                              C.byref(h)), "gsi_create")
        self.handle = h
        self.device = dev

    def forward(self, x: torch.Tensor, y: torch.Tensor | None = None,
                gate: torch.Tensor | None = None, rho: torch.Tensor | None = None, stream=None):
        assert x.is_cuda and x.dtype == torch.float32 and x.is_contiguous()
        n = int(x.shape[0])
        if y is None:
            y = torch.empty((n, self.O), dtype=torch.float32, device=x.device)
        if gate is None:
            gate = torch.empty(n, dtype=torch.uint8, device=x.device)
        if rho is None:
            rho = torch.empty(n, dtype=torch.float32, device=x.device)
        _check(lib.gsi_forward_n(self.handle, x.data_ptr(), n, y.data_ptr(), gate.data_ptr(),
                                 rho.data_ptr(), _stream_ptr(stream)), "gsi_forward_n")
        return y, gate, rho

    def forward_host(self, x: torch.Tensor, stream=None):
        """Host tensors in, host tensors out (copies inside the call)."""
        assert not x.is_cuda and x.dtype == torch.float32 and x.is_contiguous()
        n = int(x.shape[0])
        y = torch.empty((n, self.O), dtype=torch.float32).pin_memory()
        gate = torch.empty(n, dtype=torch.uint8).pin_memory()
        rho = torch.empty(n, dtype=torch.float32).pin_memory()
        _check(lib.gsi_forward_host(self.handle, x.data_ptr(), n, y.data_ptr(), gate.data_ptr(),
                                    rho.data_ptr(), _stream_ptr(stream)), "gsi_forward_host")
        return y, gate, rho

    def extend_basis(self, x: torch.Tensor, tau: float, k_active: torch.Tensor, stream=None):
        """gsi_extend_basis for one token x [d]; k_active is a device int32 tensor (in/out).
        Returns (appended, rho) as device tensors.  Writes the basis tensor given at creation."""
        assert x.is_cuda and x.dtype == torch.float32 and x.is_contiguous() and x.numel() == self.d
        assert k_active.is_cuda and k_active.dtype == torch.int32 and k_active.numel() == 1
        appended = torch.zeros(1, dtype=torch.int32, device=x.device)
        rho = torch.zeros(1, dtype=torch.float32, device=x.device)
        _check(lib.gsi_extend_basis(self.handle, x.data_ptr(), float(tau), k_active.data_ptr(),
                                    appended.data_ptr(), rho.data_ptr(), _stream_ptr(stream)),
               "gsi_extend_basis")
        return appended, rho

    def image(self, j: int) -> torch.Tensor:
        """Copy of the cached image of map j ([d_out_j][k] bf16)."""
        p = C.c_void_p()
        _check(lib.gsi_get_image(self.handle, j, C.byref(p)), "gsi_get_image")
        base = self.workspace.data_ptr()
        off = p.value - base
        nbytes = self.d_out[j] * self.k * 2
        return self.workspace[off:off + nbytes].view(torch.bfloat16).view(self.d_out[j], self.k).clone()

    def image_fp8(self):
        """The FP8 image of all maps as stored (GSI_FLAG_FP8_IMAGE handles): codes
        ``[sum d_out][k]`` uint8 and row scales ``[sum d_out]`` fp32, copied out of
        the tiled layout the header documents (a rearrangement of bytes only)."""
        p, n = C.c_void_p(), C.c_size_t()
        _check(lib.gsi_get_image_fp8(self.handle, C.byref(p), C.byref(n)), "gsi_get_image_fp8")
        off = p.value - self.workspace.data_ptr()
        raw = self.workspace[off:off + n.value]
        O, k = sum(self.d_out), self.k
        R, KT = (O + 15) // 16, k // 16
        raw = raw.view(R, KT * 256 + 64)
        # tile bytes [R][K][g][t][c8][r8][e]: element (row g + 8 r8, column 2 t + 8 c8 + e)
        tiles = raw[:, :KT * 256].reshape(R, KT, 8, 4, 2, 2, 2)
        codes = tiles.permute(0, 5, 2, 1, 4, 3, 6).reshape(R * 16, k)[:O].clone()
        scales = raw[:, KT * 256:].contiguous().view(torch.float32).reshape(R * 16)[:O].clone()
        return codes, scales

    def status(self) -> int:
        v = C.c_int()
        _check(lib.gsi_get_status(self.handle, C.byref(v)), "gsi_get_status")
        return v.value

    def close(self):
        if getattr(self, "handle", None):
            lib.gsi_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class Stack:
    """An ordered chain of groups stepped as one decode step."""

    def __init__(self, layers, stream=None, mode: int = 0, concurrent=()):
        """concurrent: indices i such that groups i and i+1 do not read each other's outputs
        and may share a phase of the persistent kernel (gsi_stack_set_concurrent)."""
        self.layers = list(layers)
        self._mode = int(mode)
        n = len(self.layers)
        dev = self.layers[0].device
        self.B = self.layers[0].max_tokens
        nbytes = int(lib.gsi_stack_workspace_bytes(n))
        self.workspace = torch.zeros(nbytes, dtype=torch.uint8, device=dev)
        arr = (C.c_void_p * n)(*[l.handle for l in self.layers])
        h = C.c_void_p()
        _check(lib.gsi_stack_create(n, arr, self.workspace.data_ptr(), nbytes,
                                    _stream_ptr(stream), C.byref(h)), "gsi_stack_create")
        self.handle = h
        self.device = dev
        if self._mode:
            _check(lib.gsi_stack_set_mode(self.handle, self._mode), "gsi_stack_set_mode")
        for first in concurrent:
            _check(lib.gsi_stack_set_concurrent(self.handle, int(first), 1), "gsi_stack_set_concurrent")

    def is_persistent(self) -> bool:
        v = C.c_int()
        _check(lib.gsi_stack_is_persistent(self.handle, C.byref(v)), "gsi_stack_is_persistent")
        return bool(v.value)

    def bind(self, xs, ys=None, n_steps: int = 1, want_rho: bool = True, stream=None):
        """xs[g]: [n_steps][B][d] fp32 device tensors.  Allocates y and the logs."""
        n = len(self.layers)
        if ys is None:
            ys = [torch.empty((self.B, l.O), dtype=torch.float32, device=self.device)
                  for l in self.layers]
        self.xs, self.ys, self.n_steps = list(xs), list(ys), int(n_steps)
        for x, l in zip(self.xs, self.layers):
            assert x.is_cuda and x.dtype == torch.float32 and x.is_contiguous()
            assert x.numel() == n_steps * self.B * l.d
        self.gate_log = torch.zeros((n_steps, n, self.B), dtype=torch.uint8, device=self.device)
        self.rho_log = (torch.zeros((n_steps, n, self.B), dtype=torch.float32, device=self.device)
                        if want_rho else None)
        io = (GsiStackIo * n)(*[GsiStackIo(x.data_ptr(), y.data_ptr())
                                for x, y in zip(self.xs, self.ys)])
        _check(lib.gsi_stack_bind(self.handle, io, n_steps, self.gate_log.data_ptr(),
                                  None if self.rho_log is None else self.rho_log.data_ptr(),
                                  _stream_ptr(stream)), "gsi_stack_bind")

    def set_trace(self, on: bool = True):
        """Per-section SM-cycle counters, one row per CTA (persistent launch only); the
        sections are listed at gsi_stack_set_trace in the header."""
        self.trace = torch.zeros((256, 16), dtype=torch.int64, device=self.device) if on else None
        _check(lib.gsi_stack_set_trace(self.handle, self.trace.data_ptr() if on else None),
               "gsi_stack_set_trace")
        return self.trace

    def set_spin_limit(self, polls: int):
        """Polls a cross-CTA wait of the persistent kernel may take (0 = default)."""
        _check(lib.gsi_stack_set_spin_limit(self.handle, int(polls)), "gsi_stack_set_spin_limit")

    def seek(self, step: int, stream=None):
        _check(lib.gsi_stack_seek(self.handle, int(step), _stream_ptr(stream)), "gsi_stack_seek")

    def step(self, stream=None):
        _check(lib.gsi_stack_step(self.handle, _stream_ptr(stream)), "gsi_stack_step")

    def launches_per_step(self) -> int:
        v = C.c_int()
        _check(lib.gsi_stack_launches_per_step(self.handle, C.byref(v)),
               "gsi_stack_launches_per_step")
        return v.value

    def step_host(self, xs_host, ys_host, gate_host, stream=None):
        n = len(self.layers)
        xa = (C.c_void_p * n)(*[x.data_ptr() for x in xs_host])
        ya = (C.c_void_p * n)(*[y.data_ptr() for y in ys_host])
        _check(lib.gsi_stack_step_host(self.handle, xa, ya, gate_host.data_ptr(),
                                       _stream_ptr(stream)), "gsi_stack_step_host")

    def status(self) -> int:
        v = C.c_int()
        _check(lib.gsi_stack_get_status(self.handle, C.byref(v)), "gsi_stack_get_status")
        return v.value

    def close(self):
        if getattr(self, "handle", None):
            lib.gsi_stack_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
