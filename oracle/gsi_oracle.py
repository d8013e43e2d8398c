"""ctypes loader for the plain-C fp64 oracle (``gsi_oracle.c``).

TEST INFRASTRUCTURE ONLY: nothing in the product path may import this module.
It marshals numpy arrays into the C functions and holds no arithmetic of the
method itself; each C function cites the passage of the paper it follows
(Algorithm 1, Eq. (3.1)-(3.3), Section 4.2).

Array conventions: bf16 data travel as ``numpy.uint16`` bit patterns; the basis
P is ``[d][k]`` (uint16 bf16 bits or float32), weights W are ``[o][d]`` uint16,
activations x are ``[T][d]`` float32.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gsi_oracle.c")
_LIB = os.path.join(_HERE, "libgsi_oracle.so")
_lock = threading.Lock()
_lib = None

BF16 = 0
F32 = 1


def build(force: bool = False) -> str:
    """Compile ``gsi_oracle.c`` with gcc (OpenMP over output rows / tokens)."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + f".tmp{os.getpid()}"
            subprocess.check_call(
                ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-Wall", "-o", tmp, _SRC, "-lm"]
            )
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        vp, i, f, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_size_t
        lib.gsi_oracle_num_threads.restype = i
        lib.gsi_oracle_set_threads.argtypes = [i]
        lib.gsi_oracle_bf16_to_f64.argtypes = [vp, sz, vp]
        lib.gsi_oracle_f64_to_bf16_rne_array.argtypes = [vp, sz, vp]
        lib.gsi_oracle_image.argtypes = [vp, vp, i, i, i, i, vp]
        lib.gsi_oracle_image.restype = i
        lib.gsi_oracle_project.argtypes = [vp, i, vp, i, i, i, f, vp, vp, vp, vp, vp, vp]
        lib.gsi_oracle_project.restype = i
        lib.gsi_oracle_map.argtypes = [vp, vp, vp, vp, vp, vp, i, i, i, i, vp, vp]
        lib.gsi_oracle_map.restype = i
        lib.gsi_oracle_extend.argtypes = [vp, i, i, i, i, vp, ctypes.c_double, vp, vp]
        lib.gsi_oracle_extend.restype = i
        lib.gsi_oracle_e4m3_decode_array.argtypes = [vp, sz, vp]
        lib.gsi_oracle_f32_to_e4m3_array.argtypes = [vp, sz, vp]
        lib.gsi_oracle_quantise_image_e4m3.argtypes = [vp, i, i, vp, vp, vp]
        lib.gsi_oracle_quantise_image_e4m3.restype = i
        _lib = lib
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype):
    a = np.ascontiguousarray(a)
    if a.dtype != dtype:
        raise TypeError(f"expected {dtype}, got {a.dtype}")
    return a


def _basis(P):
    P = np.ascontiguousarray(P)
    if P.dtype == np.uint16:
        return P, BF16
    if P.dtype == np.float32:
        return P, F32
    raise TypeError("basis must be uint16 (bf16 bits) or float32")


def num_threads() -> int:
    return int(_load().gsi_oracle_num_threads())


def set_threads(n: int) -> None:
    _load().gsi_oracle_set_threads(int(n))


def bf16_to_f64(bits) -> np.ndarray:
    bits = _c(bits, np.uint16)
    out = np.empty(bits.shape, np.float64)
    _load().gsi_oracle_bf16_to_f64(_ptr(bits), bits.size, _ptr(out))
    return out


def f64_to_bf16_rne(v) -> np.ndarray:
    v = _c(v, np.float64)
    out = np.empty(v.shape, np.uint16)
    _load().gsi_oracle_f64_to_bf16_rne_array(_ptr(v), v.size, _ptr(out))
    return out


def image(W, P) -> np.ndarray:
    """M = W V_k in fp64, unrounded (Eq. (3.2), Section 4.2)."""
    W = _c(W, np.uint16)
    P, pd = _basis(P)
    o, d = W.shape
    d2, k = P.shape
    assert d == d2
    M = np.empty((o, k), np.float64)
    rc = _load().gsi_oracle_image(_ptr(W), _ptr(P), pd, o, d, k, _ptr(M))
    if rc:
        raise RuntimeError("gsi_oracle_image failed")
    return M


def e4m3_decode(codes) -> np.ndarray:
    """Values of E4M3 codes (Section 7.4 reading: the FP8 format of the image)."""
    codes = _c(codes, np.uint8)
    out = np.empty(codes.shape, np.float64)
    _load().gsi_oracle_e4m3_decode_array(_ptr(codes), codes.size, _ptr(out))
    return out


def e4m3_encode(v) -> np.ndarray:
    """Nearest E4M3 code of each float32 (ties to even, saturating)."""
    v = _c(v, np.float32)
    out = np.empty(v.shape, np.uint8)
    _load().gsi_oracle_f32_to_e4m3_array(_ptr(v), v.size, _ptr(out))
    return out


def quantise_image_e4m3(M) -> dict:
    """The image as stored in FP8 (Section 7.4): per-row scale, E4M3 codes of
    the BF16 image, and the image those codes stand for (``Mq``, fp64)."""
    M = _c(M, np.float64)
    o, k = M.shape
    codes = np.empty((o, k), np.uint8)
    scales = np.empty(o, np.float32)
    Mq = np.empty((o, k), np.float64)
    rc = _load().gsi_oracle_quantise_image_e4m3(_ptr(M), o, k, _ptr(codes), _ptr(scales), _ptr(Mq))
    if rc:
        raise RuntimeError("gsi_oracle_quantise_image_e4m3 failed")
    return {"codes": codes, "scales": scales, "Mq": Mq}


def project(x, P, eps: float) -> dict:
    """Algorithm 1 lines 1-4: g, r, rho and the gate byte (1 = slow path)."""
    x = _c(x, np.float32)
    P, pd = _basis(P)
    T, d = x.shape
    d2, k = P.shape
    assert d == d2
    out = dict(
        g=np.empty((T, k), np.float64),
        r=np.empty((T, d), np.float64),
        rho=np.empty(T, np.float64),
        norm_x=np.empty(T, np.float64),
        norm_r=np.empty(T, np.float64),
        gate=np.empty(T, np.uint8),
    )
    rc = _load().gsi_oracle_project(
        _ptr(x), T, _ptr(P), pd, d, k, float(np.float32(eps)),
        _ptr(out["g"]), _ptr(out["r"]), _ptr(out["rho"]),
        _ptr(out["norm_x"]), _ptr(out["norm_r"]), _ptr(out["gate"]),
    )
    if rc:
        raise RuntimeError("gsi_oracle_project failed")
    return out


def extend(P, k_act: int, x, tau: float) -> dict:
    """Online basis extension by one vector (Sections 5.4 and 7.2): rho of the token
    against columns [0, k_act) of the stored basis P [d][k_cap]; if rho > tau (and a
    column is free) the unit vector v = twice-orthogonalised residual, in fp64.
    ``v_bits`` is v rounded to bf16 (round to nearest even), the value a bf16 basis
    stores in column k_act."""
    P, pd = _basis(P)
    d, k_cap = P.shape
    x = _c(np.asarray(x, np.float64).reshape(-1), np.float64)
    assert x.size == d
    rho = ctypes.c_double()
    v = np.zeros(d, np.float64)
    rc = _load().gsi_oracle_extend(_ptr(P), pd, d, k_cap, int(k_act), _ptr(x), float(tau),
                                   ctypes.byref(rho), _ptr(v))
    if rc < 0:
        raise RuntimeError("gsi_oracle_extend failed")
    out = dict(rho=rho.value, extended=bool(rc))
    if rc:
        out["v"] = v
        out["v_bits"] = f64_to_bf16_rne(v)
    return out


def apply_map(M, W, g, r, gate, x=None, want_alt: bool = False):
    """y = M g (+ W r on gated tokens); optionally Algorithm 1 read literally."""
    M = _c(M, np.float64)
    W = _c(W, np.uint16)
    g = _c(g, np.float64)
    r = _c(r, np.float64)
    gate = _c(gate, np.uint8)
    o, d = W.shape
    T, k = g.shape
    assert M.shape == (o, k) and r.shape == (T, d) and gate.shape == (T,)
    y = np.empty((T, o), np.float64)
    y_alt = None
    if want_alt:
        x = _c(x, np.float32)
        assert x.shape == (T, d)
        y_alt = np.empty((T, o), np.float64)
    rc = _load().gsi_oracle_map(
        _ptr(M), _ptr(W), _ptr(g), _ptr(r), _ptr(x) if want_alt else None,
        _ptr(gate), T, o, d, k, _ptr(y), _ptr(y_alt),
    )
    if rc:
        raise RuntimeError("gsi_oracle_map failed")
    return (y, y_alt) if want_alt else y


def forward(x, P, eps: float, Ws, gate_override=None, rows=None, fp8_image: bool = False) -> dict:
    """The whole layer for one input group: the maps in ``Ws`` share x, P, g, r
    and one gate decision per token.

    ``rows`` (one index array per map, or None) restricts each map to a sample
    of its output rows; the projection and the gate always use the full basis.
    ``gate_override`` substitutes given gate bytes when forming y (used for
    tokens whose rho sits on the threshold); the oracle's own decision is still
    returned as ``gate``.  ``fp8_image`` stores the image in FP8 first.
    """
    pr = project(x, P, eps)
    gate_used = pr["gate"] if gate_override is None else _c(gate_override, np.uint8)
    ys = []
    for j, W in enumerate(Ws):
        W = _c(W, np.uint16)
        if rows is not None and rows[j] is not None:
            W = np.ascontiguousarray(W[np.asarray(rows[j])])
        M = image(W, P)
        if fp8_image:   # the image as stored in FP8 (Section 7.4)
            M = quantise_image_e4m3(M)["Mq"]
        ys.append(apply_map(M, W, pr["g"], pr["r"], gate_used))
    pr["y"] = ys
    pr["gate_used"] = gate_used
    return pr
