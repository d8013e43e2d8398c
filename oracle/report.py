"""Reporting formulas of the paper, written out (test infrastructure).

Each is pinned by the values the paper prints (tests/golden/).
"""
from __future__ import annotations


def effective_speedup(f: float, compression: float) -> float:
    """Eq. (3.4): S = 1 / (f / (d/k) + (1 - f)), f = fast-path fraction,
    compression = d/k."""
    return 1.0 / (f / compression + (1.0 - f))


def effective_parameter_fraction(f: float, k: int, d: int) -> float:
    """Bracket of Eq. (5.1) divided by d: f*k/d + (1 - f); multiply by the
    parameter count of the linear maps for P_eff."""
    return f * k / d + (1.0 - f)


def effective_parameters(layers) -> float:
    """Eq. (5.1): sum over layers of N_W * d_out * [f*k + (1-f)*d].
    ``layers`` is an iterable of (N_W, d_out, d, k, f)."""
    return sum(nw * do * (f * k + (1.0 - f) * d) for nw, do, d, k, f in layers)


def image_storage_bytes(n_layers: int, sum_d_out: int, k: int, bytes_per: int = 2) -> int:
    """Section 4.2: L * (sum of d_out over the maps of a layer) * k elements."""
    return n_layers * sum_d_out * k * bytes_per


def basis_storage_bytes(n_layers: int, d: int, k: int, bytes_per: int = 2) -> int:
    """Section 4.2: L * d * k elements."""
    return n_layers * d * k * bytes_per
