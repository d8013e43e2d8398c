"""Shared comparison logic: CUDA path vs fp64 oracle on the same stored inputs."""
from __future__ import annotations

import numpy as np
import torch

import synthetic as S
from oracle import gsi_oracle as O

Y_TOL = 1e-2        # max-abs error <= Y_TOL * ||y_ref||_inf per token and map (bf16 weights, fp32 accumulation)
BAND = 1e-3         # gate bytes may differ only where |rho_oracle/eps - 1| < BAND
RHO_RTOL = 2e-5     # fp32 explicit residual vs fp64


def compare_group(x, P, Ws, eps, y_gpu, gate_gpu, rho_gpu=None, rows=None, static=False, fp8=False,
                  y_tol=Y_TOL, row_mask=None):
    """x [T][d] fp32 (cpu tensor), P stored basis (cpu tensor), Ws list of bf16
    cpu tensors (already row-sampled if ``rows`` given: then y_gpu holds the
    same sampled columns per map).  Returns a dict of statistics; raises on a
    violation of the acceptance bar.  ``fp8``: the oracle stores the image in FP8 first
    (Section 7.4).  ``row_mask`` (one boolean array per map, or None) restricts the
    comparison of y to the marked output rows; ``y_tol`` replaces Y_TOL."""
    xn = x.numpy()
    Pn = S.bits_of(P)
    Wn = [S.to_bf16_bits(W) for W in Ws]
    eps32 = float(np.float32(eps))
    pr = O.project(xn, Pn, eps32)
    gate_o = pr["gate"]
    gate_g = np.asarray(gate_gpu, dtype=np.uint8)
    with np.errstate(divide="ignore", invalid="ignore"):
        near = np.abs(pr["rho"] / eps32 - 1.0) < BAND if eps32 > 0 else np.zeros_like(gate_o, bool)
    mism = gate_o != gate_g
    bad = mism & ~near
    assert not bad.any(), (
        f"gate mismatch outside the +-{BAND} band at tokens {np.nonzero(bad)[0][:8]}, "
        f"rho={pr['rho'][bad][:8]}, eps={eps32}")
    # y against the oracle evaluated with the GPU's gate decision
    used = np.zeros_like(gate_g) if static else gate_g
    off = 0
    max_rel = 0.0
    for j, W in enumerate(Wn):
        M = O.image(W, Pn)
        if fp8:
            M = O.quantise_image_e4m3(M)["Mq"]
        y_ref = O.apply_map(M, W, pr["g"], pr["r"], used)
        o = W.shape[0]
        yg = np.asarray(y_gpu[:, off:off + o], dtype=np.float64)
        off += o
        scale = np.max(np.abs(y_ref), axis=1)          # ||y||_inf over ALL rows of the map
        if row_mask is not None and row_mask[j] is not None:
            keep = np.asarray(row_mask[j], bool)
            yg, y_ref = yg[:, keep], y_ref[:, keep]
            if yg.shape[1] == 0:
                continue
        err = np.max(np.abs(yg - y_ref), axis=1)
        finite = np.isfinite(scale) & (scale > 0)
        if finite.any():
            rel = err[finite] / scale[finite]
            max_rel = max(max_rel, float(rel.max()))
            assert rel.max() <= y_tol, f"map {j}: max-abs error {rel.max():.3e} * ||y||_inf > {y_tol}"
        zero = np.isfinite(scale) & (scale == 0)
        assert np.all(err[zero] == 0)
    if rho_gpu is not None:
        rg = np.asarray(rho_gpu, dtype=np.float64)
        ok = np.isfinite(pr["rho"]) & (pr["rho"] > 1e-5)
        if ok.any():
            assert np.max(np.abs(rg[ok] / pr["rho"][ok] - 1.0)) <= RHO_RTOL
    return dict(gate_rate=float(gate_g.mean()), near=int(near.sum()), flips=int(mism.sum()),
                max_rel_err=max_rel, oracle=pr)


def boundary_rows(n_rows, n_random, rng, grid=148):
    """Output rows a sampled-row test always looks at, besides `n_random` random ones: the first
    and last rows of the map, the edges of the 16-row tiles, the first and last rows of the
    slabs the CTAs own (image rows dealt in tiles of 16 over 148, 42 and 106 CTAs, the shares
    the benchmark's schedule uses; W rows dealt ceil(n / grid) per CTA), i.e. the ragged tails
    the kernels clamp."""
    rows = {0, 1, 15, 16, 17, n_rows - 17, n_rows - 16, n_rows - 2, n_rows - 1}
    tiles = (n_rows + 15) // 16
    for share in (grid, 42, 106):
        for c in (0, 1, share // 2, share - 2, share - 1):
            a = c * tiles // share if tiles >= share else min(c, tiles)
            rows.update({16 * a - 1, 16 * a, 16 * a + 15})
    per = (n_rows + grid - 1) // grid
    for c in (1, grid // 2, grid - 1):
        rows.update({c * per - 1, c * per, c * per + per - 1})
    rows = {r for r in rows if 0 <= r < n_rows}
    extra = rng.choice(n_rows, min(n_random, n_rows), replace=False)
    return np.array(sorted(rows | set(int(e) for e in extra)))


def image_ulp_check(W, P, wp_gpu):
    """The stored image is bf16_rne(W P) with fp32 accumulation: it must lie
    within one bf16 ulp of the fp64 product (half an ulp of rounding plus ties),
    widened by the fp32 accumulation error bound 2^-23 * (|W| |P|).  Returns the
    fraction of entries that differ from bf16_rne(M_fp64)."""
    Wb, Pb = S.to_bf16_bits(W), S.bits_of(P)
    M = O.image(Wb, Pb)
    got_bits = S.to_bf16_bits(wp_gpu)
    got = O.bf16_to_f64(got_bits)
    Wa = np.abs(O.bf16_to_f64(Wb))
    Pa = np.abs(O.bf16_to_f64(Pb)) if Pb.dtype == np.uint16 else np.abs(Pb.astype(np.float64))
    bound = 2.0 ** -8 * np.abs(M) + 2.0 ** -23 * (Wa @ Pa) + 1e-40
    worst = np.max(np.abs(got - M) / bound)
    assert worst <= 1.0, f"image error {worst:.3f} x the one-ulp bound"
    ref_bits = O.f64_to_bf16_rne(M)
    return float((ref_bits != got_bits).mean())
