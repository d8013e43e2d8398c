"""Pins for the fp64 oracle: what the paper and the mathematics fix.

None of these retype the oracle's formulae against themselves: each compares
the oracle with a library mat-vec in a special case, an exact identity, an
inequality the paper proves, exact rational arithmetic, or a printed value.
"""
import math
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import gsi_oracle as O
from oracle import report as R

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def f32_to_bf16_bits_trunc_safe(a):
    """Quantise fp64/fp32 numbers to values exactly representable in bf16 and
    return (bits, values) using numpy only (independent of the oracle's own
    decoder): keep the top 16 bits of the fp32 pattern after adding the
    round-to-nearest-even bias."""
    f = np.asarray(a, np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    bias = ((u >> 16) & 1) + 0x7FFF
    bits = ((u + bias) >> 16).astype(np.uint16)
    vals = (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    return bits, vals


def rand_problem(rng, o, d, k, T, p_f32=False, noise=0.05):
    Wb, W = f32_to_bf16_bits_trunc_safe(rng.normal(0, 0.02, (o, d)))
    q, _ = np.linalg.qr(rng.normal(size=(d, k)))
    if p_f32:
        P_store = q.astype(np.float32)
        P = P_store.astype(np.float64)
    else:
        P_store, P = f32_to_bf16_bits_trunc_safe(q)
    x = (q @ rng.normal(size=(k, T)) + noise * rng.normal(size=(d, T))).T.astype(np.float32)
    return Wb, W, P_store, P, q, np.ascontiguousarray(x)


# ---------------------------------------------------------------- conversions
def test_bf16_decode_matches_numpy_bit_view():
    bits = np.arange(0, 65536, dtype=np.uint32).astype(np.uint16)
    ref = (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    got = O.bf16_to_f64(bits)
    finite = np.isfinite(ref)
    assert np.array_equal(got[finite], ref[finite])
    assert np.array_equal(np.isnan(got), np.isnan(ref))


def test_bf16_rne_matches_integer_rounding_and_ties():
    rng = np.random.default_rng(0)
    v = np.concatenate([rng.normal(0, 1, 5000), rng.normal(0, 1e-3, 5000),
                        [1 + 2.0 ** -8, 1 + 3 * 2.0 ** -8, -(1 + 2.0 ** -8), 0.0, 255.5 * 2.0 ** -7]])
    # fp32-exact inputs so the numpy integer trick is a single rounding too
    v = v.astype(np.float32).astype(np.float64)
    ref_bits, _ = f32_to_bf16_bits_trunc_safe(v)
    assert np.array_equal(O.f64_to_bf16_rne(v), ref_bits)
    # ties to even, by hand
    assert O.f64_to_bf16_rne(np.array([1 + 2.0 ** -8]))[0] == 0x3F80
    assert O.f64_to_bf16_rne(np.array([1 + 3 * 2.0 ** -8]))[0] == 0x3F82


# ------------------------------------------------------------ special cases
def test_P1_eps_zero_fires_everything_and_equals_dense_matvec():
    """eps = 0: rho >= 0 always, so every token takes the slow path and the
    layer is the dense product W x (Section 3.2)."""
    rng = np.random.default_rng(1)
    Wb, W, Ps, P, q, x = rand_problem(rng, 24, 40, 8, 9)
    out = O.forward(x, Ps, 0.0, [Wb])
    assert out["gate"].all()
    ref = x.astype(np.float64) @ W.T
    assert np.max(np.abs(out["y"][0] - ref)) <= 1e-12 * np.max(np.abs(ref))


def test_P2_x_in_span_never_fires_and_image_is_exact():
    """x in span(P) with an fp32-stored orthonormal P: r = 0 up to the storage
    rounding of P, no token is gated, and M g = W x (Eq. (3.2) with r = 0)."""
    rng = np.random.default_rng(2)
    o, d, k, T = 16, 64, 16, 7
    Wb, W = f32_to_bf16_bits_trunc_safe(rng.normal(0, 0.02, (o, d)))
    # a basis whose entries are exact in fp32 *and* exactly orthonormal:
    # signed permutation columns scaled by 1 -> P^T P = I exactly
    perm = rng.permutation(d)[:k]
    P = np.zeros((d, k))
    P[perm, np.arange(k)] = rng.choice([-1.0, 1.0], k)
    x = (P @ rng.normal(size=(k, T))).T.astype(np.float32)
    out = O.forward(x, P.astype(np.float32), 1e-6, [Wb])
    assert not out["gate"].any()
    assert np.max(out["rho"]) == 0.0
    ref = x.astype(np.float64) @ W.T
    assert np.max(np.abs(out["y"][0] - ref)) <= 1e-13 * np.max(np.abs(ref))


def test_P2b_x_in_span_of_generic_basis():
    rng = np.random.default_rng(3)
    o, d, k, T = 12, 48, 10, 5
    Wb, W, Ps, P, q, _ = rand_problem(rng, o, d, k, T, p_f32=True)
    x64 = (P @ rng.normal(size=(k, T))).T
    x = x64.astype(np.float32)
    out = O.forward(x, Ps, 0.01, [Wb])
    # fp32 storage of P and x leaves rho ~ 1e-7, far below any eps in use
    assert np.max(out["rho"]) < 1e-6
    assert not out["gate"].any()
    ref = x.astype(np.float64) @ W.T
    assert np.max(np.abs(out["y"][0] - ref)) <= 1e-6 * np.max(np.abs(ref))


def test_P3_k_equals_d_square_orthogonal_basis():
    """k = d: the basis spans everything, r = 0 and y = W x."""
    rng = np.random.default_rng(4)
    o, d, T = 10, 16, 6
    Wb, W, Ps, P, q, x = rand_problem(rng, o, d, d, T, p_f32=True)
    out = O.forward(x, Ps, 0.05, [Wb])
    assert np.max(out["rho"]) < 1e-6 and not out["gate"].any()
    ref = x.astype(np.float64) @ W.T
    assert np.max(np.abs(out["y"][0] - ref)) <= 1e-6 * np.max(np.abs(ref))


# ------------------------------------------------------------------ identities
def test_P4_exact_decomposition_identity_for_any_basis():
    """Eq. (3.2): M g + W r = W x for every token and ANY matrix P (the stored
    bf16 basis is not orthonormal; the identity does not need it)."""
    rng = np.random.default_rng(5)
    Wb, W, Ps, P, q, x = rand_problem(rng, 20, 96, 24, 11)
    pr = O.project(x, Ps, 0.05)
    M = O.image(Wb, Ps)
    ones = np.ones(x.shape[0], np.uint8)
    y, y_alt = O.apply_map(M, Wb, pr["g"], pr["r"], ones, x=x, want_alt=True)
    ref = x.astype(np.float64) @ W.T
    scale = np.max(np.abs(ref))
    assert np.max(np.abs(y - ref)) <= 1e-12 * scale
    assert np.max(np.abs(y_alt - ref)) <= 1e-12 * scale
    # and on the oracle's own gate the two readings of the slow path agree
    y2, y2_alt = O.apply_map(M, Wb, pr["g"], pr["r"], pr["gate"], x=x, want_alt=True)
    assert np.max(np.abs(y2 - y2_alt)) <= 1e-12 * scale
    # a completely non-orthogonal "basis" still satisfies the identity
    Pb, Pv = f32_to_bf16_bits_trunc_safe(rng.normal(size=(96, 24)) * 0.1)
    pr = O.project(x, Pb, 0.05)
    M = O.image(Wb, Pb)
    y = O.apply_map(M, Wb, pr["g"], pr["r"], ones)
    assert np.max(np.abs(y - ref)) <= 1e-11 * scale


def test_image_is_W_times_P_by_library_matmul():
    rng = np.random.default_rng(6)
    Wb, W, Ps, P, q, x = rand_problem(rng, 17, 50, 6, 1)
    M = O.image(Wb, Ps)
    assert M.shape == (17, 6)
    assert np.max(np.abs(M - W @ P)) <= 1e-14
    # orientation: row a of M depends on row a of W only
    Wb2 = Wb.copy()
    Wb2[3] = 0
    M2 = O.image(Wb2, Ps)
    assert np.all(M2[3] == 0) and np.array_equal(np.delete(M2, 3, 0), np.delete(M, 3, 0))


def test_projection_pieces_by_library_routines():
    rng = np.random.default_rng(7)
    Wb, W, Ps, P, q, x = rand_problem(rng, 4, 72, 12, 13)
    pr = O.project(x, Ps, 0.05)
    x64 = x.astype(np.float64)
    g = x64 @ P
    r = x64 - g @ P.T
    assert np.max(np.abs(pr["g"] - g)) <= 1e-13
    assert np.max(np.abs(pr["r"] - r)) <= 1e-13
    assert np.allclose(pr["norm_x"], np.linalg.norm(x64, axis=1), rtol=1e-14)
    assert np.allclose(pr["norm_r"], np.linalg.norm(r, axis=1), rtol=1e-12)
    assert np.allclose(pr["rho"], pr["norm_r"] / pr["norm_x"], rtol=1e-15)


def test_P5_generator_basis_is_orthonormal_before_storage():
    import synthetic as S
    q = S.gen_basis(768, 64, 123).numpy()
    assert np.max(np.abs(q.T @ q - np.eye(64))) <= 1e-12
    pt = S.gen_true_basis(S.gen_basis(256, 32, 5), 24, 20, 9).numpy()
    assert np.max(np.abs(pt.T @ pt - np.eye(24))) <= 1e-12
    qq = S.gen_basis(256, 32, 5).numpy()
    # the 4 extra directions are orthogonal to span(Q)
    assert np.max(np.abs(qq.T @ pt[:, 20:])) <= 1e-12
    _, Pv = f32_to_bf16_bits_trunc_safe(q)
    dev = np.linalg.norm(Pv.T @ Pv - np.eye(64), 2)
    assert 1e-4 < dev < 5e-3  # bf16 storage loses orthonormality at the 1e-3 level


# ---------------------------------------------------------------- inequalities
def test_P6_theorem_3_1_error_bound_on_fast_tokens():
    """Theorem 3.1: on the fast path ||W x - M g|| = ||W r|| <= ||W||_2 eps ||x||;
    on the slow path the error is zero."""
    rng = np.random.default_rng(8)
    o, d, k, T = 32, 128, 32, 64
    Wb, W, Ps, P, q, x = rand_problem(rng, o, d, k, T, noise=0.03)
    eps = 0.052  # near the median rho of this draw, so both paths occur
    out = O.forward(x, Ps, eps, [Wb])
    gate = out["gate"].astype(bool)
    assert gate.any() and (~gate).any()  # the case exercises both paths
    dense = x.astype(np.float64) @ W.T
    err = np.linalg.norm(out["y"][0] - dense, axis=1)
    w2 = np.linalg.norm(W, 2)
    nx = np.linalg.norm(x.astype(np.float64), axis=1)
    assert np.all(err[~gate] <= w2 * np.float64(np.float32(eps)) * nx[~gate] * (1 + 1e-12))
    assert np.all(err[~gate] <= w2 * out["norm_r"][~gate] * (1 + 1e-12))
    assert np.all(err[~gate] > 0)
    assert np.all(err[gate] <= 1e-12 * np.max(np.abs(dense)))


def test_P7_monotone_in_k_for_nested_bases():
    """Proposition 2.3: rho(k+1) <= rho(k) for nested orthonormal bases, so the
    gated set shrinks as k grows."""
    rng = np.random.default_rng(9)
    d, T = 64, 40
    q, _ = np.linalg.qr(rng.normal(size=(d, 32)))
    x = rng.normal(size=(T, d)).astype(np.float32)
    prev_rho, prev_gate = None, None
    for k in (1, 2, 5, 8, 16, 31, 32):
        pr = O.project(x, np.ascontiguousarray(q[:, :k]).astype(np.float32), 0.8)
        if prev_rho is not None:
            assert np.all(pr["rho"] <= prev_rho + 1e-6)
            assert np.all(pr["gate"] <= prev_gate)
        prev_rho, prev_gate = pr["rho"], pr["gate"]


def test_P8_pythagoras_scale_and_rotation_invariance():
    rng = np.random.default_rng(10)
    o, d, k, T = 8, 80, 12, 9
    Wb, W, _, _, q, x = rand_problem(rng, o, d, k, T, p_f32=True, noise=0.3)
    # an fp64-orthonormal basis that survives fp32 storage only to 1e-7:
    Ps = q.astype(np.float32)
    pr = O.project(x, Ps, 0.05)
    x64 = x.astype(np.float64)
    pyth = np.sqrt(1.0 - np.sum(pr["g"] ** 2, axis=1) / np.sum(x64 ** 2, axis=1))
    assert np.allclose(pr["rho"], pyth, rtol=1e-5)
    # scale invariance (power-of-two scaling is exact in fp32)
    out1 = O.forward(x, Ps, 0.2, [Wb])
    out4 = O.forward(x * np.float32(4.0), Ps, 0.2, [Wb])
    assert np.allclose(out1["rho"], out4["rho"], rtol=1e-13)
    assert np.array_equal(out1["gate"], out4["gate"])
    assert np.allclose(4.0 * out1["y"][0], out4["y"][0], rtol=1e-12, atol=1e-15)
    # basis rotation P -> P Q leaves rho, the gate and y unchanged
    rot, _ = np.linalg.qr(rng.normal(size=(k, k)))
    Pr = (q @ rot).astype(np.float32)
    out_r = O.forward(x, Pr, 0.2, [Wb])
    assert np.allclose(out1["rho"], out_r["rho"], rtol=1e-5)
    assert np.array_equal(out1["gate"], out_r["gate"])
    assert np.allclose(out1["y"][0], out_r["y"][0], atol=1e-6 * np.max(np.abs(out1["y"][0])))


# ------------------------------------------------------------- brute force
def _exact_layer(W, P, x, eps):
    """Algorithm 1 in exact rational arithmetic (tiny shapes)."""
    o, d = len(W), len(W[0])
    k = len(P[0])
    g = [sum(P[i][j] * x[i] for i in range(d)) for j in range(k)]
    r = [x[i] - sum(P[i][j] * g[j] for j in range(k)) for i in range(d)]
    nr2 = sum(v * v for v in r)
    nx2 = sum(v * v for v in x)
    fast = nr2 < eps * eps * nx2  # rho < eps  <=>  ||r||^2 < eps^2 ||x||^2 (all >= 0)
    M = [[sum(W[a][i] * P[i][j] for i in range(d)) for j in range(k)] for a in range(o)]
    if fast:
        y = [sum(M[a][j] * g[j] for j in range(k)) for a in range(o)]
    else:
        y = [sum(W[a][i] * x[i] for i in range(d)) for a in range(o)]
    return g, r, nr2, nx2, (0 if fast else 1), y


def test_P11_brute_force_rational_arithmetic():
    rng = np.random.default_rng(11)
    o, d, k, T = 5, 12, 3, 8
    Wb, W = f32_to_bf16_bits_trunc_safe(rng.normal(0, 0.5, (o, d)))
    q, _ = np.linalg.qr(rng.normal(size=(d, k)))
    Pb, P = f32_to_bf16_bits_trunc_safe(q)
    x = (q @ rng.normal(size=(k, T)) + rng.normal(size=(d, T)) * np.linspace(0.0, 0.5, T)).T
    x = np.ascontiguousarray(x.astype(np.float32))
    eps = np.float32(0.25)
    out = O.forward(x, Pb, float(eps), [Wb])
    Wf = [[Fraction(float(v)) for v in row] for row in W]
    Pf = [[Fraction(float(v)) for v in row] for row in P]
    ef = Fraction(float(eps))
    seen = set()
    for t in range(T):
        xf = [Fraction(float(v)) for v in x[t]]
        g, r, nr2, nx2, gate, y = _exact_layer(Wf, Pf, xf, ef)
        seen.add(gate)
        assert out["gate"][t] == gate
        assert np.allclose(out["g"][t], [float(v) for v in g], rtol=0, atol=1e-14)
        assert np.allclose(out["r"][t], [float(v) for v in r], rtol=0, atol=1e-14)
        assert math.isclose(out["rho"][t], math.sqrt(nr2 / nx2), rel_tol=1e-12)
        assert np.allclose(out["y"][0][t], [float(v) for v in y], rtol=0, atol=1e-13)
    assert seen == {0, 1}


def test_P11b_tokens_constructed_on_either_side_of_the_threshold():
    """x = 4 e_1 + t e_2 with P = [e_1]: rho = t / sqrt(16 + t^2) exactly.
    With eps = 0.6, rho = 0.6 at t = 3 (a 3-4-5 triangle): the strict test
    rho < eps must fire exactly at equality and above."""
    d = 8
    P = np.zeros((d, 1), np.float32)
    P[0, 0] = 1.0
    Wb, W = f32_to_bf16_bits_trunc_safe(np.arange(1, 2 * d + 1, dtype=np.float64).reshape(2, d) / 8)
    ts = np.array([2.9990234375, 3.0, 3.0009765625, 0.0, 100.0], np.float32)
    x = np.zeros((len(ts), d), np.float32)
    x[:, 0] = 4.0
    x[:, 1] = ts
    # eps chosen so that eps*||x|| is exact: 0.6 is not representable, so use
    # the 3-4-5 triangle scaled: rho(t=3) = 3/5; compare against eps = 0.6f.
    eps = np.float32(0.6)
    out = O.forward(x, P, float(eps), [Wb])
    epsd = float(eps)
    expected = [0 if (float(t) / math.sqrt(16 + float(t) ** 2) < epsd) else 1 for t in ts]
    assert list(out["gate"]) == expected
    assert expected[0] == 0 and expected[2] == 1 and expected[3] == 0 and expected[4] == 1
    # fast tokens: y = W[:,0]*4 ; slow tokens: y = W x
    for t in range(len(ts)):
        ref = W @ x[t].astype(np.float64) if expected[t] else W[:, 0] * 4.0
        assert np.allclose(out["y"][0][t], ref, rtol=1e-15, atol=0)


def test_C3_zero_and_nonfinite_inputs():
    P = np.eye(4, 2, dtype=np.float32)
    Wb, W = f32_to_bf16_bits_trunc_safe(np.ones((3, 4)))
    x = np.zeros((2, 4), np.float32)
    x[1, 2] = np.inf
    out = O.forward(x, P, 0.05, [Wb])
    assert list(out["gate"]) == [1, 1]          # 0 < 0 is false; NaN compares false
    assert np.all(out["y"][0][0] == 0.0)
    assert np.isnan(out["rho"][0])


def test_gate_override_and_row_sampling():
    rng = np.random.default_rng(12)
    Wb, W, Ps, P, q, x = rand_problem(rng, 16, 32, 4, 6, noise=0.2)
    full = O.forward(x, Ps, 0.1, [Wb])
    rows = np.array([0, 5, 15])
    part = O.forward(x, Ps, 0.1, [Wb], rows=[rows])
    assert np.array_equal(part["y"][0], full["y"][0][:, rows])
    flipped = (1 - full["gate"]).astype(np.uint8)
    alt = O.forward(x, Ps, 0.1, [Wb], gate_override=flipped)
    assert np.array_equal(alt["gate"], full["gate"])
    dense = x.astype(np.float64) @ W.T
    was_fast = full["gate"] == 0
    assert np.allclose(alt["y"][0][was_fast], dense[was_fast], atol=1e-12)


# ---------------------------------------------------- printed worked examples
def test_P9_effective_speedup_reproduces_printed_tables():
    rows = 0
    for line in open(os.path.join(GOLDEN, "eq34_speedup_table.txt")):
        if line.startswith("#") or not line.strip():
            continue
        _, d, k, _, f, s = line.split()
        got = R.effective_speedup(float(f) / 100.0, int(d) / int(k))
        # printed to one decimal; f itself is printed to 0.1 %, which moves S by
        # at most |dS/df| * 5e-4
        ratio = int(d) / int(k)
        slack = 0.0005 * got * got * (1 - 1 / ratio)
        assert abs(got - float(s)) <= 0.05 + slack + 1e-9, line
        rows += 1
    assert rows == 26


def test_P10_effective_parameters_and_storage_examples():
    frac = R.effective_parameter_fraction(0.998, 256, 4096)
    assert round(frac, 4) == 0.0644
    peff = R.effective_parameters([(1, 6e9 / 4096, 4096, 256, 0.998)])
    assert abs(peff - 386e6) / 386e6 < 0.005
    assert abs(R.image_storage_bytes(28, 32768, 256) / 1e6 - 469) < 1
    assert abs(R.basis_storage_bytes(28, 4096, 256) / 1e6 - 59) < 0.5


# ---- online basis extension (Sections 5.4 and 7.2) ----------------------------------
def _partial_basis(d, k_act, k_cap, seed, dtype=np.float32):
    rng = np.random.default_rng(seed)
    q, _ = np.linalg.qr(rng.standard_normal((d, k_act)))
    P = np.zeros((d, k_cap), dtype)
    P[:, :k_act] = q.astype(dtype)
    return P, rng


def test_E1_extension_vector_is_the_last_column_of_a_library_qr():
    """Appending the twice-orthogonalised residual is Gram-Schmidt on [V x]: the new vector
    equals (up to sign) the last column of numpy's Householder QR of that matrix."""
    d, k_act = 96, 12
    P, rng = _partial_basis(d, k_act, 16, 41)
    x = rng.standard_normal(d)
    out = O.extend(P, k_act, x, 0.05)
    assert out["extended"]
    q, _ = np.linalg.qr(np.concatenate([P[:, :k_act].astype(np.float64), x[:, None]], axis=1))
    last = q[:, -1]
    assert min(np.linalg.norm(out["v"] - last), np.linalg.norm(out["v"] + last)) < 1e-6
    assert abs(np.linalg.norm(out["v"]) - 1.0) < 1e-15
    # rho is the first-pass residual ratio: the same number the layer's gate computes
    pr = O.project(x.astype(np.float32)[None, :], np.ascontiguousarray(P[:, :k_act]), 0.05)
    x32 = x.astype(np.float32).astype(np.float64)
    out32 = O.extend(P, k_act, x32, 0.05)
    assert abs(out32["rho"] - pr["rho"][0]) <= 1e-14 * pr["rho"][0]


def test_E2_second_orthogonalisation_is_needed_and_enough():
    """With a stored basis that is orthonormal only to ~1e-7 (fp32 storage) and a token that
    is almost inside the span, one Gram-Schmidt pass leaves V^T v ~ 1e-7 / rho; the second
    pass brings it to rounding level.  A dropped second pass fails this pin."""
    d, k_act = 128, 24
    P, rng = _partial_basis(d, k_act, 32, 42)
    V = P[:, :k_act].astype(np.float64)
    x = V @ rng.standard_normal(k_act) + 1e-3 * rng.standard_normal(d)
    out = O.extend(P, k_act, x, 1e-6)
    assert out["extended"] and 1e-4 < out["rho"] < 1e-2
    assert np.abs(V.T @ out["v"]).max() < 1e-11
    r1 = x - V @ (V.T @ x)                      # one pass only
    one = r1 / np.linalg.norm(r1)
    assert np.abs(V.T @ one).max() > 1e-6 * 0.1  # visibly worse: what the second pass removes


def test_E3_special_cases():
    d = 40
    rng = np.random.default_rng(43)
    x = rng.standard_normal(d)
    # empty basis: the new vector is x / ||x||, rho = 1
    out = O.extend(np.zeros((d, 8), np.float32), 0, x, 0.5)
    assert out["extended"] and abs(out["rho"] - 1.0) < 1e-15
    assert np.allclose(out["v"], x / np.linalg.norm(x), rtol=0, atol=1e-15)
    # token inside the span: below any reasonable threshold, nothing appended
    P, rng = _partial_basis(d, 6, 8, 44, np.float64)
    P32 = P.astype(np.float32)
    xin = P32[:, :6].astype(np.float64) @ rng.standard_normal(6)
    out = O.extend(P32, 6, xin, 1e-3)
    assert not out["extended"] and out["rho"] < 1e-6
    # full basis: nothing appended even above the threshold
    out = O.extend(P32[:, :6].copy(), 6, x, 0.05)
    assert not out["extended"] and out["rho"] > 0.05
    # threshold is strict: rho == tau does not extend
    r = O.extend(P32, 6, x, 0.0)["rho"]
    assert not O.extend(P32, 6, x, r)["extended"]
    assert O.extend(P32, 6, x, np.nextafter(r, 0.0))["extended"]


def test_E4_after_the_extension_the_token_lies_in_the_span():
    """Storing v (here in fp32) as column k_act puts x inside the span of the stored basis:
    its residual ratio drops from rho to storage rounding level, and the image column of the
    extended basis is W v (Section 4.2 applied to the new column)."""
    d, k_act, o = 80, 10, 24
    P, rng = _partial_basis(d, k_act, 16, 45)
    x = rng.standard_normal(d).astype(np.float32)
    out = O.extend(P, k_act, x.astype(np.float64), 0.05)
    assert out["extended"] and out["rho"] > 0.5
    P2 = P.copy()
    P2[:, k_act] = out["v"].astype(np.float32)
    after = O.project(x[None, :], np.ascontiguousarray(P2[:, :k_act + 1]), 0.05)
    assert after["rho"][0] < 1e-6 and after["gate"][0] == 0
    W = O.f64_to_bf16_rne(rng.standard_normal((o, d)) * 0.1)
    col = O.image(W, np.ascontiguousarray(P2[:, k_act:k_act + 1]))
    assert np.allclose(col[:, 0], O.bf16_to_f64(W) @ P2[:, k_act].astype(np.float64), rtol=0, atol=1e-14)


# ---------------------------------------------------------------- FP8 image (Section 7.4)
def _e4m3_table():
    """Every non-negative finite E4M3 value from the format's definition, by
    exact rational arithmetic (independent of the oracle's decoder)."""
    vals = []
    for e in range(16):
        for m in range(8):
            if e == 15 and m == 7:
                continue
            vals.append(Fraction(m, 8) * Fraction(1, 64) if e == 0
                        else (1 + Fraction(m, 8)) * Fraction(2) ** (e - 7))
    return vals


def test_F1_e4m3_decode_is_the_format_definition():
    codes = np.arange(256, dtype=np.uint8)
    v = O.e4m3_decode(codes)
    table = _e4m3_table()
    assert len(table) == 127
    assert [Fraction(float(x)) for x in v[:127]] == table          # exact, all finite codes
    assert np.isnan(v[0x7F]) and np.isnan(v[0xFF])
    np.testing.assert_array_equal(v[128:255], -v[0:127])
    # landmarks: smallest subnormal, smallest normal, one, largest finite
    assert v[0x01] == 2.0 ** -9 and v[0x08] == 2.0 ** -6 and v[0x38] == 1.0 and v[0x7E] == 448.0
    assert np.all(np.diff(v[:127]) > 0)


def test_F2_e4m3_encode_is_nearest_with_ties_to_even_by_brute_force():
    table = _e4m3_table()
    tf = np.array([float(t) for t in table])
    rng = np.random.default_rng(7)
    samples = np.concatenate([
        tf,                                               # the values themselves
        (tf[:-1] + tf[1:]) / 2,                           # every midpoint (exact in fp32: 5 significant bits)
        np.nextafter(((tf[:-1] + tf[1:]) / 2).astype(np.float32), np.float32(np.inf)).astype(np.float64),
        np.nextafter(((tf[:-1] + tf[1:]) / 2).astype(np.float32), np.float32(0)).astype(np.float64),
        np.abs(rng.normal(0, 100, 4000)), np.abs(rng.normal(0, 1, 4000)), np.abs(rng.normal(0, 0.01, 4000)),
    ]).astype(np.float32)
    samples = samples[samples <= 448]
    got = O.e4m3_encode(samples)
    for s, c in zip(samples.tolist(), got.tolist()):
        fs = Fraction(s)
        dist = [abs(fs - t) for t in table]
        best = min(dist)
        cands = [i for i, dd in enumerate(dist) if dd == best]
        want = cands[0] if len(cands) == 1 else [i for i in cands if i % 2 == 0][0]
        assert c == want, (s, c, want)
    # sign, saturation, NaN
    neg = O.e4m3_encode(-samples)
    np.testing.assert_array_equal(neg & 0x7F, got)
    assert np.all((neg >> 7) == 1)
    big = np.array([448.0, 449.0, 463.9, 464.0, 1e6, np.inf, -np.inf, -500.0], np.float32)
    np.testing.assert_array_equal(O.e4m3_encode(big), [0x7E] * 6 + [0xFE] * 2)
    assert O.e4m3_encode(np.array([np.nan], np.float32))[0] & 0x7F == 0x7F


def test_F3_e4m3_encode_agrees_with_the_library_conversion():
    torch = pytest.importorskip("torch")
    if not hasattr(torch, "float8_e4m3fn"):
        pytest.skip("no float8 in this torch")
    rng = np.random.default_rng(11)
    v = np.concatenate([rng.normal(0, 120, 20000), rng.normal(0, 1, 20000), rng.normal(0, 0.004, 20000)])
    v = np.clip(v, -448, 448).astype(np.float32)
    lib = torch.from_numpy(v).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    got = O.e4m3_encode(v)
    # -0 and +0 are the same number
    same = (lib == got) | (((lib | got) & 0x7F) == 0)
    assert same.all()


def test_F4_fp8_image_scales_codes_and_error_bound():
    rng = np.random.default_rng(3)
    Wb, W, P_store, P, q, x = rand_problem(rng, 40, 96, 16, 4)
    M = O.image(Wb, P_store)
    M[7] = 0.0                                             # a zero row
    M[9, 3] = 50.0 * np.abs(M[9]).max()                    # a row with a wide spread (subnormal codes)
    qz = O.quantise_image_e4m3(M)
    codes, scales, Mq = qz["codes"], qz["scales"], qz["Mq"]
    _, mb = f32_to_bf16_bits_trunc_safe(M)                 # the BF16 image, by numpy
    amax = np.abs(mb).max(axis=1)
    # scale: amax / 448 as one fp32 division (numpy float32 arithmetic), 1 for the zero row
    want_scale = np.where(amax > 0, amax.astype(np.float32) / np.float32(448), np.float32(1))
    np.testing.assert_array_equal(scales, want_scale)
    assert np.all(codes[7] == 0) and np.all(Mq[7] == 0)
    # the largest element of every other row takes the largest code
    for a in range(40):
        if a != 7:
            assert codes[a, np.abs(mb[a]).argmax()] & 0x7F == 0x7E
    # the stored image is decode(code) * scale, and lies within half a code spacing of the BF16 image
    np.testing.assert_array_equal(Mq, O.e4m3_decode(codes) * scales.astype(np.float64)[:, None])
    t = np.abs(mb) / scales.astype(np.float64)[:, None]
    spacing = np.where(t < 2.0 ** -6, 2.0 ** -9, 2.0 ** (np.floor(np.log2(np.maximum(t, 2.0 ** -6))) - 3))
    err = np.abs(Mq - mb) / scales.astype(np.float64)[:, None]
    assert np.all(err <= spacing / 2 * (1 + 1e-6) + 1e-6 * t)
    assert np.any(t[9] < 2.0 ** -6)                        # the subnormal range is exercised
    # forward(fp8_image=True) is forward() with the image replaced by Mq
    Ws = [Wb]
    a = O.forward(x, P_store, 0.05, Ws, fp8_image=True)
    g = a["g"]
    M0 = O.quantise_image_e4m3(O.image(Wb, P_store))["Mq"]
    fast = a["gate"] == 0
    if fast.any():
        np.testing.assert_allclose(a["y"][0][fast], (g @ M0.T)[fast], rtol=1e-12, atol=1e-14)


def test_F5_fp8_image_output_error_is_bounded_against_the_unquantised_layer():
    """y with the FP8 image differs from y with the exact image by at most
    sum_j |Mq_ij - M_ij| |g_j|, and every |Mq_ij - M_ij| is at most 2^-4 |bf16(M_ij)| (normal
    codes) or scale * 2^-10 (subnormal codes) plus the BF16 rounding 2^-9 |M_ij|."""
    rng = np.random.default_rng(21)
    Wb, W, P_store, P, q, x = rand_problem(rng, 64, 128, 32, 6)
    a = O.forward(x, P_store, 0.05, [Wb])
    b = O.forward(x, P_store, 0.05, [Wb], fp8_image=True)
    np.testing.assert_array_equal(a["gate"], b["gate"])          # the gate does not see the image
    M = O.image(Wb, P_store)
    qz = O.quantise_image_e4m3(M)
    per_entry = np.maximum(2.0 ** -4 * np.abs(M) * (1 + 2.0 ** -8), qz["scales"].astype(np.float64)[:, None] * 2.0 ** -10) \
        + 2.0 ** -9 * np.abs(M)
    assert np.all(np.abs(qz["Mq"] - M) <= per_entry)
    bound = np.abs(a["g"]) @ per_entry.T                          # [T][o]
    diff = np.abs(b["y"][0] - a["y"][0])
    assert np.all(diff <= bound * (1 + 1e-12) + 1e-300)
    assert diff.max() > 0                                          # the quantisation is visible
    # and in the aggregate it is a few percent of ||y||_inf, not more (3 mantissa bits)
    assert diff.max() <= 0.05 * np.abs(a["y"][0]).max()
