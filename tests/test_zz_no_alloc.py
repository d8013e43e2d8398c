"""The allocation-free entry point against the regular one.

Some callers of this library may not allocate device memory at all: a plugin
inside an application that owns the whole GPU heap, code invoked while another
component's stream capture is open, a hot path that must never enter the CUDA
allocator.  ``gsi_forward_static`` serves them from a scratch array compiled
into the library.  This test drives it through the C ABI, twice in a row (the
array keeps the first call's contents, so the second call proves the clearing),
and compares with ``gsi_forward_n`` and with the fp64 oracle.  It is collected last on purpose.
"""
import ctypes as C

import numpy as np
import pytest
import torch

import synthetic as S
from _parity import Y_TOL, compare_group

pytestmark = pytest.mark.gpu


def _case(seed, d, k, d_out, n_tokens):
    q = S.gen_basis(d, k, seed)
    P = S.store_basis(q)
    Ws = [S.gen_weight(o, d, seed + 1 + j) for j, o in enumerate(d_out)]
    pt = S.gen_true_basis(q, k // 2, k // 2, seed + 9)
    x, _ = S.gen_activations(pt, n_tokens, 0.003, 0.0,
                             dict(z=seed + 3, noise=seed + 4, outlier_mask=0, outlier_values=0))
    x[::2] = torch.randn((len(range(0, n_tokens, 2)), d),
                         generator=torch.Generator().manual_seed(seed))  # these fire
    return x.contiguous(), P, Ws


def test_static_entry_point_matches_workspace_entry_point_twice():
    import paper_2605_03109_b200 as G
    eps = 0.05
    for seed, (d, k, d_out, n) in enumerate([(768, 64, (3072,), 4), (4096, 256, (1024, 512), 3)]):
        x, P, Ws = _case(100 + seed, d, k, d_out, n)
        Wd = [W.cuda() for W in Ws]
        Pd, xd = P.cuda(), x.cuda()
        ref_layer = G.Layer(Wd, Pd, eps, max_tokens=n)
        y_ref, gate_ref, rho_ref = ref_layer.forward(xd)
        W_P = torch.cat([G.gsi_build_image(W, Pd) for W in Wd], dim=0).contiguous()
        torch.cuda.synchronize()
        assert gate_ref.any() and not gate_ref.all()      # both paths are exercised
        y = torch.empty_like(y_ref)
        gate = torch.empty_like(gate_ref)
        rho = torch.empty_like(rho_ref)
        for call in range(2):
            y.fill_(float("nan"))
            gate.fill_(7)
            G.gsi_forward_static(Wd, Pd, W_P, eps, xd, y, gate, rho)
            torch.cuda.synchronize()
            assert torch.equal(gate, gate_ref), f"call {call}"
            scale = y_ref.abs().amax(dim=1, keepdim=True)
            assert ((y - y_ref).abs() <= Y_TOL * scale).all(), f"call {call}"
            assert torch.allclose(rho, rho_ref, rtol=1e-5, atol=0), f"call {call}"
            # ... and against the oracle itself, at the acceptance bar of every other entry point
            compare_group(x, P, Ws, eps, y.cpu().numpy(), gate.cpu().numpy(), rho.cpu().numpy())


def test_static_entry_point_rejects_what_its_scratch_cannot_hold():
    import paper_2605_03109_b200 as G
    lib = G.lib
    warr = (C.c_void_p * 1)(4096)
    darr = (C.c_int * 1)(64)
    UNSUPPORTED, INVALID = 2, 1

    def call(d=1024, k=64, n=1, P=4096, WP=8192, x=4096, y=4096, gate=4096):
        return lib.gsi_forward_static(warr, darr, 1, P, 0, WP, d, k, 0.05, x, n, y, gate, None, None)

    assert call(n=5) == UNSUPPORTED          # more tokens than the array holds
    assert call(k=1024, d=2048) == UNSUPPORTED
    assert call(d=32768) == UNSUPPORTED
    assert call(k=60) == UNSUPPORTED
    assert call(P=None) == INVALID
    assert call(x=None) == INVALID
    assert call(n=0) == 0                    # nothing to do, nothing launched
