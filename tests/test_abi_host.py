"""Host-side checks of the C ABI that need no GPU: the library loads, exports
every symbol the header declares, and rejects bad arguments before touching a
device."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "gsi.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = set(re.findall(r"\b(gsi_[a-z0-9_]+)\s*\(", text))
    return sorted(names)


def test_library_exports_every_declared_symbol():
    import paper_2605_03109_b200 as G
    names = declared_symbols()
    assert len(names) >= 19
    for n in names:
        assert hasattr(G.lib, n), n
    assert set(G.EXPORTED) == set(names)


def test_status_strings():
    import paper_2605_03109_b200 as G
    assert G.gsi_status_string(0) == "ok"
    assert "workspace" in G.gsi_status_string(6)
    assert "timed out" in G.gsi_status_string(5)


def test_descriptor_validation_without_a_device():
    import paper_2605_03109_b200 as G
    ok = G.gsi_workspace_bytes(4096, 256, [4096, 16384], 0.05, 1)
    assert ok > (4096 + 16384) * 256 * 2
    assert G.gsi_workspace_bytes(4096, 250, [4096], 0.05, 1) == 0       # k not a multiple of 8
    assert G.gsi_workspace_bytes(4096, 256, [4097], 0.05, 1) == 0       # d_out not a multiple of 8
    assert G.gsi_workspace_bytes(4100, 256, [4096], 0.05, 1) == 0       # d not a multiple of 8
    assert G.gsi_workspace_bytes(64, 128, [64], 0.05, 1) == 0           # k > d
    assert G.gsi_workspace_bytes(4096, 2048, [64], 0.05, 1) == 0        # k > 1024
    assert G.gsi_workspace_bytes(4096, 256, [4096], 0.05, 65) == 0      # batch too large
    assert G.gsi_workspace_bytes(4096, 256, [4096], -1.0, 1) == 0       # negative eps
    assert G.gsi_workspace_bytes(4096, 256, [4096], float("nan"), 1) == 0
    assert G.gsi_workspace_bytes(4096, 256, [8] * 9, 0.05, 1) == 0      # too many maps
    assert G.gsi_workspace_bytes(4096, 0, [4096], 0.05, 1, flags=G.GSI_FLAG_DENSE) > 0
    # workspace grows with the batch
    assert G.gsi_workspace_bytes(4096, 256, [4096], 0.05, 64) > G.gsi_workspace_bytes(4096, 256, [4096], 0.05, 1)


def test_null_and_misaligned_arguments_are_rejected_on_the_host():
    import paper_2605_03109_b200 as G
    from paper_2605_03109_b200.binding import make_desc
    lib = G.lib
    INVALID, UNSUPPORTED, WORKSPACE = 1, 2, 6
    assert lib.gsi_build_image(None, None, 8, 8, 8, 0, None, None) == INVALID
    assert lib.gsi_build_image(256, 256, 8, 8, 8, 0, 257, None) == INVALID      # misaligned output
    assert lib.gsi_build_image(256, 512, 9, 8, 8, 0, 1024, None) == UNSUPPORTED
    assert lib.gsi_build_image(256, 512, 8, 8, 8, 7, 1024, None) == INVALID     # bad dtype
    desc = make_desc(64, 8, [64], 0.05, 1)
    h = C.c_void_p()
    warr = (C.c_void_p * 1)(4096)
    assert lib.gsi_create(C.byref(desc), None, 4096, 4096, 1 << 30, None, C.byref(h)) == INVALID
    assert lib.gsi_create(C.byref(desc), warr, None, 4096, 1 << 30, None, C.byref(h)) == INVALID
    assert lib.gsi_create(C.byref(desc), warr, 4096, 4096 + 8, 1 << 30, None, C.byref(h)) == INVALID
    assert lib.gsi_create(C.byref(desc), warr, 4096, 4096, 16, None, C.byref(h)) == WORKSPACE
    assert lib.gsi_create(C.byref(desc), warr, 4096, 4096, 1 << 30, None, None) == INVALID
    assert h.value is None
    assert lib.gsi_forward(None, None, None, None, None) == INVALID
    assert lib.gsi_forward_n(None, None, 1, None, None, None, None) == INVALID
    assert lib.gsi_destroy(None) == INVALID
    assert lib.gsi_stack_create(0, None, None, 0, None, C.byref(h)) == INVALID
    assert lib.gsi_stack_step(None, None) == INVALID
    assert lib.gsi_stack_destroy(None) == INVALID
    assert lib.gsi_stack_workspace_bytes(0) == 0
    assert lib.gsi_stack_workspace_bytes(84) > 0
    assert lib.gsi_stack_set_concurrent(None, 0, 1) == INVALID
    assert lib.gsi_stack_set_mode(None, 0) == INVALID
    assert lib.gsi_stack_set_spin_limit(None, 1) == INVALID
    assert lib.gsi_extend_basis(None, 4096, 0.05, 4096, None, None, None) == INVALID
    assert lib.gsi_get_status(None, None) == INVALID
