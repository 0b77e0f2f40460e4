"""The C-ABI library loads and exports every symbol declared in include/vgc.h; host-side argument
checks reject bad calls before anything is enqueued (no GPU needed)."""
import ctypes
import os
import re

import pytest

import paper_1802_06058_b200 as vgc

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "vgc.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(vgc_[a-z_0-9]+)\s*\(", text)))


@pytest.fixture(scope="module")
def lib():
    vgc.build()
    return vgc.load_library()


def test_every_declared_symbol_is_exported(lib):
    names = _declared_functions()
    assert len(names) >= 9
    for name in names:
        assert hasattr(lib, name), name
    assert set(vgc.EXPORTS) <= set(names)


def test_status_strings_and_version(lib):
    assert lib.vgc_status_string(0) == b"ok"
    assert lib.vgc_status_string(3) == b"workspace too small"
    assert lib.vgc_version() >= 1000


def test_workspace_queries_are_pure_host_functions(lib):
    n = 138344128
    need = lib.vgc_compress_workspace_bytes(n, 16)
    assert 8 * n < need < 8 * n + (4 << 20)
    assert lib.vgc_sqgrad_linear_workspace_bytes(32, 256, 128) % 256 == 0
    assert lib.vgc_sqgrad_conv_workspace_bytes(32, 64, 56, 56, 64, 3, 3, 1, 1, 1, 1) > 0
    assert lib.vgc_sqgrad_conv_workspace_bytes(32, 64, 2, 2, 64, 3, 3, 1, 1, 0, 0) == 0   # kernel > image


def test_sqgrad_workspace_follows_the_work_plan(lib):
    """A launch whose tiles are shared between thread blocks needs two partial tiles (64 KB each) per block beside the
    status word; one whose blocks take whole tiles needs the status word only."""
    shared = lib.vgc_sqgrad_conv_workspace_bytes(32, 64, 56, 56, 64, 1, 1, 1, 1, 0, 0)        # one tile, 3136 slices
    assert shared >= 256 + 2 * 148 * 65536
    whole = lib.vgc_sqgrad_conv_workspace_bytes(2, 640, 8, 8, 1280, 1, 1, 1, 1, 0, 0)         # 50 tiles, 4 slices
    assert 256 <= whole < 65536
    assert lib.vgc_sqgrad_conv_batch_workspace_bytes(8, 32, 256, 14, 14, 1024, 1, 1, 1, 1, 0, 0) >= 256
    assert lib.vgc_sqgrad_conv_batch_workspace_bytes(0, 32, 256, 14, 14, 1024, 1, 1, 1, 1, 0, 0) == 0


def test_compress_rejects_bad_arguments_on_the_host(lib):
    fake = ctypes.c_void_p(0x1000)          # never dereferenced: every call below fails validation first
    msg = vgc._MessageStruct(0x1000, 16, 0x1000, 0x1000, 0x1000, 0x1000, None, 0x1000)
    call = lambda n, K, alpha, zeta, g=fake, ws=fake, ws_bytes=1 << 40: lib.vgc_compress(
        g, fake, fake, fake, n, fake, K, alpha, zeta, ctypes.byref(msg), ws, ws_bytes, None)
    assert call(0, 1, 2.0, 0.999) == 0                        # empty buffer: no-op
    assert call((1 << 28) + 1, 1, 2.0, 0.999) == 1            # index would not fit 28 bits
    assert call(100, 0, 2.0, 0.999) == 1
    assert call(100, 1, -1.0, 0.999) == 1
    assert call(100, 1, float("nan"), 0.999) == 1
    assert call(100, 1, float("inf"), 0.999) == 1
    assert call(100, 1, 2.0, float("nan")) == 1
    assert call(100, 1, 2.0, 0.999, g=ctypes.c_void_p(0x1004)) == 1     # misaligned
    assert call(100, 1, 2.0, 0.999, g=None) == 1
    assert call(100, 1, 2.0, 0.999, ws_bytes=16) == 3         # workspace too small


def test_decode_and_sqgrad_reject_bad_arguments_on_the_host(lib):
    fake = ctypes.c_void_p(0x1000)
    views = (vgc._ViewStruct * 1)(vgc._ViewStruct(0x1000, 0x1000, None, 16))
    assert lib.vgc_decode_accumulate(views, 0, fake, 1, 1.0, fake, 10, fake, None) == 0
    assert lib.vgc_decode_accumulate(views, 1, fake, 1, 1.0, fake, 10, fake, None) == 1   # null group_exp
    assert lib.vgc_decode_accumulate(views, 1, fake, 1, 1.0, None, 10, fake, None) == 1
    assert lib.vgc_sqgrad_linear(fake, fake, 4, 0, 8, 1.0, 0, fake, None, 0, None) == 0   # empty layer
    # empty mini-batch, accumulate: nothing to add, no workspace needed, nothing enqueued
    assert lib.vgc_sqgrad_linear(None, None, 0, 8, 8, 1.0, 1, fake, None, 0, None) == 0
    assert lib.vgc_sqgrad_conv(None, None, 0, 3, 8, 8, 5, 3, 3, 1, 1, 1, 1, 1.0, 1, fake, None, 0, None) == 0
    assert lib.vgc_sqgrad_linear_workspace_bytes(0, 8, 8) == 0
    assert lib.vgc_sqgrad_linear(fake, fake, 4, 8, 8, 1.0, 0, fake, None, 0, None) == 3   # B > 0 needs its workspace
    assert lib.vgc_sqgrad_linear(fake, fake, -1, 8, 8, 1.0, 0, fake, None, 0, None) == 1
    assert lib.vgc_sqgrad_linear(None, fake, 4, 8, 8, 1.0, 0, fake, None, 0, None) == 1
    assert lib.vgc_sqgrad_conv(fake, fake, 2, 3, 4, 4, 5, 7, 7, 1, 1, 0, 0, 1.0, 0, fake, None, 0, None) == 1


def test_binding_refuses_cpu_tensors():
    import torch
    t = torch.zeros(8)
    with pytest.raises(TypeError):
        vgc.vgc_sqgrad_linear(t.view(2, 4), t.view(2, 4), 1.0, torch.zeros(16))
