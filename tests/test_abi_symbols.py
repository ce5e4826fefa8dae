"""The built library loads without a GPU and exports every entry point that include/ais.h declares (CPU only)."""

import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "ais.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ais_[a-z0-9_]+)\s*\(", text)))


def test_header_declares_the_path():
    names = _declared()
    for must in ("ais_quantize_fp8", "ais_logprob_fwd", "ais_diagnostics", "ais_loss_bwd", "ais_workspace_bytes"):
        assert must in names


def test_library_exports_every_declared_symbol():
    from paper_2605_13907_b200 import build
    lib_path = build.build_library()
    lib = ctypes.CDLL(lib_path)
    for name in _declared():
        assert hasattr(lib, name), name
    lib.ais_version.restype = ctypes.c_int
    assert lib.ais_version() >= 100
    lib.ais_strerror.restype = ctypes.c_char_p
    assert b"workspace" in lib.ais_strerror(-4)


def test_host_side_validation_needs_no_gpu():
    import paper_2605_13907_b200 as ais
    p = ais.default_params()
    assert p.C == 5.0 and abs(p.delta - 0.02) < 1e-7 and abs(p.gamma - 1.2) < 1e-6 and p.alpha_override != p.alpha_override
    good = ais.binding.make_shape(1000, 4096, 151936, 8, 8, 128)
    assert ais.workspace_bytes(good, p) >= ais.workspace_min_bytes(good, p) > 0
    bad = ais.binding.make_shape(1000, 4100, 151936, 8, 8, 128)        # d not a multiple of 128
    assert ais.workspace_bytes(bad, p) == 0
    p.C = 0.5                                                           # truncation below 1 is rejected
    assert ais.workspace_bytes(good, p) == 0
    import torch
    with pytest.raises(ais.AisError):                                   # CPU tensors are refused: no CPU path
        ais.quantize_fp8(torch.zeros(4, 128, dtype=torch.bfloat16), 128)


def test_microscaling_entry_points_validate_on_the_host():
    """Sizes of the packed scale arrays, the shape rules of the two block-scaled variants and the argument checks that
    come before any device call."""
    import paper_2605_13907_b200 as ais
    lib = ais.lib()
    assert ais.mx_scale_bytes(1, 128) == 2 * 512                       # rows padded to 256: two chunks of 128 rows
    assert ais.mx_scale_bytes(256, 4096) == 2 * 32 * 512
    assert ais.mx_scale_bytes(257, 4096) == 4 * 32 * 512
    assert ais.mx_scale_bytes(10, 100) == 0                            # columns must be a multiple of 128
    p = ais.default_params()
    assert p.seq_level_weights == 0
    assert ais.workspace_bytes(ais.make_shape(1000, 4096, 151936, 8, 8, ais.FP8_MX32), p) > 0
    assert ais.workspace_bytes(ais.make_shape(1000, 4096, 151936, 8, 8, ais.FP4_MX32), p) > 0
    assert ais.workspace_bytes(ais.make_shape(1000, 4224, 151936, 8, 8, ais.FP4_MX32), p) == 0    # FP4 wants d % 256 == 0
    assert ais.workspace_bytes(ais.make_shape(1000, 4096, 151936, 8, 8, -7), p) == 0
    null = ctypes.c_void_p(None)
    one = ctypes.c_void_p(256)                                         # never dereferenced: the checks below fail first
    for fn in (lib.ais_quantize_mxfp8, lib.ais_quantize_mxfp4):
        assert fn(null, 4, 128, 128, one, 128, one, null) == -1       # AIS_ERR_NULL
        assert fn(one, 4, 100, 128, one, 128, one, null) == -2        # AIS_ERR_SHAPE: columns not a multiple of 128
        assert fn(one, 4, 256, 128, one, 256, one, null) == -2        # row stride shorter than the row


def test_head_layout_rules_are_checked_on_the_host():
    """ais_shape.w_layout: [d, V] heads need ldw >= V (a multiple of 8), take fp32 block scales only, and the column
    quantiser refuses shapes it cannot tile; an unknown layout value is an invalid shape."""
    import paper_2605_13907_b200 as ais
    p = ais.default_params()
    ok = ais.make_shape(1000, 4096, 151936, 8, 8, 128, w_layout=ais.W_DV)
    assert ok.ldw == 151936 and ais.workspace_bytes(ok, p) > 0
    assert ais.workspace_bytes(ais.make_shape(1000, 4096, 151936, 8, 8, 128, ldw=4096, w_layout=ais.W_DV), p) == 0    # ldw < V
    assert ais.workspace_bytes(ais.make_shape(1000, 4096, 151936, 8, 8, 128, ldw=151940, w_layout=ais.W_DV), p) == 0  # not a multiple of 8
    assert ais.workspace_bytes(ais.make_shape(1000, 4096, 151936, 8, 8, 0, w_layout=ais.W_DV), p) == 0                # per-tensor: [V, d] only
    assert ais.workspace_bytes(ais.make_shape(1000, 4096, 151936, 8, 8, ais.FP8_MX32, w_layout=ais.W_DV), p) == 0
    assert ais.workspace_bytes(ais.make_shape(1000, 4096, 151936, 8, 8, 128, w_layout=7), p) == 0
    lib = ais.lib()
    null = ctypes.c_void_p(None)
    one = ctypes.c_void_p(256)                                         # never dereferenced: the checks below fail first
    fn = lib.ais_quantize_fp8_cols
    assert fn(null, 128, 64, 64, 128, one, 128, one, 64, null) == -1  # AIS_ERR_NULL
    assert fn(one, 100, 64, 64, 128, one, 128, one, 64, null) == -2   # rows not a multiple of 128
    assert fn(one, 128, 64, 64, 48, one, 128, one, 64, null) == -2    # block size
    assert fn(one, 128, 64, 64, 128, one, 64, one, 64, null) == -2    # codes' row stride shorter than a column
    assert fn(one, 128, 64, 64, 128, one, 136, one, 64, null) == -3   # codes' row stride not a multiple of 16
