"""The C-ABI library builds, loads, and exports every symbol the header declares (no GPU needed)."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "mxattn.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(mxattn_[a-z0-9_]+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    from paper_2607_24377_b200 import build
    path = build.build()
    L = ctypes.CDLL(path)
    syms = declared_symbols()
    assert "mxattn_quantize_mxfp4" in syms and "mxattn_forward" in syms and len(syms) >= 10
    for s in syms:
        assert hasattr(L, s), s


def test_argument_errors_need_no_device():
    import paper_2607_24377_b200 as mx
    L = mx.lib()
    # null pointers / bad sizes / bad enums are rejected before any CUDA call
    assert L.mxattn_quantize_mxfp4(None, None, None, 4, 32, 1, 1, None) == -1
    assert L.mxattn_quantize_mxfp4(16, 16, 16, 0, 32, 1, 1, None) == -1
    assert L.mxattn_quantize_mxfp4(16, 16, 16, 4, 32, 2, 1, None) == -1
    assert L.mxattn_quantize_mxfp4(16, 16, 16, 4, 32, 1, 7, None) == -1
    assert L.mxattn_quantize_mxfp4(16, 16, 16, 4, 48, 1, 1, None) == -2          # cols % 32
    assert L.mxattn_quantize_mxfp4(24, 16, 16, 4, 32, 1, 1, None) == -3          # misaligned
    assert L.mxattn_quantize_mxfp4_batched(16, 16, 16, 1, 4, 64, 1, 1, 1, None) == -2   # tile layout needs cols 128
    assert mx.forward_workspace_bytes(1, 2, 1024, 1024, 64) == 0
    assert mx.forward_workspace_bytes(1, 2, 1024, 1024, 128) > 3 * 2 * 8 * 8704
    assert L.mxattn_forward(16, 16, 16, 16, 1, 2, 128, 128, 64, 0.1, 3, None) == -2
    assert L.mxattn_forward(16, 16, 16, 16, 1, 2, 128, 128, 128, 0.1, 64, None) == -1     # unknown flag
    assert L.mxattn_forward(16, 16, 16, 16, 1, 2, 128, 128, 128, -1.0, 3, None) == -1
    mx.set_workspace(None)
    assert L.mxattn_forward(16, 16, 16, 16, 1, 2, 128, 128, 128, 0.1, 3, None) == -4      # no workspace
    assert mx.strerror(-6).startswith("device-side")


def test_argument_errors_of_the_diagnostic_entry_points():
    import paper_2607_24377_b200 as mx
    L = mx.lib()
    big = 1 << 40
    # row-sum diagnostic: flags other than UOS / HADAMARD, head dimension, alignment, workspace
    assert L.mxattn_rowsum_diagnostic(16, 16, 16, 1, 1, 128, 128, 128, 0.1, 2, 16, big, None) == -1     # PNQ is no flag of it
    assert L.mxattn_rowsum_diagnostic(None, 16, 16, 1, 1, 128, 128, 128, 0.1, 1, 16, big, None) == -1
    assert L.mxattn_rowsum_diagnostic(16, 16, 16, 1, 1, 128, 128, 64, 0.1, 1, 16, big, None) == -2
    assert L.mxattn_rowsum_diagnostic(16, 24, 16, 1, 1, 128, 128, 128, 0.1, 1, 16, big, None) == -3
    assert L.mxattn_rowsum_diagnostic(16, 16, 16, 1, 1, 128, 128, 128, 0.1, 1, 16, 1024, None) == -4
    assert L.mxattn_rowsum_diagnostic(16, 16, 16, 1, 1, 128, 128, 128, 0.0, 1, 16, big, None) == -1
    # debug dump: needs the dump buffer, the fp32 output flag, a buffer of the stated size, a small problem
    assert mx.forward_debug_dump_bytes(1, 2, 1024, 1024, 128) == 2 * 8 * 8 * 9216 + 2 * 8 * 128 * 4
    assert mx.forward_debug_dump_bytes(1, 2, 1024, 1024, 64) == 0
    assert L.mxattn_forward_debug_dump(16, 16, 16, 16, 1, 2, 1024, 1024, 128, 0.1, 7, 16, big, None, big, None) == -1
    assert L.mxattn_forward_debug_dump(16, 16, 16, 16, 1, 2, 1024, 1024, 128, 0.1, 3, 16, big, 16, big, None) == -1   # bf16 output
    assert L.mxattn_forward_debug_dump(16, 16, 16, 16, 1, 2, 1024, 1024, 128, 0.1, 7, 16, big, 16, 1024, None) == -4
    assert L.mxattn_forward_debug_dump(16, 16, 16, 16, 1, 40, 75600, 75600, 128, 0.1, 7, 16, big, 16, big, None) == -2
