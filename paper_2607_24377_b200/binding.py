"""ctypes binding of the C ABI in include/mxattn.h: same names, argument marshalling only.

Tensors are torch CUDA tensors used purely as device-memory handles (``data_ptr()``); the stream
is torch's current stream.  Nothing here computes.
"""
from __future__ import annotations

import ctypes
import os

import torch

HERE = os.path.dirname(os.path.abspath(__file__))

MODE_OCP, MODE_UOS, MODE_HADAMARD = 0, 1, 0x100
FLAG_UOS, FLAG_PNQ, FLAG_OUT_FP32, FLAG_HADAMARD = 1, 2, 4, 8
LAYOUT_CANONICAL, LAYOUT_TILE = 0, 1

_lib = None


class MxAttnError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {strerror(code)} ({code})")


def lib_path() -> str:
    return os.path.join(HERE, "libmxattn.so")


def lib() -> ctypes.CDLL:
    """Load libmxattn.so (fails loudly if it has not been built: there is no fallback path)."""
    global _lib
    if _lib is None:
        path = lib_path()
        if not os.path.exists(path):
            raise ImportError(f"{path} is missing: run `python -m paper_2607_24377_b200.build` "
                              "(or __graft_entry__.build()); the CUDA library is the only implementation")
        L = ctypes.CDLL(path)
        vp, i64, ci, cf, cu, sz = (ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_float,
                                   ctypes.c_uint, ctypes.c_size_t)
        L.mxattn_quantize_mxfp4.argtypes = [vp, vp, vp, i64, i64, ci, ci, vp]
        L.mxattn_quantize_mxfp4_batched.argtypes = [vp, vp, vp, i64, i64, i64, ci, ci, ci, vp]
        L.mxattn_quantize_mxfp4_qmax.argtypes = [vp, vp, vp, i64, i64, i64, ci, cf, ci, vp]
        L.mxattn_tensor_amax.argtypes = [vp, vp, i64, i64, i64, vp]
        L.mxattn_quantize_nvfp4.argtypes = [vp, vp, vp, vp, vp, i64, i64, i64, ci, ci, vp]
        L.mxattn_forward_workspace_bytes.argtypes = [ci, ci, i64, i64, ci]
        L.mxattn_forward_workspace_bytes.restype = sz
        L.mxattn_set_workspace.argtypes = [vp, sz]
        L.mxattn_forward.argtypes = [vp, vp, vp, vp, ci, ci, i64, i64, ci, cf, cu, vp]
        L.mxattn_forward_static.argtypes = [vp, vp, vp, vp, ci, ci, i64, i64, ci, cf, cu, vp]
        L.mxattn_forward_ws.argtypes = [vp, vp, vp, vp, ci, ci, i64, i64, ci, cf, cu, vp, sz, vp]
        L.mxattn_rowsum_diagnostic.argtypes = [vp, vp, vp, ci, ci, i64, i64, ci, cf, cu, vp, sz, vp]
        L.mxattn_forward_debug_dump_bytes.argtypes = [ci, ci, i64, i64, ci]
        L.mxattn_forward_debug_dump_bytes.restype = sz
        L.mxattn_forward_debug_dump.argtypes = [vp, vp, vp, vp, ci, ci, i64, i64, ci, cf, cu, vp, sz, vp, sz, vp]
        L.mxattn_forward_cycle_profile_bytes.argtypes = [ci, ci, i64, i64, ci]
        L.mxattn_forward_cycle_profile_bytes.restype = sz
        L.mxattn_forward_cycle_profile.argtypes = [vp, vp, vp, vp, ci, ci, i64, i64, ci, cf, cu, vp, sz, vp, sz, vp]
        L.mxattn_forward_bf16_workspace_bytes.argtypes = [ci, ci, i64, i64, ci]
        L.mxattn_forward_bf16_workspace_bytes.restype = sz
        L.mxattn_forward_bf16.argtypes = [vp, vp, vp, vp, ci, ci, i64, i64, ci, cf, cu, vp, sz, vp]
        L.mxattn_forward_nvfp4_workspace_bytes.argtypes = [ci, ci, i64, i64, ci]
        L.mxattn_forward_nvfp4_workspace_bytes.restype = sz
        L.mxattn_forward_nvfp4.argtypes = [vp, vp, vp, vp, ci, ci, i64, i64, ci, cf, cu, vp, sz, vp]
        L.mxattn_forward_prequantized.argtypes = [vp] * 7 + [ci, ci, i64, i64, ci, cf, cu, vp, vp]
        L.mxattn_forward_host_arena_bytes.argtypes = [ci, ci, i64, i64, ci, cu]
        L.mxattn_forward_host_arena_bytes.restype = sz
        L.mxattn_forward_host.argtypes = [vp, vp, vp, vp, ci, ci, i64, i64, ci, cf, cu, vp, sz, vp]
        L.mxattn_probe_fp4_gemm.argtypes = [vp, vp, vp, vp, vp, i64, i64, i64, i64, ci, ci, ci, vp, vp]
        L.mxattn_quantizer_status.argtypes = [ctypes.POINTER(ctypes.c_int), vp]
        L.mxattn_device_status.argtypes = [vp, ctypes.POINTER(ctypes.c_int), vp]
        L.mxattn_selftest_bounded_wait.argtypes = [vp, i64, vp]
        L.mxattn_selftest_pair_abandon.argtypes = [vp, i64, ci, vp]
        L.mxattn_last_launch_count.argtypes = []
        L.mxattn_strerror.argtypes = [ci]
        L.mxattn_strerror.restype = ctypes.c_char_p
        _lib = L
    return _lib


def strerror(code: int) -> str:
    return lib().mxattn_strerror(int(code)).decode()


def _check(rc: int, where: str):
    if rc != 0:
        raise MxAttnError(rc, where)


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _ptr(t) -> int:
    return 0 if t is None else t.data_ptr()


def quantize_mxfp4(inp, codes, e8m0_scales, rows, cols, block_axis, mode):
    _check(lib().mxattn_quantize_mxfp4(_ptr(inp), _ptr(codes), _ptr(e8m0_scales), rows, cols,
                                       block_axis, mode, _stream()), "mxattn_quantize_mxfp4")


def quantize_mxfp4_batched(inp, codes, e8m0_scales, batch, rows, cols, block_axis, mode, layout):
    _check(lib().mxattn_quantize_mxfp4_batched(_ptr(inp), _ptr(codes), _ptr(e8m0_scales), batch, rows,
                                               cols, block_axis, mode, layout, _stream()),
           "mxattn_quantize_mxfp4_batched")


def quantize_mxfp4_qmax(inp, codes, e8m0_scales, batch, rows, cols, block_axis, qmax, layout):
    _check(lib().mxattn_quantize_mxfp4_qmax(_ptr(inp), _ptr(codes), _ptr(e8m0_scales), batch, rows, cols,
                                            block_axis, qmax, layout, _stream()), "mxattn_quantize_mxfp4_qmax")


def tensor_amax(inp, amax, batch, rows, cols):
    _check(lib().mxattn_tensor_amax(_ptr(inp), _ptr(amax), batch, rows, cols, _stream()), "mxattn_tensor_amax")


def quantize_nvfp4(inp, codes, e4m3_scales, tensor_amax, tensor_scale, batch, rows, cols, block_axis, layout):
    _check(lib().mxattn_quantize_nvfp4(_ptr(inp), _ptr(codes), _ptr(e4m3_scales), _ptr(tensor_amax), _ptr(tensor_scale),
                                       batch, rows, cols, block_axis, layout, _stream()), "mxattn_quantize_nvfp4")


def forward_workspace_bytes(B, H, Nq, Nkv, d) -> int:
    return int(lib().mxattn_forward_workspace_bytes(B, H, Nq, Nkv, d))


def set_workspace(ws, nbytes=None):
    _check(lib().mxattn_set_workspace(_ptr(ws), 0 if ws is None else (ws.numel() * ws.element_size()
                                                                       if nbytes is None else nbytes)),
           "mxattn_set_workspace")


def forward(q, k, v, o, B, H, Nq, Nkv, d, softmax_scale, flags):
    _check(lib().mxattn_forward(_ptr(q), _ptr(k), _ptr(v), _ptr(o), B, H, Nq, Nkv, d,
                                softmax_scale, flags, _stream()), "mxattn_forward")


STATIC_SCRATCH_BYTES = 32 << 20


def forward_static(q, k, v, o, B, H, Nq, Nkv, d, softmax_scale, flags):
    """mxattn_forward_static: the forward pass for callers that may not allocate device memory;
    its scratch is a fixed 32 MiB array inside the library (see include/mxattn.h for the rules)."""
    _check(lib().mxattn_forward_static(_ptr(q), _ptr(k), _ptr(v), _ptr(o), B, H, Nq, Nkv, d,
                                       softmax_scale, flags, _stream()), "mxattn_forward_static")


def forward_ws(q, k, v, o, B, H, Nq, Nkv, d, softmax_scale, flags, workspace):
    _check(lib().mxattn_forward_ws(_ptr(q), _ptr(k), _ptr(v), _ptr(o), B, H, Nq, Nkv, d, softmax_scale,
                                   flags, _ptr(workspace),
                                   0 if workspace is None else workspace.numel() * workspace.element_size(),
                                   _stream()), "mxattn_forward_ws")


def rowsum_diagnostic(q, k, out, B, H, Nq, Nkv, d, softmax_scale, flags, workspace):
    _check(lib().mxattn_rowsum_diagnostic(_ptr(q), _ptr(k), _ptr(out), B, H, Nq, Nkv, d, softmax_scale, flags,
                                          _ptr(workspace), 0 if workspace is None else workspace.numel() * workspace.element_size(),
                                          _stream()), "mxattn_rowsum_diagnostic")


def forward_debug_dump_bytes(B, H, Nq, Nkv, d) -> int:
    return int(lib().mxattn_forward_debug_dump_bytes(B, H, Nq, Nkv, d))


def forward_debug_dump(q, k, v, o, B, H, Nq, Nkv, d, softmax_scale, flags, workspace, dump):
    _check(lib().mxattn_forward_debug_dump(_ptr(q), _ptr(k), _ptr(v), _ptr(o), B, H, Nq, Nkv, d, softmax_scale, flags,
                                           _ptr(workspace), workspace.numel() * workspace.element_size(),
                                           _ptr(dump), 0 if dump is None else dump.numel() * dump.element_size(), _stream()),
           "mxattn_forward_debug_dump")


def forward_cycle_profile_bytes(B, H, Nq, Nkv, d) -> int:
    return int(lib().mxattn_forward_cycle_profile_bytes(B, H, Nq, Nkv, d))


def forward_cycle_profile(q, k, v, o, B, H, Nq, Nkv, d, softmax_scale, flags, workspace, profile):
    _check(lib().mxattn_forward_cycle_profile(_ptr(q), _ptr(k), _ptr(v), _ptr(o), B, H, Nq, Nkv, d, softmax_scale, flags,
                                              _ptr(workspace), workspace.numel() * workspace.element_size(),
                                              _ptr(profile), 0 if profile is None else profile.numel() * profile.element_size(), _stream()),
           "mxattn_forward_cycle_profile")


def forward_bf16_workspace_bytes(B, H, Nq, Nkv, d) -> int:
    return int(lib().mxattn_forward_bf16_workspace_bytes(B, H, Nq, Nkv, d))


def forward_bf16(q, k, v, o, B, H, Nq, Nkv, d, softmax_scale, flags, workspace):
    _check(lib().mxattn_forward_bf16(_ptr(q), _ptr(k), _ptr(v), _ptr(o), B, H, Nq, Nkv, d, softmax_scale, flags,
                                     _ptr(workspace), workspace.numel() * workspace.element_size(), _stream()),
           "mxattn_forward_bf16")


def forward_nvfp4_workspace_bytes(B, H, Nq, Nkv, d) -> int:
    return int(lib().mxattn_forward_nvfp4_workspace_bytes(B, H, Nq, Nkv, d))


def forward_nvfp4(q, k, v, o, B, H, Nq, Nkv, d, softmax_scale, flags, workspace):
    _check(lib().mxattn_forward_nvfp4(_ptr(q), _ptr(k), _ptr(v), _ptr(o), B, H, Nq, Nkv, d, softmax_scale, flags,
                                      _ptr(workspace), 0 if workspace is None else workspace.numel() * workspace.element_size(),
                                      _stream()), "mxattn_forward_nvfp4")


def forward_prequantized(q_codes, q_scales, k_codes, k_scales, v_codes, v_scales, o,
                         B, H, Nq, Nkv, d, softmax_scale, flags, status):
    _check(lib().mxattn_forward_prequantized(_ptr(q_codes), _ptr(q_scales), _ptr(k_codes), _ptr(k_scales),
                                             _ptr(v_codes), _ptr(v_scales), _ptr(o), B, H, Nq, Nkv, d,
                                             softmax_scale, flags, _ptr(status), _stream()),
           "mxattn_forward_prequantized")


def forward_host_arena_bytes(B, H, Nq, Nkv, d, flags) -> int:
    return int(lib().mxattn_forward_host_arena_bytes(B, H, Nq, Nkv, d, flags))


def forward_host(q_host, k_host, v_host, o_host, B, H, Nq, Nkv, d, softmax_scale, flags, arena):
    """q_host.. are CPU tensors (pinned recommended); arena is a CUDA byte tensor."""
    _check(lib().mxattn_forward_host(q_host.data_ptr(), k_host.data_ptr(), v_host.data_ptr(),
                                     o_host.data_ptr(), B, H, Nq, Nkv, d, softmax_scale, flags,
                                     _ptr(arena), arena.numel() * arena.element_size(), _stream()),
           "mxattn_forward_host")


def probe_fp4_gemm(a_codes, a_scales, b_codes, b_scales, c, M, N, K, k_steps, resident, out_fp32, status, tile_n=256):
    _check(lib().mxattn_probe_fp4_gemm(_ptr(a_codes), _ptr(a_scales), _ptr(b_codes), _ptr(b_scales), _ptr(c), M, N, K,
                                       k_steps, int(resident), int(out_fp32), int(tile_n), _ptr(status), _stream()),
           "mxattn_probe_fp4_gemm")


def quantizer_status() -> int:
    out = ctypes.c_int(0)
    _check(lib().mxattn_quantizer_status(ctypes.byref(out), _stream()), "mxattn_quantizer_status")
    return out.value


def device_status(workspace) -> int:
    out = ctypes.c_int(0)
    _check(lib().mxattn_device_status(_ptr(workspace), ctypes.byref(out), _stream()), "mxattn_device_status")
    return out.value


def selftest_bounded_wait(status, limit_cycles: int):
    _check(lib().mxattn_selftest_bounded_wait(_ptr(status), int(limit_cycles), _stream()), "mxattn_selftest_bounded_wait")


def selftest_pair_abandon(status, limit_cycles: int, meetings: int):
    _check(lib().mxattn_selftest_pair_abandon(_ptr(status), int(limit_cycles), int(meetings), _stream()),
           "mxattn_selftest_pair_abandon")


def last_launch_count() -> int:
    return int(lib().mxattn_last_launch_count())
