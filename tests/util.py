"""Helpers shared by the GPU parity tests (host-side marshalling only)."""
import numpy as np
import torch

import synth_inputs as si


def to_dev_bf16(bits: np.ndarray) -> torch.Tensor:
    """uint16 bf16 bit patterns -> CUDA bf16 tensor (bit-identical)."""
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def bits_to_f64(bits: np.ndarray) -> np.ndarray:
    return si.bf16_bits_to_f32(bits).astype(np.float64)


def tile_code_offset(r, c):
    return r * 64 + ((c ^ ((r >> 1) & 3)) << 4)


def tile_scale_offset(r, c):
    return (r & 31) * 16 + (r >> 5) * 4 + c


def canonical_to_tile_axis1(codes: np.ndarray, scales: np.ndarray):
    """[rows,64] codes / [rows,4] scales of ONE matrix -> tile images (rows padded with zero codes, scale 127)."""
    rows = codes.shape[0]
    nt = -(-rows // 128)
    cp = np.zeros((nt * 128, 64), np.uint8); cp[:rows] = codes
    sp = np.full((nt * 128, 4), 127, np.uint8); sp[:rows] = scales
    tc = np.zeros((nt, 8192), np.uint8); ts = np.zeros((nt, 512), np.uint8)
    r = np.arange(128)
    for t in range(nt):
        for c in range(4):
            off = tile_code_offset(r, c)
            for b in range(16):
                tc[t, off + b] = cp[t * 128 + r, c * 16 + b]
            ts[t, tile_scale_offset(r, c)] = sp[t * 128 + r, c]
    return tc, ts


def canonical_to_tile_axis0(codes: np.ndarray, scales: np.ndarray):
    """[128, rows_pad/2] codes / [128, rows_pad/32] scales (transposed canonical) -> tile images."""
    nt = codes.shape[1] // 64
    tc = np.zeros((nt, 8192), np.uint8); ts = np.zeros((nt, 512), np.uint8)
    n = np.arange(128)
    for t in range(nt):
        for c in range(4):
            off = tile_code_offset(n, c)
            for b in range(16):
                tc[t, off + b] = codes[n, t * 64 + c * 16 + b]
            ts[t, tile_scale_offset(n, c)] = scales[n, t * 4 + c]
    return tc, ts
