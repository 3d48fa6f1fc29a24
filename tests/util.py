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


E2M1_VALUES = np.array([0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0])


def decode_tile_axis1(tile_codes: np.ndarray, tile_scales: np.ndarray) -> np.ndarray:
    """One 8192-byte tile image + its 512-byte scale atom -> the [128, 128] float64 values it encodes
    (rows x 128 elements, blocks of 32 along the row).  Pure byte shuffling plus the E2M1 / E8M0 tables."""
    r = np.arange(128)
    out = np.zeros((128, 128))
    for c in range(4):
        off = tile_code_offset(r, c)
        byts = np.stack([tile_codes[off + b] for b in range(16)], axis=1)        # [128, 16]
        nib = np.empty((128, 32), np.uint8)
        nib[:, 0::2] = byts & 15
        nib[:, 1::2] = byts >> 4
        val = E2M1_VALUES[nib & 7] * np.where(nib & 8, -1.0, 1.0)
        e = tile_scales[tile_scale_offset(r, c)].astype(np.int32) - 127
        out[:, 32 * c:32 * c + 32] = np.ldexp(val, e[:, None])
    return out
