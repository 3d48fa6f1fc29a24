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


# ------------------------------------------------------------------------------------------------
# Canary words around device buffers.  Every buffer a kernel writes (outputs, workspaces) can be taken from
# `guarded()`: the usable region sits between two guard bands filled with a fixed byte, and `check()` verifies after
# the kernels have run that no guard byte changed -- an out-of-bounds write just before or after the buffer
# fails the test even where it would not change the compared output.
GUARD_BYTES = 4096          # a multiple of 256, so the guarded region keeps the allocation's alignment
GUARD_FILL = 0xC5


class Guarded:
    def __init__(self, shape, dtype, fill=None):
        n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        self.n = n
        self.pad = (-n) % 256
        self.raw = torch.full((GUARD_BYTES + n + self.pad + GUARD_BYTES,), GUARD_FILL, dtype=torch.uint8, device="cuda")
        self.t = self.raw[GUARD_BYTES:GUARD_BYTES + n].view(dtype).view(shape)
        if fill is not None:
            self.t.fill_(fill)

    def check(self):
        torch.cuda.synchronize()
        front = self.raw[:GUARD_BYTES]
        back = self.raw[GUARD_BYTES + self.n:]
        assert bool((front == GUARD_FILL).all()), "a kernel wrote in front of its buffer"
        assert bool((back == GUARD_FILL).all()), "a kernel wrote behind its buffer"


def guarded(shape, dtype, fill=None) -> Guarded:
    return Guarded(tuple(shape) if not isinstance(shape, int) else (shape,), dtype, fill)
