"""MXFP4 block quantization, written out from the paper's definitions (test infrastructure only).

Section 2 "MXFP4 Block Quantization": a block is 32 elements sharing a power-of-two scale
sigma = 2^e stored as E8M0 (byte e + 127); elements are projected by round-to-nearest onto the
E2M1 grid {0, .5, 1, 1.5, 2, 3, 4, 6} (with sign), saturating at 6.

Scale rules (Eq. 5 "OCP", Eq. 6-7 the floor / ceiling families, Eq. 13 + Algorithm 1 "UOS"):

    OCP   e = floor(log2 M) - 2                  (= e_floor(8), normalized max in [4, 8))
    ceil  e = ceil(log2(M / Qmax))               (normalized max in (Qmax/2, Qmax])
    UOS   the ceiling rule with Qmax = 29/4 = 7.25
    TFS   the ceiling rule with Qmax = 6;  OAS at block 32 = the ceiling rule with Qmax = 7 (Appendix G)

log2 is never evaluated in floating point: floor/ceil are decided exactly from the binary
exponent and mantissa of M (``numpy.frexp`` is exact).

Readings taken where the paper is silent (each is listed in the design notes):
  * round-to-nearest breaks ties to the even E2M1 code (IEEE RNE, what the OCP MX spec and
    Blackwell's conversion instruction do): .25->0, .75->1, 1.25->1, 1.75->2, 2.5->2, 3.5->4, 5->4;
  * the sign bit of the input is always kept (a negative value that rounds to zero gives code 0x8);
  * e is clamped to the E8M0 range [-127, 127] and rounding proceeds with the clamped scale;
  * all-zero block: sigma = 1 (byte 127), all codes 0 (Section 2, last paragraph; Algorithm 1).
"""
from __future__ import annotations

import dataclasses

import numpy as np

BLOCK = 32

# Section 2, Eq. 3 (non-negative half); index = low 3 bits of the 4-bit code, bit 3 = sign.
E2M1_VALUES = np.array([0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0], dtype=np.float64)
# Appendix B: round-to-nearest decision boundaries between neighbouring grid values.
E2M1_THRESHOLDS = np.array([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0], dtype=np.float64)


@dataclasses.dataclass(frozen=True)
class ScaleRule:
    """family 'floor' -> e = floor(log2(M/q)) + 1;  family 'ceil' -> e = ceil(log2(M/q))  (Eq. 6-7)."""
    family: str
    q: float


OCP = ScaleRule("floor", 8.0)    # Eq. 5: floor(log2 M) - 2 == floor(log2(M/8)) + 1 (Appendix G, Eq. 57)
UOS = ScaleRule("ceil", 7.25)    # Eq. 13 with q* = 29/4 (Theorem 1); the exponent step of Algorithm 1
TFS = ScaleRule("ceil", 6.0)     # Eq. 8
OAS = ScaleRule("ceil", 7.0)     # Appendix G


def e2m1_index(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even projection of non-negative x onto the E2M1 grid; returns index 0..7.

    Everything above 5 maps to index 7 (value 6): saturation (Section 2, below Eq. 4).
    A tie at a threshold goes to the neighbour with the even index.
    """
    x = np.asarray(x, dtype=np.float64)
    idx = np.zeros(x.shape, dtype=np.uint8)
    for i, t in enumerate(E2M1_THRESHOLDS):
        lower_is_even = (i % 2 == 0)      # threshold i separates index i and i+1
        # tie stays at the lower index when that one is even, else moves up
        idx += ((x > t) if lower_is_even else (x >= t)).astype(np.uint8)
    return idx


def shared_exponent(M: np.ndarray, rule: ScaleRule) -> np.ndarray:
    """Exact integer e for block maxima M >= 0 (M == 0 -> e = 0), clamped to [-127, 127]."""
    M = np.asarray(M, dtype=np.float64)
    f, p = np.frexp(M)                      # M = f * 2^p, f in [0.5, 1), exact
    fq, pq = np.frexp(np.float64(rule.q))   # q = fq * 2^pq
    # M / q = (f / fq) * 2^(p - pq) with f / fq in (0.5, 2)
    if rule.family == "ceil":
        # smallest e with M <= q * 2^e
        e = (p - pq) + (f > fq)
    elif rule.family == "floor":
        # floor(log2(M/q)) + 1 : largest k with 2^k <= M/q, plus one
        e = (p - pq) + (f >= fq)
    else:
        raise ValueError(rule.family)
    e = np.where(M == 0.0, 0, e)
    return np.clip(e, -127, 127).astype(np.int32)


def quantize_blocks(x: np.ndarray, rule: ScaleRule):
    """Block quantization (Section 2; Algorithm 1 for the UOS rule) of an array of blocks x[..., 32]
    (any float dtype, finite values): the block maximum fixes the shared exponent by `rule` (an all-zero
    block gets sigma = 1), every element is divided by sigma = 2^e -- exactly -- and projected onto the
    E2M1 grid; the sign is carried separately.

    Returns (codes uint8 [..., 32] with bit 3 = sign and bits 0-2 = grid index, e int32 [...]).
    """
    x64 = np.asarray(x, dtype=np.float64)
    assert x64.shape[-1] == BLOCK
    mag = np.abs(x64)
    e = shared_exponent(mag.max(axis=-1), rule)
    idx = e2m1_index(np.ldexp(mag, -e[..., None]))
    sign = np.signbit(x64).astype(np.uint8)
    return (sign << 3) | idx, e


def dequantize_blocks(codes: np.ndarray, e: np.ndarray) -> np.ndarray:
    """sigma * grid value with sign, float64, exact (Eq. 4)."""
    val = E2M1_VALUES[codes & 7]
    val = np.where((codes & 8) != 0, -val, val)
    return np.ldexp(val, np.asarray(e)[..., None])


def quantize_dequantize(x: np.ndarray, axis: int, rule: ScaleRule) -> np.ndarray:
    """Q(x) with blocks of 32 along `axis` (zero-extended at the tail); same shape as x, float64."""
    x = np.asarray(x, dtype=np.float64)
    xm = np.moveaxis(x, axis, -1)
    n = xm.shape[-1]
    npad = -n % BLOCK
    if npad:
        xm = np.concatenate([xm, np.zeros(xm.shape[:-1] + (npad,))], axis=-1)
    blocks = xm.reshape(xm.shape[:-1] + (-1, BLOCK))
    codes, e = quantize_blocks(blocks, rule)
    deq = dequantize_blocks(codes, e).reshape(xm.shape)[..., :n]
    return np.moveaxis(deq, -1, axis)


# ----------------------------------------------------------------------------- canonical packing
def pack_nibbles(codes: np.ndarray) -> np.ndarray:
    """[..., 2k] -> low nibble, [..., 2k+1] -> high nibble of byte k."""
    c = np.asarray(codes, dtype=np.uint8)
    return (c[..., 0::2] | (c[..., 1::2] << 4)).astype(np.uint8)


def e8m0_bytes(e: np.ndarray) -> np.ndarray:
    return (np.asarray(e, dtype=np.int32) + 127).astype(np.uint8)


def quantize_matrix_canonical(x: np.ndarray, block_axis: int, rule: ScaleRule):
    """Quantize a [rows, cols] matrix and emit the library's canonical byte layout.

    block_axis = 1 (Q, K: blocks along cols): codes [rows, cols/2], scales [rows, cols/32].
    block_axis = 0 (V: blocks along rows): outputs are TRANSPOSED, contiguous along the block
        axis, which is zero-extended to a multiple of 128: codes [cols, rows_pad/2],
        scales [cols, rows_pad/32] (a block of padding has code 0 and scale byte 127).
    """
    x = np.asarray(x, dtype=np.float64)
    rows, cols = x.shape
    if block_axis == 1:
        assert cols % BLOCK == 0
        codes, e = quantize_blocks(x.reshape(rows, cols // BLOCK, BLOCK), rule)
        return pack_nibbles(codes.reshape(rows, cols)), e8m0_bytes(e)
    if block_axis == 0:
        rows_pad = -(-rows // 128) * 128
        xt = np.zeros((cols, rows_pad), dtype=np.float64)
        xt[:, :rows] = x.T
        codes, e = quantize_blocks(xt.reshape(cols, rows_pad // BLOCK, BLOCK), rule)
        return pack_nibbles(codes.reshape(cols, rows_pad)), e8m0_bytes(e)
    raise ValueError(block_axis)


# ----------------------------------------------------------------------------- Hadamard rotation
def hadamard_matrix(n: int) -> np.ndarray:
    """Sylvester Hadamard matrix H_n (n a power of two): H[i, j] = (-1)^popcount(i & j), entries +-1."""
    i = np.arange(n)
    bits = i[:, None] & i[None, :]
    pop = np.zeros_like(bits)
    while bits.any():
        pop += bits & 1
        bits >>= 1
    return np.where(pop % 2 == 0, 1.0, -1.0)


def hadamard_rotate(x: np.ndarray) -> np.ndarray:
    """x R_H along the last axis with R_H = H_n / sqrt(n): the fixed orthogonal Hadamard rotation of
    Algorithm 2 lines 1-2 (Section 4.3), written as its definition.

    The matrix product runs in float64.  For bf16 inputs every entry of x H_n is a sum of 128 numbers with
    8-bit significands, which float64 holds exactly (unless the exponents in one row span more than about
    2^37), so the only roundings are the float64 division by sqrt(n) and ONE rounding to fp32 at the end --
    fp32 being the precision in which the quantizer sees the rotated values.  Returns fp32."""
    x64 = np.asarray(x, dtype=np.float64)
    n = x64.shape[-1]
    return ((x64 @ hadamard_matrix(n)) / np.sqrt(np.float64(n))).astype(np.float32)
