"""NVFP4 block quantization on the CPU (test infrastructure only).

NVFP4 is the comparison format of the paper: its Introduction describes it as E2M1 elements in blocks of 16
with an E4M3 scale per block plus one more scale per tensor, and the "NVFP4" baseline of Section 5.2 quantizes
Q, K, V and the softmax tile with it for the two attention GEMMs, without smoothing or extra softmax scaling.
The paper gives no more than that, so the
arithmetic below is a READING (listed in the design notes): the widely published two-level recipe,

    tensor level   g   = 2688 / A          A = largest magnitude of the tensor, 2688 = 448 * 6
                   s_T = 1 / g             (fp32 decode scale of the tensor)
    block level    d_b = E4M3( (M_b * g) / 6 )     M_b = largest magnitude of the 16-element block
    element        code = E2M1( x * (g / d_b) )    value(code) * d_b * s_T  approximates x

so that the largest element of the tensor maps to 6 * 448 in units of s_T and every block maximum lands near
the top of the E2M1 grid.  Because the results are integer codes, the precision and order of every step are
part of the reading; they are the ones a kernel can follow exactly, IEEE fp32 throughout:

    g   = fl32(2688 / A)                   (A = 0: g = 1)
    s_T = fl32(1 / g)
    y_b = fl32( fl32(M_b * g) * fl32(1/6) )
    d_b = y_b rounded to the nearest E4M3 value, ties to the even code, saturating at 448 (no infinities)
    r_b = fl32(g / d_b)                    (d_b = 0: r_b = 0, every code of the block is zero)
    code = sign | E2M1 index of fl32(|x| * r_b), round-to-nearest-even, saturating at 6

E4M3 here is the OCP 8-bit float with 4 exponent bits (bias 7) and 3 mantissa bits, subnormals, no
infinities, largest finite value 448 (code 0x7E); block scales are never negative.
"""
from __future__ import annotations

import numpy as np

from . import mxfp4

BLOCK = 16
E4M3_MAX = 448.0
F32 = np.float32
ONE_SIXTH = F32(1.0) / F32(6.0)                 # fl32(1/6)
TENSOR_RANGE = F32(2688.0)                      # 448 * 6


def e4m3_table() -> np.ndarray:
    """The 127 finite non-negative E4M3 values in code order (code = index): exponent field e (4 bits, bias 7),
    mantissa field m (3 bits); e = 0 is subnormal, m / 8 * 2^-6; otherwise (1 + m / 8) * 2^(e - 7).  Code 0x7F is NaN."""
    vals = []
    for code in range(127):
        e, m = code >> 3, code & 7
        vals.append(m / 8.0 * 2.0 ** -6 if e == 0 else (1.0 + m / 8.0) * 2.0 ** (e - 7))
    return np.array(vals, dtype=np.float64)


_E4M3 = e4m3_table()
_E4M3_MID = (_E4M3[:-1] + _E4M3[1:]) / 2.0      # exact in float64


def e4m3_round(y: np.ndarray) -> np.ndarray:
    """Code (0..126) of the E4M3 value nearest to y >= 0; a tie goes to the even code; everything above 448
    saturates to 448."""
    y = np.asarray(y, dtype=np.float64)
    code = np.searchsorted(_E4M3_MID, y, side="left")          # number of midpoints strictly below y
    tie = (code < 126) & (y == _E4M3_MID[np.minimum(code, 125)])
    # y sits exactly on the midpoint between code and code + 1: keep `code` if it is even, else move up
    code = np.where(tie & (code % 2 == 1), code + 1, code)
    return code.astype(np.uint8)


def e4m3_decode(code: np.ndarray) -> np.ndarray:
    return _E4M3[np.asarray(code, dtype=np.int64)]


def tensor_encode_scale(amax) -> np.float32:
    """g = fl32(2688 / A) for the tensor's largest magnitude A (fp32); 1 for an all-zero tensor."""
    a = F32(amax)
    return F32(1.0) if a == 0 else TENSOR_RANGE / a


def quantize_blocks(x: np.ndarray, amax):
    """x[..., 16] (finite) -> (codes uint8 [..., 16] with bit 3 = sign, e4m3 scale codes uint8 [...], s_T fp32).

    `amax`: the tensor-level maximum magnitude the blocks belong to (a scalar, or an array broadcastable to
    the block shape x.shape[:-1] when several tensors are quantized at once)."""
    x32 = np.asarray(x, dtype=F32)
    assert x32.shape[-1] == BLOCK
    amax = np.asarray(amax, dtype=F32)
    g = np.where(amax == 0, F32(1.0), TENSOR_RANGE / np.where(amax == 0, F32(1.0), amax)).astype(F32)
    s_t = (F32(1.0) / g).astype(F32)
    mag = np.abs(x32)
    m_b = mag.max(axis=-1)
    y = ((m_b * g).astype(F32) * ONE_SIXTH).astype(F32)
    sc = e4m3_round(y)
    d = e4m3_decode(sc).astype(F32)                                   # exact: E4M3 values are fp32 values
    with np.errstate(divide="ignore", invalid="ignore"):
        r = np.where(d == 0, F32(0.0), (np.broadcast_to(g, d.shape) / np.where(d == 0, F32(1.0), d))).astype(F32)
    idx = mxfp4.e2m1_index((mag * r[..., None]).astype(F32))
    sign = np.signbit(x32).astype(np.uint8)
    return (sign << 3) | idx, sc, s_t


def dequantize_blocks(codes: np.ndarray, sc: np.ndarray, s_t) -> np.ndarray:
    """value(code) * d_b * s_T in float64 (exact products of an E2M1 value, an E4M3 value and an fp32)."""
    val = mxfp4.E2M1_VALUES[codes & 7]
    val = np.where((codes & 8) != 0, -val, val)
    return val * e4m3_decode(sc)[..., None] * np.asarray(s_t, dtype=np.float64)[..., None]


def _blocked(x: np.ndarray, axis: int, pad_to: int):
    xm = np.moveaxis(np.asarray(x, dtype=np.float64), axis, -1)
    n = xm.shape[-1]
    npad = -n % pad_to
    if npad:
        xm = np.concatenate([xm, np.zeros(xm.shape[:-1] + (npad,))], axis=-1)
    return xm, n


def quantize_dequantize(x: np.ndarray, axis: int, amax=None) -> np.ndarray:
    """NVFP4(x) with 16-blocks along `axis` (zero-extended at the tail); same shape as x, float64.
    amax: the tensor-level maximum (default: the maximum magnitude of x itself)."""
    x = np.asarray(x, dtype=np.float64)
    if amax is None:
        amax = np.abs(x).max() if x.size else 0.0
    xm, n = _blocked(x, axis, BLOCK)
    blocks = xm.reshape(xm.shape[:-1] + (-1, BLOCK))
    codes, sc, s_t = quantize_blocks(blocks, F32(amax))
    deq = dequantize_blocks(codes, sc, np.broadcast_to(s_t, sc.shape)).reshape(xm.shape)[..., :n]
    return np.moveaxis(deq, -1, axis)


def quantize_matrix_canonical(x: np.ndarray, block_axis: int, amax=None):
    """[rows, cols] matrix -> the library's canonical NVFP4 byte layout and the tensor decode scale.

    block_axis = 1: codes [rows, cols/2] (element 2k in the low nibble of byte k), scales [rows, cols/16] E4M3 codes.
    block_axis = 0: TRANSPOSED, the block axis zero-extended to a multiple of 128: codes [cols, rows_pad/2],
        scales [cols, rows_pad/16] (a block of padding has code 0 and scale code 0).
    Returns (codes, scales, s_T fp32)."""
    x = np.asarray(x, dtype=np.float64)
    rows, cols = x.shape
    if amax is None:
        amax = np.abs(x).max()
    if block_axis == 1:
        assert cols % BLOCK == 0
        codes, sc, s_t = quantize_blocks(x.reshape(rows, cols // BLOCK, BLOCK), F32(amax))
        return mxfp4.pack_nibbles(codes.reshape(rows, cols)), sc, F32(s_t)
    if block_axis == 0:
        rows_pad = -(-rows // 128) * 128
        xt = np.zeros((cols, rows_pad)); xt[:, :rows] = x.T
        codes, sc, s_t = quantize_blocks(xt.reshape(cols, rows_pad // BLOCK, BLOCK), F32(amax))
        return mxfp4.pack_nibbles(codes.reshape(cols, rows_pad)), sc, F32(s_t)
    raise ValueError(block_axis)
