"""Row-sum diagnostic for MXFP4 quantization of attention probabilities (test infrastructure only).

Section 5.3 "Validation of Pre-Normalization Quantization" (Figure "Row-sum diagnostics", panels
A, B, D): the attention probabilities of a row are materialized, P = softmax(S), block-quantized
with 32-blocks along the key axis, and the row sum of the quantized values is compared with one.
The error P-hat 1 - 1 is split by quantization outcome:

    zeroing      elements with p > 0 that quantize to 0                      (contribution -p)
    saturation   elements whose scaled value p / sigma exceeds the top grid value 6   (p-hat - p < 0)
    downward     all other elements with p-hat < p
    upward       elements with p-hat > p

and the row's entropy -sum p ln p is the abscissa of panel D.

Readings (the paper gives no formulas for this diagnostic):
  * S = Q-hat K-hat^T * softmax_scale with Q, K quantized as in the forward pass (the scores the
    attention loop sees); the rule (OCP or UOS) is the same for Q, K and P;
  * P is rounded once to fp32 before it is quantized (the precision the quantizer sees, as for P-tilde);
  * blocks are aligned to key index multiples of 32, the last one zero-extended;
  * the reference sum is the sum of the fp32 probabilities (1 up to rounding), so the four
    contributions add up to  P-hat 1 - P 1  exactly.
"""
from __future__ import annotations

import numpy as np

from . import mxfp4
from .attention import quantize_qkv

COLUMNS = ("rowsum", "zeroing", "saturation", "downward", "upward", "entropy")


def decompose_rows(p: np.ndarray, rule: mxfp4.ScaleRule) -> np.ndarray:
    """p [rows, n]: non-negative fp32-representable probabilities.  Returns [rows, 6] float64 (COLUMNS)."""
    p = np.asarray(p, dtype=np.float64)
    rows, n = p.shape
    npad = -n % mxfp4.BLOCK
    pp = np.concatenate([p, np.zeros((rows, npad))], axis=1) if npad else p
    blocks = pp.reshape(rows, -1, mxfp4.BLOCK)
    codes, e = mxfp4.quantize_blocks(blocks, rule)
    p_hat = mxfp4.dequantize_blocks(codes, e)
    scaled = np.ldexp(blocks, -e[..., None])                  # p / sigma, exact
    diff = p_hat - blocks
    zero = (p_hat == 0) & (blocks > 0)
    sat = scaled > 6.0                                         # beyond the largest grid value (Section 2)
    down = (diff < 0) & ~zero & ~sat
    up = diff > 0
    out = np.empty((rows, 6))
    out[:, 0] = p_hat.sum(axis=(1, 2))
    out[:, 1] = np.where(zero, diff, 0.0).sum(axis=(1, 2))
    out[:, 2] = np.where(sat, diff, 0.0).sum(axis=(1, 2))
    out[:, 3] = np.where(down, diff, 0.0).sum(axis=(1, 2))
    out[:, 4] = np.where(up, diff, 0.0).sum(axis=(1, 2))
    with np.errstate(divide="ignore", invalid="ignore"):
        out[:, 5] = -np.where(p > 0, p * np.log(p), 0.0).sum(axis=1)
    return out


def softmax_rows_f32(s: np.ndarray) -> np.ndarray:
    """Row softmax in float64, rounded once to fp32 (returned as float64 values)."""
    s = np.asarray(s, dtype=np.float64)
    x = s - s.max(axis=1, keepdims=True)
    with np.errstate(under="ignore"):
        ex = np.exp(x)
    return (ex / ex.sum(axis=1, keepdims=True)).astype(np.float32).astype(np.float64)


def diagnostic_head(q, k, softmax_scale: float, uos: bool = True, rows=None, rotate: bool = False) -> np.ndarray:
    """The diagnostic for one head: q [Nq, d], k [Nkv, d] bf16-representable floats -> [len(rows), 6]."""
    rule = mxfp4.UOS if uos else mxfp4.OCP
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    qd, kd, _ = quantize_qkv(q, k, np.zeros((k.shape[0], q.shape[1])), rule, rotate)
    if rows is not None:
        qd = qd[np.asarray(rows)]
    s = (qd @ kd.T) * float(np.float32(softmax_scale))
    return decompose_rows(softmax_rows_f32(s), rule)
