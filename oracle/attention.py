"""MXAttention forward on the CPU, written from the definitions of Algorithm 2 (test infrastructure only).

What is computed, per head and per query row (rows are independent; the query tile size never
enters the result):

  * Q-hat, K-hat: Q and K quantized in 32-blocks along the head dimension, optionally after the
    fixed Hadamard rotation; V-hat: V quantized in 32-blocks along the token axis (Algorithm 2,
    the quantization steps before the loop; Section 4.3).
  * The keys are visited in tiles of B_c = 128, in ascending order.  A tile contributes
      - its scores  S = Q-hat K-hat_tile^T * softmax_scale,
      - the new running maximum and the decay  alpha = exp(m_old - m_new)  of the state kept so far
        (the FlashAttention-2 recurrence of Section 2),
      - the un-normalized probabilities  P~ = exp(S - m_new), rounded ONCE to fp32 -- the precision
        in which the quantizer sees them --, and their quantized form  P-hat = Q(P~)  in 32-blocks
        along the key axis,
      - the row-sum increment: P-hat 1 under pre-normalization quantization (Eq. 22), P~ 1 under
        the direct placement (Eq. 12),
      - the accumulator increment  P-hat V-hat_tile.
  * O = accumulator / row sum.

The same scale rule (UOS, or the OCP floor rule) serves all four tensors Q, K, V and P~
(Section 4.3; the "MXFP4 (OCP)" baseline of Section 5.2).  float64 everywhere except the single
fp32 rounding of P~.

Readings: B_c is fixed to 128 and tiles are visited in ascending order (the result depends on
both, because P-hat depends on the history of the running maximum); key columns beyond Nkv are
excluded from the row maximum and contribute P~ = 0; the last V block along tokens is
zero-extended.
"""
from __future__ import annotations

import numpy as np

from . import mxfp4, nvfp4

B_C = 128


def _mxfp4_tile_quantizer(rule):
    """P~ [nq, B_C] -> Q(P~) with 32-blocks along the key axis under `rule`."""
    def quantize(p_tilde):
        nq = p_tilde.shape[0]
        codes, e = mxfp4.quantize_blocks(p_tilde.reshape(nq, B_C // mxfp4.BLOCK, mxfp4.BLOCK), rule)
        return mxfp4.dequantize_blocks(codes, e).reshape(nq, B_C)
    return quantize


def _nvfp4_tile_quantizer(p_tilde):
    """P~ [nq, B_C] -> NVFP4(P~) with 16-blocks along the key axis.  The tensor-level maximum of P~ is known
    without looking at the data: exp(S - m_new) <= 1, with equality in every row once a tile holds the row
    maximum; so the tensor scale is the constant 1 / 2688 (a reading: the paper does not say how its NVFP4
    baseline scales the softmax tile)."""
    nq = p_tilde.shape[0]
    codes, sc, s_t = nvfp4.quantize_blocks(p_tilde.reshape(nq, B_C // nvfp4.BLOCK, nvfp4.BLOCK), 1.0)
    return nvfp4.dequantize_blocks(codes, sc, np.broadcast_to(s_t, sc.shape)).reshape(nq, B_C)


def quantize_qkv(q, k, v, rule, rotate: bool = False, fmt: str = "mxfp4"):
    """Dequantized Q-hat, K-hat, V-hat (float64) of one head. q [Nq,d], k,v [Nkv,d].
    rotate: apply the fixed Hadamard rotation x -> x H_d / sqrt(d) to Q and K first (Algorithm 2,
    the rotation steps; the plain definition, `mxfp4.hadamard_rotate`).
    fmt "nvfp4": the comparison format of Section 5.2 instead of MXFP4 (16-blocks, E4M3 block scales, one
    tensor-level scale per matrix of the head; `rule` is not used)."""
    if rotate:
        q = mxfp4.hadamard_rotate(q)
        k = mxfp4.hadamard_rotate(k)
    if fmt == "nvfp4":
        return (nvfp4.quantize_dequantize(q, axis=1), nvfp4.quantize_dequantize(k, axis=1),
                nvfp4.quantize_dequantize(v, axis=0))
    qd = mxfp4.quantize_dequantize(q, axis=1, rule=rule)
    kd = mxfp4.quantize_dequantize(k, axis=1, rule=rule)
    vd = mxfp4.quantize_dequantize(v, axis=0, rule=rule)
    return qd, kd, vd


def tile_probabilities(s, m_new, width: int, quantizer):
    """Un-normalized probabilities of one key tile and their quantized form.

    s [nq, width] scores of the tile's valid keys, m_new [nq] the running maximum including this tile.
    Returns (p_tilde, p_hat), both [nq, B_C]: exp(s - m_new) rounded once to fp32, zero in the columns
    past `width`; and `quantizer` (a map [nq, B_C] -> [nq, B_C] that quantizes in blocks along the key axis;
    None: the identity) applied to it."""
    nq = s.shape[0]
    p_tilde = np.zeros((nq, B_C))
    with np.errstate(under="ignore"):
        p_tilde[:, :width] = np.exp(s - m_new[:, None]).astype(np.float32)
    if quantizer is None:
        return p_tilde, p_tilde
    return p_tilde, quantizer(p_tilde)


def row_sum_increment(p_tilde, p_hat, pnq: bool):
    """What a tile adds to the softmax denominator: the quantized probabilities under PNQ (Eq. 22), so
    that numerator and denominator see the same values; the unquantized ones under the direct placement
    (Eq. 12)."""
    return (p_hat if pnq else p_tilde).sum(axis=1)


def forward_head(q, k, v, softmax_scale: float, uos: bool = True, pnq: bool = True,
                 rows=None, quantize_inputs: bool = True, quantize_p: bool = True,
                 return_state: bool = False, rotate: bool = False, fmt: str = "mxfp4"):
    """Algorithm 2 for one head.

    fmt "nvfp4" runs the same loop with the NVFP4 quantizer in place of MXFP4 for all four tensors (the
    "NVFP4" baseline of Section 5.2; `uos` is then ignored, `pnq` still chooses where the row sum comes from).

    q [Nq,d], k [Nkv,d], v [Nkv,d]: float arrays holding bf16-representable values.
    rows: optional index array of query rows to compute (default all).
    quantize_inputs / quantize_p = False replace the respective quantizer by the identity
    (used only to pin the recurrence against dense attention).
    Returns O [len(rows), d] float64; with return_state also a dict with the per-tile
    quantities needed for the effective-row analysis of Appendix H (Lemma 2).
    """
    rule = mxfp4.UOS if uos else mxfp4.OCP
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    if quantize_inputs:
        qd, kd, vd = quantize_qkv(q, k, v, rule, rotate, fmt)
    else:
        qd, kd, vd = q, k, v
    if rows is not None:
        qd = qd[np.asarray(rows)]
    nq, d = qd.shape
    nkv = kd.shape[0]
    scale = float(np.float32(softmax_scale))          # the fp32 argument value, used as given

    # state of the online softmax: running maximum, denominator, un-normalized output
    m = np.full(nq, -np.inf)
    l = np.zeros(nq)
    o = np.zeros((nq, d))
    state = {"m": [], "p_hat": [], "p_tilde": []} if return_state else None
    tile_quantizer = None if not quantize_p else (_nvfp4_tile_quantizer if fmt == "nvfp4" else _mxfp4_tile_quantizer(rule))

    for start in range(0, nkv, B_C):
        stop = min(start + B_C, nkv)
        width = stop - start
        s = (qd @ kd[start:stop].T) * scale
        m_new = np.maximum(m, s.max(axis=1))
        alpha = np.exp(m - m_new)                     # decay of the state kept so far; exp(-inf) = 0 on the first tile
        p_tilde, p_hat = tile_probabilities(s, m_new, width, tile_quantizer)
        l = alpha * l + row_sum_increment(p_tilde, p_hat, pnq)
        o = alpha[:, None] * o + p_hat[:, :width] @ vd[start:stop]
        m = m_new
        if return_state:
            state["m"].append(m.copy())
            state["p_hat"].append(p_hat[:, :width].copy())
            state["p_tilde"].append(p_tilde[:, :width].copy())
    out = o / l[:, None]
    if return_state:
        state["l"] = l
        state["o_tilde"] = o
        state["vd"] = vd
        return out, state
    return out


def forward(q, k, v, softmax_scale: float, uos: bool = True, pnq: bool = True, rotate: bool = False, fmt: str = "mxfp4"):
    """All heads. q [B,H,Nq,d], k,v [B,H,Nkv,d] -> O [B,H,Nq,d] float64."""
    q = np.asarray(q)
    B, H = q.shape[:2]
    out = np.empty(q.shape, dtype=np.float64)
    for b in range(B):
        for h in range(H):
            out[b, h] = forward_head(q[b, h], k[b, h], v[b, h], softmax_scale, uos, pnq, rotate=rotate, fmt=fmt)
    return out


def dense_attention_head(q, k, v, softmax_scale: float, rows=None) -> np.ndarray:
    """Eq. 1 in float64: softmax(Q K^T * scale) V for one head, no quantization."""
    q = np.asarray(q, dtype=np.float64)
    if rows is not None:
        q = q[np.asarray(rows)]
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    s = (q @ k.T) * float(np.float32(softmax_scale))
    s -= s.max(axis=1, keepdims=True)
    p = np.exp(s)
    p /= p.sum(axis=1, keepdims=True)
    return p @ v


def _round_to_bf16(x: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 round-to-nearest-even, returned as float64 (finite inputs)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) & np.uint32(0xFFFF0000)
    return r.view(np.float32).astype(np.float64)


def forward_head_bf16(q, k, v, softmax_scale: float, rows=None):
    """The unquantized bf16 variant of the same recurrence (Section 2, Eq. 2-3; tiles of 128 keys):
    bf16 Q, K, V as given, the exponentials rounded to bf16 (RNE) for the P V product, the row sum
    taken from the fp32 exponentials."""
    q = np.asarray(q, dtype=np.float64)
    if rows is not None:
        q = q[np.asarray(rows)]
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    nq, d = q.shape
    scale = float(np.float32(softmax_scale))
    m = np.full(nq, -np.inf); l = np.zeros(nq); o = np.zeros((nq, d))
    for j0 in range(0, k.shape[0], B_C):
        s = (q @ k[j0:j0 + B_C].T) * scale
        m_new = np.maximum(m, s.max(axis=1))
        alpha = np.exp(m - m_new)
        with np.errstate(under="ignore"):
            p32 = np.exp(s - m_new[:, None]).astype(np.float32)
        l = alpha * l + p32.astype(np.float64).sum(axis=1)
        o = alpha[:, None] * o + _round_to_bf16(p32) @ v[j0:j0 + B_C]
        m = m_new
    return o / l[:, None]
