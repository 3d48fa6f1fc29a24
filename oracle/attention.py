"""MXAttention forward, step by step as Algorithm 2 states it (test infrastructure only).

Per head and per query row (rows are independent; the query tile size never enters):

    Q-hat, K-hat = Q(.) with 32-blocks along the head dimension        (Alg. 2 lines 3-4)
    V-hat        = Q(.) with 32-blocks along the token axis            (Alg. 2 line 5)
    for each KV tile j of B_c = 128 keys, ascending:                   (line 8)
        S      = Q-hat K-hat_j^T * softmax_scale                       (line 9)
        m_new  = max(m, rowmax S)                                      (line 10)
        alpha  = exp(m - m_new)                                        (line 11)
        P~     = exp(S - m_new)            rounded once to fp32        (line 12)
        P-hat  = Q(P~) with 32-blocks along the key axis               (line 13)
        l      = alpha l + P-hat 1   (PNQ, Eq. 22)  |  alpha l + P~ 1  (direct, Eq. 12)   (line 14)
        O~     = alpha O~ + P-hat V-hat_j                              (line 15)
        m      = m_new                                                 (line 16)
    O = O~ / l                                                         (line 18)

The Hadamard rotation of lines 1-2 is optional (`rotate`).  The same scale rule (UOS or the
OCP floor rule) is used for all four tensors Q, K, V and P~ (Section 4.3; the "MXFP4 (OCP)"
baseline of Section 5.2).  float64 everywhere except the single fp32 rounding of P~, which is
the precision in which the quantizer sees the exponentials.

Readings: B_c is fixed to 128 and tiles are visited in ascending order (the result depends on
both, because P-hat depends on the running-max history); key columns beyond Nkv are excluded
from the row max and contribute P~ = 0; the last V block along tokens is zero-extended.
"""
from __future__ import annotations

import numpy as np

from . import mxfp4

B_C = 128


def quantize_qkv(q, k, v, rule, rotate: bool = False):
    """Dequantized Q-hat, K-hat, V-hat (float64) of one head. q [Nq,d], k,v [Nkv,d].
    rotate: apply the fixed Hadamard rotation to Q and K first (Algorithm 2 lines 1-2)."""
    if rotate:
        q = mxfp4.hadamard_rotate_f32(q)
        k = mxfp4.hadamard_rotate_f32(k)
    qd = mxfp4.quantize_dequantize(q, axis=1, rule=rule)
    kd = mxfp4.quantize_dequantize(k, axis=1, rule=rule)
    vd = mxfp4.quantize_dequantize(v, axis=0, rule=rule)
    return qd, kd, vd


def forward_head(q, k, v, softmax_scale: float, uos: bool = True, pnq: bool = True,
                 rows=None, quantize_inputs: bool = True, quantize_p: bool = True,
                 return_state: bool = False, rotate: bool = False):
    """Algorithm 2 for one head.

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
        qd, kd, vd = quantize_qkv(q, k, v, rule, rotate)
    else:
        qd, kd, vd = q, k, v
    if rows is not None:
        qd = qd[np.asarray(rows)]
    nq, d = qd.shape
    nkv = kd.shape[0]
    scale = float(np.float32(softmax_scale))          # the fp32 argument value, used as given

    m = np.full(nq, -np.inf)
    l = np.zeros(nq)
    o = np.zeros((nq, d))
    state = {"m": [], "p_hat": [], "p_tilde": []} if return_state else None

    for j0 in range(0, nkv, B_C):
        j1 = min(j0 + B_C, nkv)
        w = j1 - j0
        s = (qd @ kd[j0:j1].T) * scale                                    # line 9
        m_new = np.maximum(m, s.max(axis=1))                              # line 10
        alpha = np.exp(m - m_new)                                         # line 11 (exp(-inf) = 0)
        p_tilde = np.zeros((nq, B_C))
        with np.errstate(under="ignore"):
            p_tilde[:, :w] = np.exp(s - m_new[:, None]).astype(np.float32)    # line 12, fp32 once
        if quantize_p:
            codes, e = mxfp4.quantize_blocks(p_tilde.reshape(nq, B_C // 32, 32), rule)   # line 13
            p_hat = mxfp4.dequantize_blocks(codes, e).reshape(nq, B_C)
        else:
            p_hat = p_tilde
        l = alpha * l + (p_hat.sum(axis=1) if pnq else p_tilde.sum(axis=1))   # line 14
        o = alpha[:, None] * o + p_hat[:, :w] @ vd[j0:j1]                      # line 15
        m = m_new                                                             # line 16
        if return_state:
            state["m"].append(m.copy())
            state["p_hat"].append(p_hat[:, :w].copy())
            state["p_tilde"].append(p_tilde[:, :w].copy())
    out = o / l[:, None]                                                  # line 18
    if return_state:
        state["l"] = l
        state["o_tilde"] = o
        state["vd"] = vd
        return out, state
    return out


def forward(q, k, v, softmax_scale: float, uos: bool = True, pnq: bool = True, rotate: bool = False):
    """All heads. q [B,H,Nq,d], k,v [B,H,Nkv,d] -> O [B,H,Nq,d] float64."""
    q = np.asarray(q)
    B, H = q.shape[:2]
    out = np.empty(q.shape, dtype=np.float64)
    for b in range(B):
        for h in range(H):
            out[b, h] = forward_head(q[b, h], k[b, h], v[b, h], softmax_scale, uos, pnq, rotate=rotate)
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
