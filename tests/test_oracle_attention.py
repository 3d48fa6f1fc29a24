"""Pins for oracle/attention.py (Algorithm 2): special cases that reduce to textbook formulas,
the paper's normalization identities, and a scalar brute force on tiny inputs.  CPU only."""
import math
from fractions import Fraction

import numpy as np
import pytest

import synth_inputs as si
from oracle import attention, mxfp4

SCALE = 1.0 / math.sqrt(128.0)


def head(nq, nkv, seed, recipe="iid", d=128):
    cfg = si.custom_config("t", 1, 1, nq, nkv, seed, recipe)
    q, k, v = si.make_head(cfg, 0, 0)
    f = lambda a: si.bf16_bits_to_f32(a).astype(np.float64)[:, :d]
    return f(q), f(k), f(v)


def rel_l2(a, b):
    return float(np.linalg.norm(a - b) / np.linalg.norm(b))


# ------------------------------------------------------------------ recurrence plumbing
@pytest.mark.parametrize("nkv", [128, 200, 1000])
def test_identity_quantizer_reduces_to_dense_softmax_attention(nkv):
    q, k, v = head(70, nkv, 11)
    got = attention.forward_head(q, k, v, SCALE, quantize_inputs=False, quantize_p=False)
    # P~ is still rounded to fp32 in the oracle, so compare at fp32 resolution here ...
    want = attention.dense_attention_head(q, k, v, SCALE)
    assert np.abs(got - want).max() < 2e-7
    # ... and check the recurrence itself to 1e-12 by repeating it in float64 right here
    m = np.full(70, -np.inf); l = np.zeros(70); o = np.zeros((70, 128))
    sc = float(np.float32(SCALE))
    for j0 in range(0, nkv, 128):
        s = q @ k[j0:j0 + 128].T * sc
        mn = np.maximum(m, s.max(1)); a = np.exp(m - mn); p = np.exp(s - mn[:, None])
        l = a * l + p.sum(1); o = a[:, None] * o + p @ v[j0:j0 + 128]; m = mn
    assert np.abs(o / l[:, None] - want).max() < 1e-12


def test_single_tile_equals_direct_formula():
    # Nkv <= 128: O = Q(exp(S - max)) V-hat / sum Q(.)  evaluated without any recurrence
    q, k, v = head(40, 96, 12)
    for uos in (True, False):
        rule = mxfp4.UOS if uos else mxfp4.OCP
        qd, kd, vd = attention.quantize_qkv(q, k, v, rule)
        s = qd @ kd.T * float(np.float32(SCALE))
        p = np.exp(s - s.max(1, keepdims=True)).astype(np.float32).astype(np.float64)
        ppad = np.zeros((40, 128)); ppad[:, :96] = p
        ph = mxfp4.quantize_dequantize(ppad, axis=1, rule=rule)[:, :96]
        want_pnq = (ph @ vd) / ph.sum(1, keepdims=True)
        want_dir = (ph @ vd) / p.sum(1, keepdims=True)
        assert np.allclose(attention.forward_head(q, k, v, SCALE, uos, True), want_pnq, rtol=0, atol=1e-14)
        assert np.allclose(attention.forward_head(q, k, v, SCALE, uos, False), want_dir, rtol=0, atol=1e-14)


def test_all_equal_scores_give_column_mean_of_quantized_v():
    _, k, v = head(4, 640, 13)
    q = np.zeros((4, 128))
    vd = mxfp4.quantize_dequantize(v, 0, mxfp4.UOS)
    got = attention.forward_head(q, k, v, SCALE, True, True)
    # every P~ = 1 -> P-hat = 1 exactly (Appendix J) -> plain mean
    assert np.allclose(got, np.broadcast_to(vd.mean(0), got.shape), rtol=0, atol=1e-14)


# ------------------------------------------------------------------ normalization (Prop. 1, Lemma 2, App. I/J)
def effective_rows(state):
    m_final = state["m"][-1]
    ph, pt = [], []
    for mj, p_hat, p_tilde in zip(state["m"], state["p_hat"], state["p_tilde"]):
        beta = np.exp(mj - m_final)[:, None]                         # Eq. 59
        ph.append(beta * p_hat); pt.append(beta * p_tilde)
    return np.concatenate(ph, 1), np.concatenate(pt, 1)


@pytest.mark.parametrize("recipe,nkv", [("iid", 1024), ("iid", 1000), ("outlier", 1024)])
def test_pnq_weights_sum_to_one_and_match_unrolled_form(recipe, nkv):
    q, k, v = head(256, nkv, 14, recipe)
    out, st = attention.forward_head(q, k, v, SCALE, True, True, return_state=True)
    ph_eff, _ = effective_rows(st)
    # Lemma 2: l = P-hat_eff 1, O~ = P-hat_eff V-hat
    assert np.allclose(st["l"], ph_eff.sum(1), rtol=1e-13)
    assert np.allclose(st["o_tilde"], ph_eff @ st["vd"], rtol=0, atol=1e-11)
    # Proposition 1: induced weights sum to one on every row
    w = ph_eff / st["l"][:, None]
    assert np.abs(w.sum(1) - 1.0).max() < 1e-6
    assert np.abs(out - w @ st["vd"]).max() < 1e-12
    # Appendix J: l >= 1 on every row
    assert st["l"].min() >= 1.0


def test_direct_placement_rows_do_not_sum_to_one():
    q, k, v = head(512, 1024, 15)
    _, st = attention.forward_head(q, k, v, SCALE, True, False, return_state=True)
    ph_eff, pt_eff = effective_rows(st)
    assert np.allclose(st["l"], pt_eff.sum(1), rtol=1e-13)            # Eq. 12: l from unquantized tiles
    rowsum = ph_eff.sum(1) / pt_eff.sum(1)                            # Eq. 14 / Eq. 66
    assert np.abs(rowsum - 1).max() > 1e-3
    # high-entropy rows are under-normalized on average (Section 5.4.2)
    assert 0.9 < rowsum.mean() < 0.995


def test_constant_v_invariant():
    q, k, _ = head(128, 1000, 16)
    v = np.ones((1000, 128))
    o_pnq = attention.forward_head(q, k, v, SCALE, True, True)
    assert np.abs(o_pnq - 1).max() < 1e-12
    o_dir = attention.forward_head(q, k, v, SCALE, True, False)
    assert np.abs(o_dir - 1).max() > 1e-3                               # the direct placement leaks the row sum


# ------------------------------------------------------------------ quality orderings vs float64 dense
def test_uos_is_closer_to_dense_attention_than_ocp():
    for recipe, seed in (("iid", 17), ("outlier", 18)):
        q, k, v = head(256, 1024, seed, recipe)
        dense = attention.dense_attention_head(q, k, v, SCALE)
        e_uos = rel_l2(attention.forward_head(q, k, v, SCALE, True, True), dense)
        e_ocp = rel_l2(attention.forward_head(q, k, v, SCALE, False, False), dense)
        assert e_uos < e_ocp < 1.0


# ------------------------------------------------------------------ scalar brute force
def scalar_quantize(block, uos):
    """32 Python floats -> dequantized floats, by exact rational arithmetic."""
    M = max(Fraction(abs(x)) for x in block)
    if M == 0:
        return [0.0] * len(block)
    e = 0
    if uos:                       # smallest e with M <= 7.25 * 2^e
        while M > Fraction(29, 4) * Fraction(2) ** e:
            e += 1
        while M <= Fraction(29, 4) * Fraction(2) ** (e - 1):
            e -= 1
    else:                         # floor(log2 M) - 2
        while Fraction(2) ** (e + 1) <= M:
            e += 1
        while Fraction(2) ** e > M:
            e -= 1
        e -= 2
    e = max(-127, min(127, e))
    grid = [Fraction(g) for g in (0, 0.5, 1, 1.5, 2, 3, 4, 6)]
    out = []
    for x in block:
        r = Fraction(abs(x)) / Fraction(2) ** e
        best = min(range(8), key=lambda i: (abs(r - grid[i]), i % 2))
        val = float(grid[best] * Fraction(2) ** e)
        out.append(-val if x < 0 else val)
    return out


@pytest.mark.parametrize("uos,pnq", [(True, True), (True, False), (False, False), (False, True)])
def test_against_scalar_python_loops(uos, pnq):
    nq, nkv, d = 3, 150, 32
    q, k, v = head(nq, nkv, 19)
    q, k, v = q[:, :d].copy(), k[:, :d].copy(), v[:, :d].copy()
    scale = 1.0 / math.sqrt(d)
    got = attention.forward_head(q, k, v, scale, uos, pnq)
    sc = float(np.float32(scale))
    qd = [scalar_quantize(list(q[i]), uos) for i in range(nq)]
    kd = [scalar_quantize(list(k[i]), uos) for i in range(nkv)]
    nkv_pad = -(-nkv // 32) * 32
    vd = [[0.0] * d for _ in range(nkv_pad)]
    for c in range(d):
        for b0 in range(0, nkv_pad, 32):
            blk = [float(v[t, c]) if t < nkv else 0.0 for t in range(b0, b0 + 32)]
            for t, val in zip(range(b0, b0 + 32), scalar_quantize(blk, uos)):
                vd[t][c] = val
    for i in range(nq):
        m, l, o = -math.inf, 0.0, [0.0] * d
        for j0 in range(0, nkv, 128):
            cols = range(j0, min(j0 + 128, nkv))
            s = {c: sum(qd[i][t] * kd[c][t] for t in range(d)) * sc for c in cols}
            m_new = max(m, max(s.values()))
            alpha = math.exp(m - m_new) if m > -math.inf else 0.0
            pt = [float(np.float32(math.exp(s[c] - m_new))) if c in s else 0.0 for c in range(j0, j0 + 128)]
            ph = []
            for b0 in range(0, 128, 32):
                ph += scalar_quantize(pt[b0:b0 + 32], uos)
            l = alpha * l + (sum(ph) if pnq else sum(pt))
            o = [alpha * o[t] + sum(ph[c - j0] * vd[c][t] for c in cols) for t in range(d)]
            m = m_new
        for t in range(d):
            assert abs(o[t] / l - got[i, t]) < 1e-12


# ------------------------------------------------------------------ tails and row sampling
def test_tail_columns_do_not_contribute():
    q, k, v = head(16, 300, 20)
    base = attention.forward_head(q, k, v, SCALE)
    # appending keys whose scores are hugely negative is the same as masking them:
    # the masked-tail implementation must agree with a run that simply has fewer keys
    k2 = np.concatenate([k, np.zeros((84, 128))]); v2 = np.concatenate([v, np.zeros((84, 128))])
    full = attention.forward_head(q, k2, v2, SCALE)           # zero keys DO contribute (score 0) -> must differ
    assert np.abs(full - base).max() > 1e-6
    # V blocks along tokens: the last block (tokens 288..299) is zero-extended, scale from valid tokens only
    vd = mxfp4.quantize_dequantize(v, 0, mxfp4.UOS)
    vpad = np.concatenate([v, np.zeros((20, 128))])
    assert np.array_equal(mxfp4.quantize_dequantize(vpad, 0, mxfp4.UOS)[:300], vd)


def test_row_sampling_equals_full_run():
    q, k, v = head(300, 700, 21)
    rows = np.array([0, 5, 127, 128, 255, 299])
    full = attention.forward_head(q, k, v, SCALE, True, True)
    assert np.allclose(attention.forward_head(q, k, v, SCALE, True, True, rows=rows), full[rows], rtol=0, atol=1e-13)


def test_all_heads_wrapper():
    cfg = si.custom_config("t", 1, 2, 64, 256, 22)
    q, k, v = si.make_all(cfg)
    f = lambda a: si.bf16_bits_to_f32(a).astype(np.float64)
    out = attention.forward(f(q), f(k), f(v), SCALE)
    assert out.shape == (1, 2, 64, 128)
    assert np.allclose(out[0, 1], attention.forward_head(f(q)[0, 1], f(k)[0, 1], f(v)[0, 1], SCALE), rtol=0, atol=1e-13)


def test_rotation_brings_the_quantized_output_closer_to_dense_attention_on_outlier_data():
    # Table 3 of the paper attributes the largest quality gain to the Hadamard rotation; on synthetic
    # channel-outlier data the ordering must at least hold
    q, k, v = head(256, 1024, 23, "outlier")
    dense = attention.dense_attention_head(q, k, v, SCALE)
    plain = rel_l2(attention.forward_head(q, k, v, SCALE, True, True), dense)
    rot = rel_l2(attention.forward_head(q, k, v, SCALE, True, True, rotate=True), dense)
    assert rot < plain


def test_rotation_with_identity_quantizer_changes_nothing():
    q, k, v = head(32, 256, 24)
    rq = mxfp4.hadamard_rotate(q).astype(np.float64); rk = mxfp4.hadamard_rotate(k).astype(np.float64)
    a = attention.forward_head(rq, rk, v, SCALE, quantize_inputs=False, quantize_p=False)
    b = attention.dense_attention_head(q, k, v, SCALE)
    assert np.abs(a - b).max() < 1e-5


def _scalar_bf16(x: float) -> float:
    """fp32 -> bf16 round-to-nearest-even by exact arithmetic on the significand (Python ints only)."""
    if x == 0.0:
        return 0.0
    mant, exp = math.frexp(abs(x))                 # |x| = mant * 2^exp, mant in [0.5, 1)
    scaled = Fraction(mant) * 256                  # 8 significant bits: integer part in [128, 256)
    lo = int(scaled)
    rem = scaled - lo
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and lo % 2 == 1):
        lo += 1
    return math.copysign(math.ldexp(lo, exp - 8), x)


def _scalar_bf16_attention(q, k, v, sc, p_for_gemm, p_for_sum):
    """The recurrence of Section 2 (Eq. 2-3) in scalar Python; `p_for_gemm` / `p_for_sum` say which version
    of the exponentials ("bf16" or "fp32") enters the P V product and the row sum."""
    nq, d = q.shape
    nkv = k.shape[0]
    pick = lambda p, kind: _scalar_bf16(p) if kind == "bf16" else p
    out = []
    for i in range(nq):
        m, l, o = -math.inf, 0.0, [0.0] * d
        for j0 in range(0, nkv, 128):
            cols = range(j0, min(j0 + 128, nkv))
            s = [sum(float(q[i, t]) * float(k[c, t]) for t in range(d)) * sc for c in cols]
            m_new = max(m, max(s))
            alpha = math.exp(m - m_new) if m > -math.inf else 0.0
            p32 = [float(np.float32(math.exp(x - m_new))) for x in s]
            l = alpha * l + sum(pick(p, p_for_sum) for p in p32)
            o = [alpha * o[t] + sum(pick(p, p_for_gemm) * float(v[c, t]) for p, c in zip(p32, cols)) for t in range(d)]
            m = m_new
        out.append([x / l for x in o])
    return np.array(out)


def test_bf16_variant_against_scalar_python_loops():
    # What distinguishes the bf16 variant: the exponentials are rounded to bf16 ONLY for the P V product, and the
    # row sum is taken from the fp32 exponentials.  The scalar restatement with exactly those choices must agree
    # to rounding-order noise; with either choice swapped it must not.
    nq, nkv, d = 3, 300, 16
    q, k, v = head(nq, nkv, 26)
    q, k, v = q[:, :d].copy(), k[:, :d].copy(), v[:, :d].copy()
    scale = 1.0 / math.sqrt(d)
    sc = float(np.float32(scale))
    got = attention.forward_head_bf16(q, k, v, scale)
    assert np.abs(_scalar_bf16_attention(q, k, v, sc, "bf16", "fp32") - got).max() < 1e-12
    assert np.abs(_scalar_bf16_attention(q, k, v, sc, "bf16", "bf16") - got).max() > 1e-6     # row sum from bf16 P
    assert np.abs(_scalar_bf16_attention(q, k, v, sc, "fp32", "fp32") - got).max() > 1e-6     # P not rounded at all
    # the scalar rounding helper and the oracle's agree, ties included
    xs = np.array([1.0, 1.00390625, 1.01171875, -3.0, 0.1, 1e-20, 3.3895313892515355e+38, 1.0000001], np.float32)
    assert [float(t) for t in attention._round_to_bf16(xs)] == [_scalar_bf16(float(t)) for t in xs]


def test_bf16_variant_oracle_is_dense_attention_up_to_bf16_rounding_of_p():
    q, k, v = head(64, 700, 25)
    a = attention.forward_head_bf16(q, k, v, SCALE)
    b = attention.dense_attention_head(q, k, v, SCALE)
    assert 1e-6 < rel_l2(a, b) < 5e-3          # only P is rounded (2^-9 relative), and it must be rounded
    # rounding helper: exact on bf16-representable values, RNE on a tie
    r = attention._round_to_bf16(np.array([1.0, 1.00390625, 1.01171875, -3.0], np.float32))
    assert list(r) == [1.0, 1.0, 1.015625, -3.0]
