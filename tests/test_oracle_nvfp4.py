"""Pins for oracle/nvfp4.py (the comparison format of the paper's Section 5.2): the E4M3 table and its rounding
against the format's definition in exact rational arithmetic, the quantizer against an exact-rational evaluation of
the two-level recipe, and the invariants that follow from it.  CPU only."""
import math
from fractions import Fraction

import numpy as np
import pytest

from oracle import attention, mxfp4, nvfp4
from synth_inputs import bf16_bits_to_f32, f32_to_bf16_bits

GRID_F = [Fraction(0), Fraction(1, 2), Fraction(1), Fraction(3, 2), Fraction(2), Fraction(3), Fraction(4), Fraction(6)]


def e4m3_value(code: int) -> Fraction:
    """The format's definition from its bit fields: 4 exponent bits (bias 7), 3 mantissa bits, subnormals at e = 0."""
    e, m = (code >> 3) & 15, code & 7
    return Fraction(m, 8) * Fraction(1, 64) if e == 0 else (1 + Fraction(m, 8)) * Fraction(2) ** (e - 7)


def exact_nearest(y: Fraction, values, saturate=True) -> int:
    """Index of the value nearest to y >= 0, ties to the even index, by exact comparison."""
    best, best_d = 0, None
    for i, v in enumerate(values):
        d = abs(y - v)
        if best_d is None or d < best_d or (d == best_d and i % 2 == 0):
            best, best_d = i, d
    return best


E4M3_F = [e4m3_value(c) for c in range(127)]


def test_e4m3_table_is_the_format():
    t = nvfp4.e4m3_table()
    assert len(t) == 127
    assert [Fraction(float(x)) for x in t] == E4M3_F
    assert t[0] == 0 and t[1] == 2.0 ** -9 and t[7] == 7 * 2.0 ** -9 and t[8] == 2.0 ** -6      # subnormals, first normal
    assert t[0x38] == 1.0 and t[0x7E] == 448.0 and t[0x40] == 2.0 and t[0x3C] == 1.5
    assert np.all(np.diff(t) > 0)                                                               # code order = value order


def test_e4m3_rounding_is_nearest_ties_to_even_saturating():
    rng = np.random.default_rng(3)
    ys = list(np.exp2(rng.uniform(-12, 9.5, 3000)).astype(np.float32))
    mids = [(a + b) / 2 for a, b in zip(E4M3_F[:-1], E4M3_F[1:])]
    ys += [np.float32(float(m)) for m in mids]                                                  # every tie (all exact in fp32)
    ys += [np.nextafter(np.float32(float(m)), np.float32(0)) for m in mids[::5]] + [np.nextafter(np.float32(float(m)), np.float32(1e9)) for m in mids[::5]]
    ys += [np.float32(0), np.float32(448), np.float32(464), np.float32(1e30), np.float32(2.0 ** -10), np.float32(2.0 ** -11)]
    got = nvfp4.e4m3_round(np.array(ys, np.float32))
    for y, g in zip(ys, got):
        want = exact_nearest(min(Fraction(float(y)), Fraction(448)), E4M3_F)
        assert int(g) == want, (float(y), int(g), want)
    assert nvfp4.e4m3_round(np.float32(2.0 ** -10)) == 0 and nvfp4.e4m3_round(np.float32(3 * 2.0 ** -10)) == 2   # ties -> even code


def exact_recipe(x, amax, g=None):
    """The two-level recipe in exact rational arithmetic for one block: d = E4M3(M g / 6), code = E2M1(|x| g / d)."""
    g = Fraction(2688) / Fraction(float(amax)) if g is None else g
    M = max(abs(Fraction(float(t))) for t in x)
    sc = exact_nearest(min(M * g / 6, Fraction(448)), E4M3_F)
    d = E4M3_F[sc]
    codes = []
    for t in x:
        a = abs(Fraction(float(t)))
        idx = 0 if d == 0 else exact_nearest(min(a * g / d, Fraction(6)), GRID_F)
        codes.append(idx | (8 if math.copysign(1.0, float(t)) < 0 else 0))
    return codes, sc


def test_block_quantizer_equals_the_exact_recipe_when_the_tensor_scale_is_a_power_of_two():
    # A = 2688 * 2^k makes g = 2^-k exact, so M g is exact and the only inexact step left, the multiplication by
    # fl32(1/6), is 6e-8 away from M g / 6: dyadic inputs whose quotients are far from every rounding boundary
    # must then give exactly the codes of the exact-rational recipe.
    rng = np.random.default_rng(5)
    for k in (-3, 0, 4):
        amax = np.float32(2688.0 * 2.0 ** k)
        for _ in range(40):
            x = bf16_bits_to_f32(f32_to_bf16_bits((rng.standard_normal(16) * 2.0 ** (k + rng.integers(0, 9))).astype(np.float32)))
            codes, sc, s_t = nvfp4.quantize_blocks(x[None, :], amax)
            want_codes, want_sc = exact_recipe(x, amax)
            assert float(s_t) == 2.0 ** k
            assert int(sc[0]) == want_sc
            # the element quotient |x| g / d is compared away from ties only (a tie of the exact recipe can be broken
            # either way by the fp32 division)
            g = Fraction(2688) / Fraction(float(amax)); d = E4M3_F[want_sc]
            for i, t in enumerate(x):
                if d == 0:
                    continue
                quo = abs(Fraction(float(t))) * g / d
                near_tie = any(abs(quo - th) < Fraction(1, 10 ** 5) * max(quo, 1) for th in (Fraction(1, 4), Fraction(3, 4), Fraction(5, 4), Fraction(7, 4), Fraction(5, 2), Fraction(7, 2), Fraction(5)))
                if not near_tie:
                    assert int(codes[0, i]) == want_codes[i], (k, i, float(t))


def test_fp32_evaluation_agrees_with_the_exact_recipe_except_at_rounding_boundaries():
    # general tensor maxima: the fp32 steps (g, M g, * fl32(1/6), g / d, x r) carry about 1e-7 of relative noise, which
    # moves a scale or a code only when the exact quotient sits that close to a boundary
    rng = np.random.default_rng(6)
    x = bf16_bits_to_f32(f32_to_bf16_bits(rng.standard_normal((600, 16)).astype(np.float32) * np.float32(3.7)))
    amax = np.abs(x).max()
    codes, sc, s_t = nvfp4.quantize_blocks(x, amax)
    bad_sc = bad_codes = 0
    for b in range(x.shape[0]):
        want_codes, want_sc = exact_recipe(x[b], amax)
        bad_sc += int(sc[b]) != want_sc
        if int(sc[b]) == want_sc:
            bad_codes += sum(int(c) != w for c, w in zip(codes[b], want_codes))
    assert bad_sc <= 1 and bad_codes <= 2, (bad_sc, bad_codes)
    assert abs(float(s_t) * 2688.0 / float(amax) - 1.0) < 3e-7


def test_invariants_scaling_negation_zero_and_the_tensor_maximum():
    rng = np.random.default_rng(7)
    x = rng.standard_normal((64, 16)).astype(np.float32)
    amax = np.abs(x).max()
    c0, s0, t0 = nvfp4.quantize_blocks(x, amax)
    # a power-of-two change of units moves only the tensor scale
    c1, s1, t1 = nvfp4.quantize_blocks(x * np.float32(2.0 ** 7), amax * np.float32(2.0 ** 7))
    assert np.array_equal(c0, c1) and np.array_equal(s0, s1) and float(t1) == float(t0) * 2.0 ** 7
    # negation flips sign bits only
    c2, s2, _ = nvfp4.quantize_blocks(-x, amax)
    assert np.array_equal(c2 ^ 8, c0) and np.array_equal(s2, s0)
    # the element holding the tensor maximum is represented as 6 * 448 * s_T, i.e. (up to the rounding of g) itself
    i, j = np.unravel_index(np.abs(x).argmax(), x.shape)
    assert (c0[i, j] & 7) == 7 and s0[i] == 0x7E
    deq = nvfp4.dequantize_blocks(c0, s0, np.broadcast_to(t0, s0.shape))
    assert abs(abs(deq[i, j]) - float(amax)) < 1e-6 * float(amax)
    # zero block inside a non-zero tensor, and an all-zero tensor
    z = x.copy(); z[3] = 0
    cz, sz, _ = nvfp4.quantize_blocks(z, amax)
    assert sz[3] == 0 and np.all(cz[3] == 0)
    cz, sz, tz = nvfp4.quantize_blocks(np.zeros((2, 16), np.float32), 0.0)
    assert np.all(cz == 0) and np.all(sz == 0) and float(tz) == 1.0
    # block maxima land near the top of the E2M1 grid: after scaling, the maximum of a block is within the E4M3
    # rounding (1/16 relative) of 6, so it rounds to 6 (index 7) or, at worst, is carried by 4
    top = (c0 & 7).max(axis=1)
    assert np.all(top[s0 > 8] >= 6)


def test_error_is_below_mxfp4_on_gaussian_data():
    # the reason the paper lists NVFP4 as the finer-grained comparison format (Introduction): 16-element blocks and a
    # 3-bit-mantissa scale beat 32-element blocks with a power-of-two scale on tensor MSE
    x = np.random.default_rng(8).standard_normal((2048, 128))
    mse = lambda dq: float(((dq - x) ** 2).mean())
    nv = mse(nvfp4.quantize_dequantize(x, 1))
    assert nv < mse(mxfp4.quantize_dequantize(x, 1, mxfp4.UOS)) < mse(mxfp4.quantize_dequantize(x, 1, mxfp4.OCP))
    assert 0.006 < nv < 0.012          # relative error of a 4-bit float with a fitted scale: about 9 % rms


def test_canonical_layouts():
    x = np.zeros((3, 32)); x[1, 0] = 6.0; x[1, 17] = -3.0; x[2, 31] = 0.75
    codes, sc, s_t = nvfp4.quantize_matrix_canonical(x, 1)
    assert codes.shape == (3, 16) and sc.shape == (3, 2) and float(s_t) == float(np.float32(1) / (np.float32(2688) / np.float32(6)))
    assert sc[1, 0] == 0x7E and codes[1, 0] == 7                     # the tensor maximum: scale 448, code 6.0
    assert sc[1, 1] == 0x76 and codes[1, 8] == ((7 | 8) << 4)        # block maximum 3 = half the tensor maximum: scale 224
    assert sc[0, 0] == 0 and np.all(codes[0] == 0)
    # 0.75 alone: y = 0.75 * 448 / 6 = 56 -> E4M3 56 = 1.75 * 2^5 (code 0x66); element 0.75 * 448 / 56 = 6
    assert sc[2, 1] == 0x66 and codes[2, 15] == (7 << 4)
    v = np.zeros((40, 8)); v[0, 5] = 2.0; v[33, 5] = -2.0
    codes, sc, _ = nvfp4.quantize_matrix_canonical(v, 0)
    assert codes.shape == (8, 64) and sc.shape == (8, 8)
    assert sc[5, 0] == 0x7E and codes[5, 0] == 7 and sc[5, 2] == 0x7E and codes[5, 16] == ((7 | 8) << 4)
    assert np.all(sc[:, 3:] == 0) and np.all(codes[:, 24:] == 0)


def test_attention_with_nvfp4_operands():
    rng = np.random.default_rng(9)
    f = lambda a: bf16_bits_to_f32(f32_to_bf16_bits(a.astype(np.float32))).astype(np.float64)
    q, k, v = f(rng.standard_normal((48, 128))), f(rng.standard_normal((300, 128))), f(rng.standard_normal((300, 128)))
    scale = 1 / math.sqrt(128)
    dense = attention.dense_attention_head(q, k, v, scale)
    rel = lambda a: float(np.linalg.norm(a - dense) / np.linalg.norm(dense))
    nv_pnq = attention.forward_head(q, k, v, scale, pnq=True, fmt="nvfp4")
    nv_dir = attention.forward_head(q, k, v, scale, pnq=False, fmt="nvfp4")
    mx = attention.forward_head(q, k, v, scale, True, True)
    assert rel(nv_pnq) < rel(mx) and rel(nv_dir) < rel(mx)          # the finer format is closer to dense attention
    assert 0.05 < rel(nv_pnq) < 0.3
    # V = 1 in every channel: P-hat V-hat is then the row sum of P-hat times V-hat's single value, so under PNQ the
    # output is exactly that value in every row, whatever the probabilities; the direct placement divides by a
    # different sum and is not
    ones = np.ones_like(v)
    o = attention.forward_head(q, k, ones, scale, pnq=True, fmt="nvfp4")
    vhat = nvfp4.quantize_dequantize(ones, 0)[0, 0]
    assert np.abs(o - vhat).max() < 1e-12 and abs(vhat - 1.0) < 1e-6
    o = attention.forward_head(q, k, ones, scale, pnq=False, fmt="nvfp4")
    assert np.abs(o - vhat).max() > 1e-4
    # single tile: the loop reduces to NVFP4(exp(S - max)) V-hat / sum, evaluated directly
    k1, v1 = k[:100], v[:100]
    qd, kd, vd = attention.quantize_qkv(q, k1, v1, None, fmt="nvfp4")
    s = (qd @ kd.T) * float(np.float32(scale))
    p = np.zeros((48, 128)); p[:, :100] = np.exp(s - s.max(1, keepdims=True)).astype(np.float32)
    c, sc, st = nvfp4.quantize_blocks(p.reshape(48, 8, 16), 1.0)
    ph = nvfp4.dequantize_blocks(c, sc, np.broadcast_to(st, sc.shape)).reshape(48, 128)[:, :100]
    want = (ph @ vd) / ph.sum(1, keepdims=True)
    assert np.abs(attention.forward_head(q, k1, v1, scale, pnq=True, fmt="nvfp4") - want).max() < 1e-12
