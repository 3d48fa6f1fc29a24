"""Pins for oracle/mxfp4.py: the oracle is checked against what the paper and arithmetic fix,
never against itself.  CPU only."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import mxfp4, uos_theory
from synth_inputs import bf16_bits_to_f32

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def scalars():
    out = {}
    for line in open(os.path.join(GOLD, "scalars.txt")):
        if line.startswith("#") or not line.strip():
            continue
        p = line.split()
        out[p[0]] = float(p[1])
    return out


# ---------------------------------------------------------------- exact reference helpers
GRID_F = [Fraction(0), Fraction(1, 2), Fraction(1), Fraction(3, 2), Fraction(2), Fraction(3), Fraction(4), Fraction(6)]


def exact_ceil_log2(r: Fraction) -> int:
    """ceil(log2 r) for a positive rational, by integer search (no floating point)."""
    e = 0
    while Fraction(2) ** e < r:
        e += 1
    while Fraction(2) ** (e - 1) >= r:
        e -= 1
    return e


def exact_floor_log2(r: Fraction) -> int:
    e = 0
    while Fraction(2) ** (e + 1) <= r:
        e += 1
    while Fraction(2) ** e > r:
        e -= 1
    return e


def exact_rne_index(x: Fraction) -> int:
    """Nearest E2M1 grid index for x >= 0, ties to the even index, saturating."""
    best, bestd = 0, None
    for i, g in enumerate(GRID_F):
        dist = abs(x - g)
        if bestd is None or dist < bestd or (dist == bestd and i % 2 == 0):
            best, bestd = i, dist
    return best


def all_positive_bf16():
    bits = np.arange(1, 0x7F80, dtype=np.uint16)          # positive finite, nonzero (incl. subnormals)
    return bits, bf16_bits_to_f32(bits).astype(np.float64)


# ---------------------------------------------------------------- grid
def test_grid_and_thresholds_match_paper():
    # Section 2 Eq. 3; Appendix B thresholds
    assert list(mxfp4.E2M1_VALUES) == [0, 0.5, 1, 1.5, 2, 3, 4, 6]
    assert list(mxfp4.E2M1_THRESHOLDS) == [0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0]
    mids = (mxfp4.E2M1_VALUES[:-1] + mxfp4.E2M1_VALUES[1:]) / 2
    assert np.array_equal(mids, mxfp4.E2M1_THRESHOLDS)


def test_saturation_everything_above_5_is_6():
    x = np.array([5.0000001, 6.0, 6.9, 7.0, 7.25, 8.0, 100.0, 1e30])
    assert np.all(mxfp4.E2M1_VALUES[mxfp4.e2m1_index(x)] == 6.0)


def test_ties_go_to_even_code():
    ties = np.array([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0])
    want = np.array([0.0, 1.0, 1.0, 2.0, 2.0, 4.0, 4.0])
    assert np.array_equal(mxfp4.E2M1_VALUES[mxfp4.e2m1_index(ties)], want)


def test_rounding_matches_nearest_neighbour_definition():
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.uniform(0, 8, 200000), np.linspace(0, 8, 3201)])
    got = mxfp4.E2M1_VALUES[mxfp4.e2m1_index(x)]
    near = uos_theory.project(x)                      # argmin |x - g|, written independently
    tie = np.isin(x, mxfp4.E2M1_THRESHOLDS)
    assert np.array_equal(got[~tie], near[~tie])
    # exact rational check on the lattice k/64 (hits every tie)
    lat = [Fraction(k, 64) for k in range(0, 8 * 64 + 1)]
    got = mxfp4.e2m1_index(np.array([float(f) for f in lat]))
    assert list(got) == [exact_rne_index(f) for f in lat]


# ---------------------------------------------------------------- scale rules, exhaustively over bf16
def test_uos_exponent_equals_exact_ceil_log2_all_bf16():
    bits, vals = all_positive_bf16()
    got = mxfp4.shared_exponent(vals, mxfp4.UOS)
    q = Fraction(29, 4)
    # every 7th pattern plus every mantissa pattern of three binades (all 128 mantissas each)
    sel = np.unique(np.concatenate([np.arange(0, bits.size, 7),
                                    np.where((bits >> 7 == 127) | (bits >> 7 == 130) | (bits >> 7 == 1))[0]]))
    for i in sel:
        want = max(-127, min(127, exact_ceil_log2(Fraction(vals[i]) / q)))
        assert got[i] == want, (hex(bits[i]), vals[i], got[i], want)


def test_ocp_exponent_equals_exact_floor_log2_minus_2_all_bf16():
    bits, vals = all_positive_bf16()
    got = mxfp4.shared_exponent(vals, mxfp4.OCP)
    # bf16 normal numbers: floor(log2 M) = biased exponent - 127, exactly
    normal = (bits >> 7) >= 1
    want = np.clip((bits[normal] >> 7).astype(np.int32) - 127 - 2, -127, 127)
    assert np.array_equal(got[normal], want)
    for i in np.where(~normal)[0][::5]:
        want_i = max(-127, exact_floor_log2(Fraction(vals[i])) - 2)
        assert got[i] == want_i


def test_uos_mantissa_rule_in_bf16_bits():
    # 7.25 = 1.8125 * 2^2: the exponent is raised exactly when the 7-bit mantissa field exceeds 104
    bits, vals = all_positive_bf16()
    normal = ((bits >> 7) >= 4) & ((bits >> 7) <= 250)
    e_ocp = mxfp4.shared_exponent(vals[normal], mxfp4.OCP)
    e_uos = mxfp4.shared_exponent(vals[normal], mxfp4.UOS)
    raised = (bits[normal] & 0x7F) > 104
    assert np.array_equal(e_uos - e_ocp, raised.astype(np.int32))


def test_normalized_maximum_ranges_table1():
    s = scalars()
    rng = np.random.default_rng(1)
    M = np.exp2(rng.uniform(-20, 20, 200000))
    M = np.concatenate([M, np.exp2(np.arange(-10, 11)), 7.25 * np.exp2(np.arange(-5, 6)),
                        6.0 * np.exp2(np.arange(-5, 6)), np.nextafter(7.25, 8) * np.exp2(np.arange(-5, 6))])
    for rule, lo, hi, lo_closed in ((mxfp4.OCP, s["ocp_norm_lo"], s["ocp_norm_hi"], True),
                                    (mxfp4.TFS, s["tfs_norm_lo"], s["tfs_norm_hi"], False),
                                    (mxfp4.UOS, s["uos_norm_lo"], s["uos_norm_hi"], False)):
        x = M / np.exp2(mxfp4.shared_exponent(M, rule))
        if lo_closed:
            assert np.all((x >= lo) & (x < hi))
            assert x.min() == lo                     # M = 2^k maps to exactly 4 under the floor rule
        else:
            assert np.all((x > lo) & (x <= hi))
            assert x.max() == hi                     # the endpoint q*2^k maps to exactly q
    # span check: the ranges are actually filled
    x = M / np.exp2(mxfp4.shared_exponent(M, mxfp4.UOS))
    assert x.min() < 3.63 and x.max() == 7.25


def test_floor8_and_ceil8_differ_only_at_powers_of_two():
    # Appendix G, Eq. 57-58
    _, vals = all_positive_bf16()
    vals = vals[(vals > 1e-30) & (vals < 1e30)]
    e_floor = mxfp4.shared_exponent(vals, mxfp4.OCP)
    e_ceil = mxfp4.shared_exponent(vals, mxfp4.ScaleRule("ceil", 8.0))
    pow2 = np.frexp(vals)[0] == 0.5
    assert np.array_equal(e_floor[~pow2], e_ceil[~pow2])
    assert np.array_equal(e_floor[pow2], e_ceil[pow2] + 1)


def test_oas_relation_to_tfs():
    # Appendix G: e_7 = e_6 - 1 when x_6 in (3, 3.5], else e_6
    rng = np.random.default_rng(2)
    M = np.exp2(rng.uniform(-8, 8, 100000))
    M = np.concatenate([M, 3.5 * np.exp2(np.arange(-4, 5)), 6.0 * np.exp2(np.arange(-4, 5))])
    e6 = mxfp4.shared_exponent(M, mxfp4.TFS)
    e7 = mxfp4.shared_exponent(M, mxfp4.OAS)
    x6 = M / np.exp2(e6)
    assert np.array_equal(e7, np.where(x6 <= 3.5, e6 - 1, e6))


def test_ocp_overflow_probability_and_uos_raise_fraction():
    # Eq. 10: under a log-uniform phase P(x_max >= 7) = log2(8/7) = 19.27 %
    s = scalars()
    rng = np.random.default_rng(3)
    M = np.exp2(rng.uniform(-6, 6, 400000))
    x = M / np.exp2(mxfp4.shared_exponent(M, mxfp4.OCP))
    assert abs((x >= 7).mean() - s["ocp_overflow_prob"]) < 3e-3
    assert abs(math.log2(8 / 7) - s["ocp_overflow_prob"]) < 1e-4      # printed to 4 digits
    raised = mxfp4.shared_exponent(M, mxfp4.UOS) - mxfp4.shared_exponent(M, mxfp4.OCP)
    assert set(np.unique(raised)) == {0, 1}
    assert abs(raised.mean() - math.log2(8 / 7.25)) < 3e-3


def test_zero_block_and_clamp():
    codes, e = mxfp4.quantize_blocks(np.zeros((2, 32)), mxfp4.UOS)
    assert np.all(codes == 0) and np.all(e == 0)
    assert np.all(mxfp4.e8m0_bytes(e) == 127)                         # sigma = 1
    tiny = np.zeros((1, 32)); tiny[0, 3] = 2.0 ** -130
    for rule in (mxfp4.OCP, mxfp4.UOS):
        codes, e = mxfp4.quantize_blocks(tiny, rule)
        assert e[0] == -127 and mxfp4.e8m0_bytes(e)[0] == 0
        assert codes[0, 3] == 0                                        # 2^-130 / 2^-127 = 0.125 -> 0
    big = np.zeros((1, 32)); big[0, 0] = float(bf16_bits_to_f32(np.array([0x7F7F], np.uint16))[0])
    _, e = mxfp4.quantize_blocks(big, mxfp4.UOS)
    assert e[0] == 126 and mxfp4.e8m0_bytes(e)[0] == 253              # never 0xFF


def test_uos_of_one_is_one_with_exponent_minus_two():
    # Appendix J worked example
    s = scalars()
    blk = np.zeros((1, 32)); blk[0, 5] = 1.0; blk[0, 6] = 0.3
    codes, e = mxfp4.quantize_blocks(blk, mxfp4.UOS)
    assert e[0] == int(s["uos_exp_of_one"])
    assert mxfp4.dequantize_blocks(codes, e)[0, 5] == 1.0
    assert codes[0, 5] == 6                                            # 1 / 2^-2 = 4 -> index 6


def test_every_bf16_value_alone_in_a_block_rounds_exactly():
    bits, vals = all_positive_bf16()
    sel = np.arange(0, bits.size, 3)
    blocks = np.zeros((sel.size, 32)); blocks[:, 7] = vals[sel]
    for rule, q in ((mxfp4.UOS, Fraction(29, 4)), (mxfp4.OCP, None)):
        codes, e = mxfp4.quantize_blocks(blocks, rule)
        for n, i in enumerate(sel[::11]):
            n = n * 11
            M = Fraction(vals[i])
            ee = exact_ceil_log2(M / q) if q is not None else exact_floor_log2(M) - 2
            ee = max(-127, min(127, ee))
            assert e[n] == ee
            assert codes[n, 7] == exact_rne_index(M / Fraction(2) ** ee)
        assert np.all(np.delete(codes, 7, axis=1) == 0)
        # a lone maximum can only land on a code >= 2 (UOS/OCP keep it in (3.6, 8) -> 4 or 6)
        inrange = (e > -127)
        assert np.all(np.isin(codes[inrange, 7], [6, 7]))


def test_as_block_maximum_with_smaller_companions():
    rng = np.random.default_rng(4)
    x = rng.standard_normal((5000, 32))
    x = bf16_bits_to_f32(__import__("synth_inputs").f32_to_bf16_bits(x.astype(np.float32))).astype(np.float64)
    for rule, q in ((mxfp4.UOS, Fraction(29, 4)), (mxfp4.OCP, None)):
        codes, e = mxfp4.quantize_blocks(x, rule)
        for r in range(0, 5000, 97):
            M = max(Fraction(abs(v)) for v in x[r])
            ee = exact_ceil_log2(M / q) if q is not None else exact_floor_log2(M) - 2
            assert e[r] == ee
            for c in range(32):
                want = exact_rne_index(Fraction(abs(x[r, c])) / Fraction(2) ** ee) | (8 if x[r, c] < 0 else 0)
                assert codes[r, c] == want


def test_invariants_scaling_negation_idempotence():
    rng = np.random.default_rng(5)
    x = bf16_bits_to_f32(__import__("synth_inputs").f32_to_bf16_bits(
        rng.standard_normal((2000, 32)).astype(np.float32))).astype(np.float64)
    for rule in (mxfp4.OCP, mxfp4.UOS, mxfp4.TFS):
        c0, e0 = mxfp4.quantize_blocks(x, rule)
        for k in (-9, 3, 17):
            c1, e1 = mxfp4.quantize_blocks(np.ldexp(x, k), rule)
            assert np.array_equal(c0, c1) and np.array_equal(e0 + k, e1)
        cn, en = mxfp4.quantize_blocks(-x, rule)
        assert np.array_equal(cn, c0 ^ 8) and np.array_equal(en, e0)
        d = mxfp4.dequantize_blocks(c0, e0)
        c2, e2 = mxfp4.quantize_blocks(d, rule)
        d2 = mxfp4.dequantize_blocks(c2, e2)
        assert np.array_equal(d, d2)                                   # Q(Q(x)) = Q(x)


def test_sign_of_values_that_round_to_zero_is_kept():
    blk = np.zeros((1, 32)); blk[0, 0] = 4.0; blk[0, 1] = -0.01; blk[0, 2] = -0.0
    codes, _ = mxfp4.quantize_blocks(blk, mxfp4.UOS)
    assert codes[0, 1] == 8 and codes[0, 2] == 8 and codes[0, 3] == 0


def test_quantization_error_is_lower_with_uos_than_ocp_or_tfs_on_gaussian_data():
    # Section 5.4.1 reports 7.25 as the dominant per-block optimum; on N(0,1) bf16 data the tensor
    # MSE must at least order UOS below both endpoints of the [6, 8] family.
    rng = np.random.default_rng(6)
    x = rng.standard_normal((20000, 32))
    mse = {}
    for name, rule in (("ocp", mxfp4.OCP), ("uos", mxfp4.UOS), ("tfs", mxfp4.TFS)):
        c, e = mxfp4.quantize_blocks(x, rule)
        mse[name] = float(((mxfp4.dequantize_blocks(c, e) - x) ** 2).mean())
    assert mse["uos"] < mse["ocp"] and mse["uos"] < mse["tfs"]


def test_canonical_packing_layouts():
    x = np.zeros((3, 64)); x[1, 0] = 1.0; x[1, 1] = -1.5; x[2, 33] = 6.0
    codes, sc = mxfp4.quantize_matrix_canonical(x, 1, mxfp4.UOS)
    assert codes.shape == (3, 32) and sc.shape == (3, 2)
    # row 1 block 0: M = 1.5 -> e = ceil(log2(1.5/7.25)) = -2 -> 1.0 -> 4 (code 6), -1.5 -> 6 (code 7 | sign)
    assert sc[1, 0] == 125 and codes[1, 0] == (6 | ((7 | 8) << 4))
    assert sc[0, 0] == 127 and sc[2, 1] == 127 and codes[2, 16] == (7 << 4)   # 6.0: e = 0, code 7 high nibble
    # axis 0: transposed, token axis padded to 128
    v = np.zeros((40, 32)); v[0, 5] = 2.0; v[33, 5] = -3.0; v[39, 31] = 0.5
    codes, sc = mxfp4.quantize_matrix_canonical(v, 0, mxfp4.UOS)
    assert codes.shape == (32, 64) and sc.shape == (32, 4)
    assert sc[5, 0] == 126 and codes[5, 0] == 6          # 2.0 / 2^-1 = 4
    assert sc[5, 1] == 126 and codes[5, 16] == ((7 | 8) << 4)   # token 33 -> byte 16 high nibble; -3/0.5 = -6
    assert sc[31, 1] == 124 and codes[31, 19] == (6 << 4)       # 0.5 / 2^-3 = 4, token 39
    assert np.all(sc[:, 2:] == 127) and np.all(codes[:, 20:] == 0)


# ---------------------------------------------------------------- Hadamard rotation (Algorithm 2 lines 1-2)
def test_hadamard_matrix_is_the_sylvester_construction():
    h2 = np.array([[1, 1], [1, -1]], dtype=np.float64)
    h = h2
    for _ in range(6):
        h = np.kron(h2, h)                                   # textbook recursion H_2n = H_2 (x) H_n
    assert np.array_equal(mxfp4.hadamard_matrix(128), h)
    assert np.array_equal(h @ h.T, 128 * np.eye(128))        # orthogonal up to the factor n


def _nearest_f32_of_fraction_over_sqrt128(F: Fraction) -> np.float32:
    """The fp32 nearest to F / sqrt(128) for an exact rational F, decided by exact rational comparisons
    (r < mid  <=>  F^2 / 128 < mid^2 for positive quantities): no floating-point product or square root
    takes part in the decision."""
    if F == 0:
        return np.float32(0.0)
    sign = -1.0 if F < 0 else 1.0
    A2 = F * F / 128                                     # r^2, exact
    c = np.float32(float(abs(F)) / math.sqrt(128.0))     # an estimate: the answer is c or a neighbour
    cands = [np.nextafter(c, np.float32(0)), c, np.nextafter(c, np.float32(np.inf))]
    best = cands[0]
    for lo, hi in zip(cands[:-1], cands[1:]):
        mid = (Fraction(float(lo)) + Fraction(float(hi))) / 2
        if A2 > mid * mid:                               # r is nearer to hi than to lo
            best = hi
        # a tie (A2 == mid^2) is impossible: sqrt(128) is irrational, F and mid are rational
    return np.float32(sign * float(best))


def test_plain_rotation_is_the_exact_product_rounded_once_to_fp32():
    # Algorithm 2, the rotation steps: y = x H_128 / sqrt(128).  Exact rational sums of the +-x_j, then the one
    # correctly rounded fp32 of the irrational quotient -- an evaluation that shares nothing with NumPy's matmul.
    rng = np.random.default_rng(12)
    x = bf16_bits_to_f32(__import__("synth_inputs").f32_to_bf16_bits(rng.standard_normal((3, 128)).astype(np.float32)))
    x[1, [3, 77]] *= 16                                   # an outlier row
    x[2] = np.where(np.arange(128) % 2 == 0, 1.0, -1.0)   # row 1 of H itself: rotates to sqrt(128) e_1
    got = mxfp4.hadamard_rotate(x)
    assert got.dtype == np.float32
    for r in range(3):
        xr = [Fraction(float(t)) for t in x[r]]
        for j in range(0, 128, 5):
            F = sum((-t if bin(i & j).count("1") % 2 else t) for i, t in enumerate(xr))
            assert got[r, j] == _nearest_f32_of_fraction_over_sqrt128(F), (r, j)
    want2 = np.zeros(128, np.float32); want2[1] = np.float32(math.sqrt(128.0))
    assert np.array_equal(got[2], want2)


def test_plain_rotation_is_an_orthogonal_involution_and_keeps_scores():
    rng = np.random.default_rng(13)
    x = bf16_bits_to_f32(__import__("synth_inputs").f32_to_bf16_bits(rng.standard_normal((200, 128)).astype(np.float32)))
    x[::7, 5] *= 16
    y = mxfp4.hadamard_rotate(x).astype(np.float64)
    # H is symmetric and H H = n I: rotating twice returns the input (up to the fp32 roundings of the two results)
    assert np.abs(mxfp4.hadamard_rotate(y).astype(np.float64) - x).max() < 4e-7 * np.abs(x).max()
    assert np.allclose((y ** 2).sum(1), (x.astype(np.float64) ** 2).sum(1), rtol=1e-6)
    k = rng.standard_normal((50, 128)).astype(np.float32)
    s0 = x.astype(np.float64) @ k.astype(np.float64).T
    s1 = y @ mxfp4.hadamard_rotate(k).astype(np.float64).T               # (Q R)(K R)^T = Q K^T
    assert np.abs(s0 - s1).max() < 1e-4
    # transposed or unnormalized variants are different maps: the first column of H is all ones, so the first
    # output is the row sum / sqrt(128)
    assert np.allclose(y[:, 0], x.astype(np.float64).sum(1) / math.sqrt(128.0), rtol=0, atol=1e-5)
    assert np.allclose(y[:, 1], (x[:, 0::2].astype(np.float64).sum(1) - x[:, 1::2].astype(np.float64).sum(1)) / math.sqrt(128.0),
                       rtol=0, atol=1e-5)


def test_rotation_spreads_channel_outliers():
    # the reason the rotation is there (Section 4.3): after it no channel dominates the block maxima
    rng = np.random.default_rng(9)
    x = rng.standard_normal((2000, 128)).astype(np.float32); x[:, [3, 40, 77]] *= 16
    err = lambda z: float(((mxfp4.quantize_dequantize(z, 1, mxfp4.UOS) - z.astype(np.float64)) ** 2).sum() / (z.astype(np.float64) ** 2).sum())
    assert err(mxfp4.hadamard_rotate(x)) < err(x)
