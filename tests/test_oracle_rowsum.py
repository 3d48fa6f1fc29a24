"""Pins for the row-sum diagnostic oracle (Section 5.3): closed-form rows whose outcome classes are known."""
import numpy as np

import synth_inputs as si
from oracle import mxfp4, rowsum


def test_uniform_row_is_reproduced_exactly():
    # p = 2^-k everywhere: normalized value 4 under both rules (e = -k-2), exactly on the grid
    for k in (5, 7, 10):
        p = np.full((3, 2 ** k), 2.0 ** -k)
        for rule in (mxfp4.OCP, mxfp4.UOS):
            out = rowsum.decompose_rows(p, rule)
            assert np.array_equal(out[:, 0], np.ones(3))
            assert np.array_equal(out[:, 1:5], np.zeros((3, 4)))
            np.testing.assert_allclose(out[:, 5], k * np.log(2.0), rtol=1e-14)


def test_zeroing_closed_form():
    # one block: max M = 1/2, the other 31 entries M/64.  e = -3 (OCP: floor(log2 .5) - 2; UOS: ceil(log2(.5/7.25)) = -3),
    # normalized small entries 8/64 = 0.125 < 0.25 -> zero.  Row sum loses 31 * M / 64.
    M = 0.5
    p = np.full((1, 32), M / 64)
    p[0, 7] = M
    for rule in (mxfp4.OCP, mxfp4.UOS):
        out = rowsum.decompose_rows(p, rule)[0]
        assert out[0] == M
        assert out[1] == -31 * M / 64 and out[2] == 0 and out[3] == 0 and out[4] == 0


def test_saturation_differs_between_ocp_and_uos():
    # block maximum 7.5 * 2^-6: OCP keeps e = floor(log2 M) - 2 -> normalized 7.5 > 6: saturates to 6 (loss 1.5 sigma);
    # UOS raises the exponent (7.5 > 7.25) -> normalized 3.75 -> rounds UP to 4 (gain .25 * 2 sigma_ocp)
    sig = 2.0 ** -6
    p = np.zeros((1, 32)); p[0, 0] = 7.5 * sig; p[0, 1] = 2 * sig
    ocp = rowsum.decompose_rows(p, mxfp4.OCP)[0]
    assert ocp[2] == -1.5 * sig and ocp[1] == 0 and ocp[3] == 0 and ocp[4] == 0
    assert ocp[0] == 8 * sig
    uos = rowsum.decompose_rows(p, mxfp4.UOS)[0]
    assert uos[2] == 0 and uos[4] == 0.5 * sig and uos[3] == 0 and uos[1] == 0       # 3.75 -> 4 at sigma = 2 sig
    assert uos[0] == 10 * sig
    # a maximum of exactly 7 saturates under both rules (7 <= 7.25 keeps the exponent, Appendix G)
    p[0, 0] = 7 * sig
    for rule in (mxfp4.OCP, mxfp4.UOS):
        assert rowsum.decompose_rows(p, rule)[0][2] == -1.0 * sig


def test_down_and_up_rounding_closed_form():
    # normalized values 4 (max), 2.4 -> 2 (down .4), 2.6 -> 3 (up .4), 1.2 -> 1 (down .2), 1.3 -> 1.5 (up .2)
    sig = 2.0 ** -9
    vals = np.array([4.0, 2.4, 2.6, 1.2, 1.3])
    p = np.zeros((1, 32)); p[0, :5] = np.float32(vals * sig)
    out = rowsum.decompose_rows(p, mxfp4.UOS)[0]
    pf = p[0, :5] / sig
    want_down = ((2 - pf[1]) + (1 - pf[3])) * sig
    want_up = ((3 - pf[2]) + (1.5 - pf[4])) * sig
    np.testing.assert_allclose(out[3], want_down, rtol=1e-12)
    np.testing.assert_allclose(out[4], want_up, rtol=1e-12)
    assert out[1] == 0 and out[2] == 0


def test_contributions_add_up_and_blocks_are_zero_extended():
    rng = np.random.default_rng(5)
    s = rng.standard_normal((64, 1000)) * 2.0
    p = rowsum.softmax_rows_f32(s)
    for rule in (mxfp4.OCP, mxfp4.UOS):
        out = rowsum.decompose_rows(p, rule)
        np.testing.assert_allclose(out[:, 1:5].sum(axis=1), out[:, 0] - p.sum(axis=1), atol=1e-15)
        # the same result when the row is explicitly padded with zeros to a multiple of 32
        out2 = rowsum.decompose_rows(np.concatenate([p, np.zeros((64, 24))], axis=1), rule)
        assert np.array_equal(out[:, :5], out2[:, :5])
        np.testing.assert_allclose(out[:, 5], out2[:, 5], rtol=1e-13)


def test_high_entropy_rows_are_under_normalized():
    # Section 5.3, panel D (qualitative): flat rows lose mass under quantization of the materialized probabilities;
    # with the UOS rule the loss is smaller than with the OCP rule
    cfg = si.custom_config("d", 1, 1, 256, 2048, 9)
    q, k, _ = si.make_head(cfg, 0, 0)
    f = lambda b: si.bf16_bits_to_f32(b).astype(np.float64)
    ocp = rowsum.diagnostic_head(f(q), f(k), cfg.softmax_scale, uos=False)
    uos = rowsum.diagnostic_head(f(q), f(k), cfg.softmax_scale, uos=True)
    assert (ocp[:, 5] > 5.0).all()                       # entropy of softmax over 2048 iid N(0,1)-scores ~ 7.1
    assert ocp[:, 0].mean() < 0.99 and (ocp[:, 0] < 1.0).mean() > 0.95
    assert uos[:, 2].mean() > ocp[:, 2].mean()           # less saturation loss (closer to 0)
    assert abs(uos[:, 0].mean() - 1.0) < abs(ocp[:, 0].mean() - 1.0)
