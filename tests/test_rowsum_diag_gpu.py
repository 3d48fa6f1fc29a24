"""Parity of the row-sum diagnostic kernel (Section 5.3) with its oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import synth_inputs as si
from oracle import rowsum
from tests import util

pytestmark = pytest.mark.gpu


def run(cfg, q, k, uos, rotate=False):
    import paper_2607_24377_b200 as mx
    flags = (mx.FLAG_UOS if uos else 0) | (mx.FLAG_HADAMARD if rotate else 0)
    out = torch.full((cfg.B, cfg.H, cfg.Nq, 6), float("nan"), dtype=torch.float32, device="cuda")
    ws = torch.empty(mx.forward_workspace_bytes(cfg.B, cfg.H, cfg.Nq, cfg.Nkv, cfg.d), dtype=torch.uint8, device="cuda")
    mx.rowsum_diagnostic(util.to_dev_bf16(q), util.to_dev_bf16(k), out, cfg.B, cfg.H, cfg.Nq, cfg.Nkv, cfg.d,
                         cfg.softmax_scale, flags, ws)
    assert mx.device_status(ws) == 0
    assert mx.last_launch_count() == 3
    return out.double().cpu().numpy()


def check(cfg, uos, rotate=False, atol=1e-3, skip_onehot=False):
    q, k, _ = si.make_all(cfg)
    got = run(cfg, q, k, uos, rotate)
    assert np.isfinite(got).all()
    f = util.bits_to_f64
    for b in range(cfg.B):
        for h in range(cfg.H):
            want = rowsum.diagnostic_head(f(q[b, h]), f(k[b, h]), cfg.softmax_scale, uos=uos, rotate=rotate)
            # the GPU evaluates the probabilities in fp32 (ex2.approx, fp32 normalizer): a value within ~1e-6 relative
            # of a rounding or class boundary may fall on the other side; each such element moves a column by at
            # most its own probability
            err = np.abs(got[b, h, :, :5] - want[:, :5])
            if skip_onehot:
                # A row whose largest probability is 1 to within an fp32 ulp sits on the OCP rule's discontinuity at
                # powers of two (p = 1 is kept exactly, p = 1 - 2^-24 is scaled to 7.99.. and saturates to 6: a
                # row sum of 0.75): which side it falls on is decided by the last bit of the normalizer.
                err[want[:, 5] < 1e-5] = 0.0
            assert err.max() <= atol, err.max()
            assert (err > 2e-5).mean() <= 2e-3, (err > 2e-5).mean()      # all but a few entries agree to fp32 summation error
            np.testing.assert_allclose(got[b, h, :, 5], want[:, 5], rtol=2e-4, atol=1e-4)
            # the four contributions add up to the row-sum error on the GPU side as well
            np.testing.assert_allclose(got[b, h, :, 1:5].sum(axis=1), got[b, h, :, 0] - 1.0, atol=2e-5)
    return got


@pytest.mark.parametrize("uos", [True, False])
def test_tiny_matches_oracle(uos):
    got = check(si.CONFIGS["tiny"], uos)
    assert got[..., 0].mean() < 1.0                 # flat rows lose mass (panel A)


@pytest.mark.parametrize("nq,nkv", [(128, 128), (1, 1), (77, 40), (300, 1000), (130, 3000)])
def test_ragged_shapes(nq, nkv):
    check(si.custom_config("r", 1, 2, nq, nkv, 500 + nq + nkv), True)


def test_structured_and_rotated():
    cfg = si.custom_config("s", 1, 2, 256, 1536, 43, "outlier")
    check(cfg, True, atol=2e-2)                     # peaked rows: single elements carry percent-level mass
    check(cfg, False, atol=2e-2, skip_onehot=True)
    check(si.custom_config("h", 1, 2, 256, 1024, 44, "wan"), True, rotate=True, atol=2e-2)


def test_argument_errors():
    import paper_2607_24377_b200 as mx
    x = torch.zeros((1, 1, 128, 128), dtype=torch.bfloat16, device="cuda")
    out = torch.empty((1, 1, 128, 6), dtype=torch.float32, device="cuda")
    ws = torch.empty(mx.forward_workspace_bytes(1, 1, 128, 128, 128), dtype=torch.uint8, device="cuda")
    with pytest.raises(mx.MxAttnError) as e:
        mx.rowsum_diagnostic(x, x, out, 1, 1, 128, 128, 128, 0.1, mx.FLAG_PNQ, ws)
    assert e.value.code == -1
    with pytest.raises(mx.MxAttnError) as e:
        mx.rowsum_diagnostic(x, x, out, 1, 1, 128, 128, 64, 0.1, 0, ws)
    assert e.value.code == -2
    with pytest.raises(mx.MxAttnError) as e:
        mx.rowsum_diagnostic(x, x, out, 1, 1, 128, 128, 128, 0.1, 0, ws[:1024])
    assert e.value.code == -4
