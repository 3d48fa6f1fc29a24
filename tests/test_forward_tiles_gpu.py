"""Tile-level parity of the softmax loop (Algorithm 2 lines 10-14) through the debug-dump entry point:
the quantized probabilities P-hat are compared with the oracle's value for value, tile by tile."""
import numpy as np
import pytest
import torch

import synth_inputs as si
from oracle import attention
from tests import util

pytestmark = pytest.mark.gpu


def run_dump(cfg, q, k, v, uos, pnq):
    import paper_2607_24377_b200 as mx
    flags = (mx.FLAG_UOS if uos else 0) | (mx.FLAG_PNQ if pnq else 0) | mx.FLAG_OUT_FP32
    out = torch.empty((cfg.B, cfg.H, cfg.Nq, cfg.d), dtype=torch.float32, device="cuda")
    ws = torch.empty(mx.forward_workspace_bytes(cfg.B, cfg.H, cfg.Nq, cfg.Nkv, cfg.d), dtype=torch.uint8, device="cuda")
    dump = torch.zeros(mx.forward_debug_dump_bytes(cfg.B, cfg.H, cfg.Nq, cfg.Nkv, cfg.d), dtype=torch.uint8, device="cuda")
    mx.forward_debug_dump(util.to_dev_bf16(q), util.to_dev_bf16(k), util.to_dev_bf16(v), out, cfg.B, cfg.H, cfg.Nq,
                          cfg.Nkv, cfg.d, cfg.softmax_scale, flags, ws, dump)
    assert mx.device_status(ws) == 0
    return out.cpu().numpy(), dump.cpu().numpy()


def check_tiles(cfg, q, k, v, uos, pnq):
    out, dump = run_dump(cfg, q, k, v, uos, pnq)
    qt, kt = -(-cfg.Nq // 128), -(-cfg.Nkv // 128)
    rec = 8192 + 512 + 512
    tiles = dump[:cfg.B * cfg.H * qt * kt * rec].reshape(cfg.B * cfg.H, qt, kt, rec)
    lsum = dump[cfg.B * cfg.H * qt * kt * rec:].view(np.float32).reshape(cfg.B * cfg.H, qt * 128)
    f = util.bits_to_f64
    n_elem = n_diff = 0
    for bh in range(cfg.B * cfg.H):
        b, h = divmod(bh, cfg.H)
        want, st = attention.forward_head(f(q[b, h]), f(k[b, h]), f(v[b, h]), cfg.softmax_scale, uos, pnq, return_state=True)
        for j in range(kt):
            w = min(128, cfg.Nkv - 128 * j)
            for t in range(qt):
                rows = min(128, cfg.Nq - 128 * t)
                t_rec = tiles[bh, t, j]
                got = util.decode_tile_axis1(t_rec[:8192], t_rec[8192:8704])
                ref = st["p_hat"][j][128 * t:128 * t + rows]
                n_elem += rows * w
                n_diff += int((got[:rows, :w] != ref).sum())
                assert (got[:rows, w:] == 0).all()                       # keys beyond Nkv do not exist
                m_got = t_rec[8704:].view(np.float32)[:rows].astype(np.float64)
                np.testing.assert_allclose(m_got, st["m"][j][128 * t:128 * t + rows], rtol=2e-6, atol=1e-6)
        np.testing.assert_allclose(lsum[bh, :cfg.Nq], st["l"], rtol=2e-5)
        np.testing.assert_allclose(out[b, h], want, rtol=0, atol=4e-3)
    return n_elem, n_diff


@pytest.mark.parametrize("uos,pnq", [(True, True), (False, False), (True, False), (False, True)])
def test_tiny_p_hat_matches_oracle_code_for_code(uos, pnq):
    cfg = si.CONFIGS["tiny"]
    q, k, v = si.make_all(cfg)
    n_elem, n_diff = check_tiles(cfg, q, k, v, uos, pnq)
    # the kernel's exponential (ex2.approx of an fp32 argument) differs from the oracle's correctly rounded
    # exp by ~1e-7 relative, so a value within that distance of an E2M1 rounding boundary or of a UOS
    # exponent boundary may land on the other side: allow a few per million
    assert n_elem == 2 * 1024 * 1024
    assert n_diff <= 8, (n_diff, n_elem)


def test_ragged_p_hat():
    cfg = si.custom_config("r", 1, 2, 300, 1000, 77)
    q, k, v = si.make_all(cfg)
    n_elem, n_diff = check_tiles(cfg, q, k, v, True, True)
    assert n_diff <= 4, (n_diff, n_elem)


def test_outlier_scores_p_hat():
    # With outlier channels the scores reach the hundreds.  The kernel evaluates the exponent as one fp32
    # fma, s*c - (m*c + e), whose constant term is rounded to fp32: an absolute error of |m*c| * 2^-24 in
    # log2 units, i.e. ~1e-5 relative in the exponential at |m*c| ~ 200, against ~1e-7 on Tiny.  More values
    # therefore land on the other side of a rounding boundary; the output stays inside the tolerance.
    cfg = si.custom_config("s", 1, 2, 256, 640, 78, "outlier")
    q, k, v = si.make_all(cfg)
    n_elem, n_diff = check_tiles(cfg, q, k, v, True, True)
    assert n_diff <= n_elem // 2000, (n_diff, n_elem)


def test_debug_dump_argument_errors():
    import paper_2607_24377_b200 as mx
    cfg = si.CONFIGS["tiny"]
    x = torch.zeros((1, 2, 1024, 128), dtype=torch.bfloat16, device="cuda")
    out = torch.empty((1, 2, 1024, 128), dtype=torch.float32, device="cuda")
    ws = torch.empty(mx.forward_workspace_bytes(1, 2, 1024, 1024, 128), dtype=torch.uint8, device="cuda")
    small = torch.empty(1024, dtype=torch.uint8, device="cuda")
    with pytest.raises(mx.MxAttnError) as e:
        mx.forward_debug_dump(x, x, x, out, 1, 2, 1024, 1024, 128, cfg.softmax_scale, mx.FLAG_OUT_FP32 | 3, ws, small)
    assert e.value.code == -4
    big = torch.empty(mx.forward_debug_dump_bytes(1, 2, 1024, 1024, 128), dtype=torch.uint8, device="cuda")
    with pytest.raises(mx.MxAttnError) as e:
        mx.forward_debug_dump(x, x, x, out, 1, 2, 1024, 1024, 128, cfg.softmax_scale, 3, ws, big)     # bf16 output
    assert e.value.code == -1
    assert mx.forward_debug_dump_bytes(1, 40, 75600, 75600, 128) > (1 << 30)
