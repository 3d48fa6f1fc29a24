"""Parity of the NVFP4 variant of the fused attention forward (the paper's Section 5.2 baseline "NVFP4": the same
loop with Q, K, V and the softmax tile in NVFP4) with the oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import synth_inputs as si
from oracle import attention
from tests import util

pytestmark = pytest.mark.gpu

REL_L2_TOL = 1e-3
MAX_ABS_TOL = 4e-3


def run(cfg, q, k, v, pnq, f32=True):
    import paper_2607_24377_b200 as mx
    dq, dk, dv = util.to_dev_bf16(q), util.to_dev_bf16(k), util.to_dev_bf16(v)
    g_out = util.guarded((cfg.B, cfg.H, cfg.Nq, cfg.d), torch.float32 if f32 else torch.bfloat16, float("nan"))
    g_ws = util.guarded(mx.forward_nvfp4_workspace_bytes(cfg.B, cfg.H, cfg.Nq, cfg.Nkv, cfg.d), torch.uint8)
    flags = (mx.FLAG_PNQ if pnq else 0) | (mx.FLAG_OUT_FP32 if f32 else 0)
    mx.forward_nvfp4(dq, dk, dv, g_out.t, cfg.B, cfg.H, cfg.Nq, cfg.Nkv, cfg.d, cfg.softmax_scale, flags, g_ws.t)
    assert mx.device_status(g_ws.t) == 0
    assert mx.last_launch_count() == 7
    g_out.check(); g_ws.check()
    return g_out.t.clone()


def oracle_out(cfg, q, k, v, pnq):
    f = util.bits_to_f64
    return attention.forward(f(q), f(k), f(v), cfg.softmax_scale, True, pnq, fmt="nvfp4")


def check(got, want):
    got = got.double().cpu().numpy()
    assert np.isfinite(got).all()
    rel = np.linalg.norm(got - want) / np.linalg.norm(want)
    mab = np.abs(got - want).max()
    assert rel <= REL_L2_TOL and mab <= MAX_ABS_TOL, (rel, mab)


@pytest.mark.parametrize("pnq", [False, True])
def test_tiny_config(pnq):
    cfg = si.CONFIGS["tiny"]
    q, k, v = si.make_all(cfg)
    check(run(cfg, q, k, v, pnq), oracle_out(cfg, q, k, v, pnq))


@pytest.mark.parametrize("nq,nkv", [(128, 128), (1, 1), (77, 40), (300, 1000), (256, 200), (640, 1296), (130, 3000)])
def test_ragged_shapes(nq, nkv):
    cfg = si.custom_config("nr", 1, 3, nq, nkv, 131 + nq + nkv)
    q, k, v = si.make_all(cfg)
    check(run(cfg, q, k, v, False), oracle_out(cfg, q, k, v, False))
    check(run(cfg, q, k, v, True), oracle_out(cfg, q, k, v, True))


@pytest.mark.parametrize("recipe", ["outlier", "wan", "hunyuan"])
def test_structured_inputs(recipe):
    cfg = si.custom_config("ns", 2, 2, 384, 1536, 141, recipe)
    q, k, v = si.make_all(cfg)
    for pnq in (False, True):
        check(run(cfg, q, k, v, pnq), oracle_out(cfg, q, k, v, pnq))


def test_bf16_output_is_the_rounded_fp32_output():
    cfg = si.custom_config("nb", 2, 2, 300, 700, 151)
    q, k, v = si.make_all(cfg)
    o32 = run(cfg, q, k, v, False, f32=True)
    o16 = run(cfg, q, k, v, False, f32=False)
    assert torch.equal(o32.to(torch.bfloat16), o16)


def test_unit_values_give_unit_rows_under_pnq_only():
    # V = 1 everywhere: with the row sum taken from the quantized probabilities the output is V-hat's single value in
    # every row; the direct placement divides by a different sum (no oracle needed for this property)
    cfg = si.custom_config("nu", 1, 2, 256, 1024, 161)
    q, k, v = si.make_all(cfg)
    v[:] = si.f32_to_bf16_bits(np.ones(v.shape, np.float32))
    o = run(cfg, q, k, v, True).double().cpu().numpy()
    assert np.abs(o - 1.0).max() < 1e-5
    o = run(cfg, q, k, v, False).double().cpu().numpy()
    assert np.abs(o - 1.0).max() > 1e-4


def test_full_size_outlier_config_sampled_rows():
    import paper_2607_24377_b200 as mx
    cfg = si.CONFIGS["outlier"]
    q, k, v = si.make_all(cfg)
    out = run(cfg, q, k, v, False)
    f = util.bits_to_f64
    num = den = worst = 0.0
    for h in (0, 7, 15, 23):
        rows = np.sort(np.random.default_rng([4343, h]).choice(cfg.Nq, 16, replace=False))
        want = attention.forward_head(f(q[0, h]), f(k[0, h]), f(v[0, h]), cfg.softmax_scale, True, False, rows=rows, fmt="nvfp4")
        got = out[0, h][torch.from_numpy(rows).cuda()].double().cpu().numpy()
        num += float(((got - want) ** 2).sum()); den += float((want ** 2).sum())
        worst = max(worst, float(np.abs(got - want).max()))
    assert (num / den) ** 0.5 <= REL_L2_TOL and worst <= MAX_ABS_TOL


def test_argument_errors():
    import paper_2607_24377_b200 as mx
    L = mx.lib()
    assert L.mxattn_forward_nvfp4(16, 16, 16, 16, 1, 2, 128, 128, 128, 0.1, 1, 16, 1 << 40, None) == -1     # UOS is no flag of it
    assert L.mxattn_forward_nvfp4(16, 16, 16, 16, 1, 2, 128, 128, 64, 0.1, 2, 16, 1 << 40, None) == -2
    assert L.mxattn_forward_nvfp4(16, 16, 16, 16, 1, 2, 128, 128, 128, 0.1, 2, 16, 1024, None) == -4
    assert mx.forward_nvfp4_workspace_bytes(1, 2, 1024, 1024, 128) > mx.forward_workspace_bytes(1, 2, 1024, 1024, 128)
