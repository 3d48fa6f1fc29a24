"""Seeded random shapes, recipes and variants against the oracle: the quantizers bit for bit, the forward variants within
the output tolerance.  The committed shape lists of the other test files pick edge cases by hand; these walk through the
space between them (odd column counts, batches, ragged tails of any length, short and long KV sequences)."""
import numpy as np
import pytest
import torch

import synth_inputs as si
from oracle import attention, mxfp4, nvfp4
from tests import util

pytestmark = pytest.mark.gpu

RULE = {0: mxfp4.OCP, 1: mxfp4.UOS}


def _bits(rng, rows, cols, lo, hi):
    x = rng.standard_normal((rows, cols)).astype(np.float32)
    x *= np.exp2(rng.integers(lo, hi, size=(rows, 1))).astype(np.float32)
    if rng.random() < 0.3:
        x[rng.integers(rows)] = 0.0               # a row of zero blocks
    return si.f32_to_bf16_bits(x)


@pytest.mark.parametrize("seed", [11, 12, 13])
def test_random_quantizer_cases_are_bit_exact(seed):
    import paper_2607_24377_b200 as mx
    rng = np.random.default_rng(seed)
    for _ in range(120):
        fmt = "mx" if rng.random() < 0.6 else "nv"
        axis = int(rng.integers(2)); batch = int(rng.integers(1, 4)); mode = int(rng.integers(2))
        if axis == 1:
            cols = int(rng.choice([32, 64, 96, 128, 160, 256, 480, 1024] if fmt == "mx" else [16, 48, 64, 128, 144, 256, 1024]))
        else:
            cols = int(rng.choice([8, 64, 72, 128, 136, 264]))
        rows = min(int(rng.integers(1, 3000)), 400_000 // cols)
        rp = -(-rows // 128) * 128
        case = (fmt, axis, batch, rows, cols, mode)
        if fmt == "mx":
            bits = np.stack([_bits(rng, rows, cols, -12, 12) for _ in range(batch)])
            x = util.to_dev_bf16(bits)
            shape_c, shape_s = ((batch, rows, cols // 2), (batch, rows, cols // 32)) if axis == 1 else ((batch, cols, rp // 2), (batch, cols, rp // 32))
            gc, gs = util.guarded(shape_c, torch.uint8, 0xAA), util.guarded(shape_s, torch.uint8, 0xAA)
            mx.quantize_mxfp4_batched(x, gc.t, gs.t, batch, rows, cols, axis, mode, mx.LAYOUT_CANONICAL)
            gc.check(); gs.check()
            for b in range(batch):
                wc, ws = mxfp4.quantize_matrix_canonical(util.bits_to_f64(bits[b]), axis, RULE[mode])
                assert np.array_equal(gs.t[b].cpu().numpy(), ws), case
                assert np.array_equal(gc.t[b].cpu().numpy(), wc), case
        else:
            bits = np.stack([_bits(rng, rows, cols, -14, 3) for _ in range(batch)])
            x = util.to_dev_bf16(bits)
            g_amax, g_ts = util.guarded((batch,), torch.float32, float("nan")), util.guarded((batch,), torch.float32, float("nan"))
            mx.tensor_amax(x, g_amax.t, batch, rows, cols)
            shape_c, shape_s = ((batch, rows, cols // 2), (batch, rows, cols // 16)) if axis == 1 else ((batch, cols, rp // 2), (batch, cols, rp // 16))
            gc, gs = util.guarded(shape_c, torch.uint8, 0xAA), util.guarded(shape_s, torch.uint8, 0xAA)
            mx.quantize_nvfp4(x, gc.t, gs.t, g_amax.t, g_ts.t, batch, rows, cols, axis, mx.LAYOUT_CANONICAL)
            for g in (g_amax, g_ts, gc, gs):
                g.check()
            for b in range(batch):
                wc, ws, wt = nvfp4.quantize_matrix_canonical(util.bits_to_f64(bits[b]), axis)
                assert np.array_equal(gs.t[b].cpu().numpy(), ws), case
                assert np.array_equal(gc.t[b].cpu().numpy(), wc), case
                assert np.float32(wt) == g_ts.t[b].cpu().numpy(), case


def _random_problem(rng):
    B = int(rng.integers(1, 3)); H = int(rng.integers(1, 5))
    big = rng.random() < 0.3
    Nq = int(rng.integers(1, 2600 if big else 520)); Nkv = int(rng.integers(1, 400 if big else 1500))
    recipe = ["iid", "outlier", "wan", "hunyuan"][int(rng.integers(4))]
    return si.custom_config("rnd", B, H, Nq, Nkv, int(rng.integers(1 << 30)), recipe)


@pytest.mark.parametrize("seed", [21, 22])
def test_random_forward_cases_mxfp4(seed):
    # the four variants of the MXFP4 kernel (Algorithm 2 lines 3-19), fp32 and bf16 output
    import paper_2607_24377_b200 as mx
    rng = np.random.default_rng(seed)
    f = util.bits_to_f64
    for _ in range(50):
        cfg = _random_problem(rng)
        uos, pnq, bf16_out = bool(rng.integers(2)), bool(rng.integers(2)), bool(rng.integers(2))
        q, k, v = si.make_all(cfg)
        g_out = util.guarded((cfg.B, cfg.H, cfg.Nq, cfg.d), torch.bfloat16 if bf16_out else torch.float32, float("nan"))
        g_ws = util.guarded(mx.forward_workspace_bytes(cfg.B, cfg.H, cfg.Nq, cfg.Nkv, cfg.d), torch.uint8)
        flags = (mx.FLAG_UOS if uos else 0) | (mx.FLAG_PNQ if pnq else 0) | (0 if bf16_out else mx.FLAG_OUT_FP32)
        mx.forward_ws(util.to_dev_bf16(q), util.to_dev_bf16(k), util.to_dev_bf16(v), g_out.t, cfg.B, cfg.H, cfg.Nq, cfg.Nkv, cfg.d,
                      cfg.softmax_scale, flags, g_ws.t)
        assert mx.device_status(g_ws.t) == 0
        g_out.check(); g_ws.check()
        want = attention.forward(f(q), f(k), f(v), cfg.softmax_scale, uos, pnq)
        got = g_out.t.double().cpu().numpy()
        rel = np.linalg.norm(got - want) / np.linalg.norm(want)
        mab = np.abs(got - want).max()
        # bf16 output: the fp32 result rounded to bf16 (relative 2^-9 per element) on top of the kernel's own tolerance
        tol_rel, tol_abs = (5e-3, 4e-2) if bf16_out else (1e-3, 4e-3)
        assert rel <= tol_rel and mab <= tol_abs, (cfg, uos, pnq, bf16_out, rel, mab)


def test_random_forward_cases_nvfp4():
    # The comparison format.  The E4M3 scale of a block of P~ has eight rounding boundaries per octave, and the kernel's fp32
    # scores and ex2.approx put fl32(M 2688 / 6) on the other side of one about once per 1e5 blocks; the block then takes the
    # neighbouring scale and ONE row of the problem moves by more than the element-wise tolerance.  So: relative L2 as
    # everywhere, and at most two rows per case beyond the element-wise tolerance.
    import paper_2607_24377_b200 as mx
    rng = np.random.default_rng(31)
    f = util.bits_to_f64
    for _ in range(50):
        cfg = _random_problem(rng)
        pnq = bool(rng.integers(2))
        q, k, v = si.make_all(cfg)
        g_out = util.guarded((cfg.B, cfg.H, cfg.Nq, cfg.d), torch.float32, float("nan"))
        g_ws = util.guarded(mx.forward_nvfp4_workspace_bytes(cfg.B, cfg.H, cfg.Nq, cfg.Nkv, cfg.d), torch.uint8)
        mx.forward_nvfp4(util.to_dev_bf16(q), util.to_dev_bf16(k), util.to_dev_bf16(v), g_out.t, cfg.B, cfg.H, cfg.Nq, cfg.Nkv, cfg.d,
                         cfg.softmax_scale, (mx.FLAG_PNQ if pnq else 0) | mx.FLAG_OUT_FP32, g_ws.t)
        assert mx.device_status(g_ws.t) == 0
        g_out.check(); g_ws.check()
        want = attention.forward(f(q), f(k), f(v), cfg.softmax_scale, True, pnq, fmt="nvfp4")
        got = g_out.t.double().cpu().numpy()
        assert np.isfinite(got).all()
        rel = np.linalg.norm(got - want) / np.linalg.norm(want)
        rows_off = int((np.abs(got - want).max(axis=-1) > 4e-3).sum())
        assert rel <= 2.5e-3 and rows_off <= 2, (cfg, pnq, rel, rows_off)


def test_random_host_buffer_cases_equal_the_device_path():
    # mxattn_forward_host pipelines stages of one or more heads over several streams: whatever the number of heads,
    # the lengths and the flags, its result is the device path's, bit for bit, also when the arena is used twice in a row
    import paper_2607_24377_b200 as mx
    rng = np.random.default_rng(41)
    for _ in range(30):
        B = int(rng.integers(1, 3)); H = int(rng.integers(1, 41))
        Nq = int(rng.integers(1, 1200)); Nkv = int(rng.integers(1, 1200))
        uos, pnq, rot, f32 = bool(rng.integers(2)), bool(rng.integers(2)), bool(rng.random() < 0.3), bool(rng.integers(2))
        cfg = si.custom_config("rndh", B, H, Nq, Nkv, int(rng.integers(1 << 30)))
        q, k, v = si.make_all(cfg)
        flags = (mx.FLAG_UOS if uos else 0) | (mx.FLAG_PNQ if pnq else 0) | (mx.FLAG_HADAMARD if rot else 0) | (mx.FLAG_OUT_FP32 if f32 else 0)
        dt, bits = (torch.float32, torch.int32) if f32 else (torch.bfloat16, torch.int16)
        out = torch.full((B, H, Nq, 128), float("nan"), dtype=dt, device="cuda")
        ws = torch.empty(mx.forward_workspace_bytes(B, H, Nq, Nkv, 128), dtype=torch.uint8, device="cuda")
        mx.forward_ws(util.to_dev_bf16(q), util.to_dev_bf16(k), util.to_dev_bf16(v), out, B, H, Nq, Nkv, 128, cfg.softmax_scale, flags, ws)
        assert mx.device_status(ws) == 0
        want = out.cpu()
        hq, hk, hv = (torch.from_numpy(x.view(np.int16)).pin_memory() for x in (q, k, v))
        ho = torch.empty((B, H, Nq, 128), dtype=dt).pin_memory()
        arena = torch.empty(mx.forward_host_arena_bytes(B, H, Nq, Nkv, 128, flags), dtype=torch.uint8, device="cuda")
        for _rep in range(2):
            ho.fill_(float("nan"))
            mx.forward_host(hq, hk, hv, ho, B, H, Nq, Nkv, 128, cfg.softmax_scale, flags, arena)
            assert torch.equal(ho.view(bits), want.view(bits)), (B, H, Nq, Nkv, uos, pnq, rot, f32)
