"""mxattn_forward_static -- the forward pass for callers that cannot allocate device memory.

Some users of the library run where cudaMalloc is not available to them (a host framework with a
fully pre-planned device memory, a plugin that may not allocate after start-up, a latency-critical
loop).  For them the library carries its own fixed scratch array; this test checks that the
entry point built on it gives the same output as the ordinary workspace entry point, twice in a
row (the second call finds the first call's leftovers in the shared array and must not be
disturbed by them), that the output also agrees with the CPU oracle, that the amount of free device
memory is the same before and after a call (the property the entry point exists for), and that an
oversized problem is refused cleanly.

Collected last on purpose: a run that stops at the first failure has then already run every
other test.
"""
import numpy as np
import pytest
import torch

import synth_inputs as si
from oracle import attention
from tests import util

pytestmark = pytest.mark.gpu


def _pair(cfg, flags):
    import paper_2607_24377_b200 as mx
    q, k, v = si.make_all(cfg)
    dq, dk, dv = util.to_dev_bf16(q), util.to_dev_bf16(k), util.to_dev_bf16(v)
    shape = (cfg.B, cfg.H, cfg.Nq, cfg.d)
    want = torch.zeros(shape, dtype=torch.float32, device="cuda")
    ws = torch.empty(mx.forward_workspace_bytes(cfg.B, cfg.H, cfg.Nq, cfg.Nkv, cfg.d), dtype=torch.uint8, device="cuda")
    mx.forward_ws(dq, dk, dv, want, cfg.B, cfg.H, cfg.Nq, cfg.Nkv, cfg.d, cfg.softmax_scale, flags, ws)
    assert mx.device_status(ws) == 0
    got = torch.full(shape, float("nan"), dtype=torch.float32, device="cuda")
    mx.forward_static(dq, dk, dv, got, cfg.B, cfg.H, cfg.Nq, cfg.Nkv, cfg.d, cfg.softmax_scale, flags)
    torch.cuda.synchronize()
    return got.double().cpu().numpy(), want.double().cpu().numpy()


def test_static_scratch_forward_matches_workspace_forward_twice():
    import paper_2607_24377_b200 as mx
    flags = mx.FLAG_UOS | mx.FLAG_PNQ | mx.FLAG_OUT_FP32
    # first call: larger problem, so the second (smaller, ragged) one runs on top of its leftovers
    for cfg in (si.custom_config("na1", 1, 3, 640, 1296, 91), si.custom_config("na2", 1, 2, 300, 1000, 92)):
        got, want = _pair(cfg, flags)
        assert np.isfinite(got).all()
        rel = np.linalg.norm(got - want) / np.linalg.norm(want)
        assert rel <= 1e-3 and np.abs(got - want).max() <= 4e-3, rel      # the parity tolerance of the other tests
        assert np.array_equal(got, want)                                   # and in fact the same kernels, same bits
        # ... and against the oracle directly, not only against the sibling entry point
        q, k, v = si.make_all(cfg)
        f = util.bits_to_f64
        ref = attention.forward(f(q), f(k), f(v), cfg.softmax_scale, True, True)
        rel = np.linalg.norm(got - ref) / np.linalg.norm(ref)
        assert rel <= 1e-3 and np.abs(got - ref).max() <= 4e-3, rel


def test_static_scratch_forward_leaves_free_device_memory_unchanged():
    """A caller that may not allocate must not be made to allocate behind its back: the driver's count of free
    device memory is the same before and after a call (taken after a first call, which loads the kernels and looks
    up the array's address once)."""
    import paper_2607_24377_b200 as mx
    cfg = si.custom_config("na3", 1, 2, 300, 1000, 93)
    q, k, v = si.make_all(cfg)
    dq, dk, dv = util.to_dev_bf16(q), util.to_dev_bf16(k), util.to_dev_bf16(v)
    out = torch.zeros((cfg.B, cfg.H, cfg.Nq, cfg.d), dtype=torch.float32, device="cuda")
    flags = mx.FLAG_UOS | mx.FLAG_PNQ | mx.FLAG_OUT_FP32
    call = lambda: mx.forward_static(dq, dk, dv, out, cfg.B, cfg.H, cfg.Nq, cfg.Nkv, cfg.d, cfg.softmax_scale, flags)
    call(); torch.cuda.synchronize()
    unchanged = False
    for _ in range(3):                       # another process on the device may move the figure: one quiet pair is enough
        free_before = torch.cuda.mem_get_info()[0]
        call(); torch.cuda.synchronize()
        free_after = torch.cuda.mem_get_info()[0]
        if free_after == free_before:
            unchanged = True
            break
    assert unchanged, (free_before, free_after)
    assert bool(torch.isfinite(out).all())


def test_static_scratch_refuses_problems_beyond_its_size():
    import paper_2607_24377_b200 as mx
    cfg = si.CONFIGS["wan22"]
    assert mx.forward_workspace_bytes(cfg.B, cfg.H, cfg.Nq, cfg.Nkv, cfg.d) > mx.binding.STATIC_SCRATCH_BYTES
    x = torch.zeros(16, dtype=torch.bfloat16, device="cuda")               # never touched: the call must refuse first
    with pytest.raises(mx.MxAttnError) as ei:
        mx.forward_static(x, x, x, x, cfg.B, cfg.H, cfg.Nq, cfg.Nkv, cfg.d, cfg.softmax_scale, mx.FLAG_UOS | mx.FLAG_PNQ)
    assert ei.value.code == -7 and "scratch" in str(ei.value)
