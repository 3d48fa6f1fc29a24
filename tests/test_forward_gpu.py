"""Parity of the fused CUDA attention forward with the oracle (Algorithm 2), through the C ABI."""
import math

import numpy as np
import pytest
import torch

import synth_inputs as si
from oracle import attention
from tests import util

pytestmark = pytest.mark.gpu

REL_L2_TOL = 1e-3      # the tolerance the benchmark spec states for the fp32 output
MAX_ABS_TOL = 4e-3


def run_forward(cfg, q, k, v, uos, pnq, f32=True, rotate=False):
    import paper_2607_24377_b200 as mx
    dq, dk, dv = util.to_dev_bf16(q), util.to_dev_bf16(k), util.to_dev_bf16(v)
    flags = (mx.FLAG_UOS if uos else 0) | (mx.FLAG_PNQ if pnq else 0) | (mx.FLAG_OUT_FP32 if f32 else 0) | \
            (mx.FLAG_HADAMARD if rotate else 0)
    # output and workspace sit between canary bands: a write outside either fails the test
    g_out = util.guarded((cfg.B, cfg.H, cfg.Nq, cfg.d), torch.float32 if f32 else torch.bfloat16, float("nan"))
    g_ws = util.guarded(mx.forward_workspace_bytes(cfg.B, cfg.H, cfg.Nq, cfg.Nkv, cfg.d), torch.uint8)
    out, ws = g_out.t, g_ws.t
    mx.forward_ws(dq, dk, dv, out, cfg.B, cfg.H, cfg.Nq, cfg.Nkv, cfg.d, cfg.softmax_scale, flags, ws)
    assert mx.device_status(ws) == 0
    assert mx.last_launch_count() == 4
    g_out.check(); g_ws.check()
    return out.clone()


def oracle_out(cfg, q, k, v, uos, pnq, rotate=False):
    f = util.bits_to_f64
    return attention.forward(f(q), f(k), f(v), cfg.softmax_scale, uos, pnq, rotate=rotate)


def check(got, want):
    got = got.double().cpu().numpy()
    assert np.isfinite(got).all()
    rel = np.linalg.norm(got - want) / np.linalg.norm(want)
    mx_abs = np.abs(got - want).max()
    assert rel <= REL_L2_TOL and mx_abs <= MAX_ABS_TOL, (rel, mx_abs)
    return rel, mx_abs


@pytest.mark.parametrize("uos,pnq", [(True, True), (True, False), (False, False), (False, True)])
def test_tiny_config_all_variants(uos, pnq):
    cfg = si.CONFIGS["tiny"]
    q, k, v = si.make_all(cfg)
    check(run_forward(cfg, q, k, v, uos, pnq), oracle_out(cfg, q, k, v, uos, pnq))


@pytest.mark.parametrize("nq,nkv", [(128, 128), (1, 1), (77, 40), (300, 1000), (256, 200), (640, 1296), (130, 3000)])
def test_ragged_shapes(nq, nkv):
    cfg = si.custom_config("r", 1, 3, nq, nkv, 31 + nq + nkv)
    q, k, v = si.make_all(cfg)
    check(run_forward(cfg, q, k, v, True, True), oracle_out(cfg, q, k, v, True, True))


# More work items (head x pair of query tiles) than the device has SMs and a short key/value sequence: the launch
# uses the variant of the kernel in which one CTA per SM walks several items.  600 items give every CTA four or five
# of them, so the double-buffered Q tiles and every barrier parity wrap at least once.
@pytest.mark.parametrize("nkv,uos,pnq", [(100, True, True), (300, True, True), (300, False, False), (896, True, True),
                                         (2500, True, False)])
def test_many_short_items_per_cta(nkv, uos, pnq):
    cfg = si.custom_config("p", 4, 30, 1100, nkv, 77 + nkv)
    q, k, v = si.make_all(cfg)
    check(run_forward(cfg, q, k, v, uos, pnq), oracle_out(cfg, q, k, v, uos, pnq))


@pytest.mark.parametrize("uos,pnq", [(True, True), (True, False)])
def test_item_walking_variant_is_bit_identical_to_one_item_per_cta(uos, pnq):
    """The same head replicated 640 times (walked, several items per CTA) against a single copy of it (5 items on 5
    CTAs): the arithmetic of a work item does not depend on which variant ran it."""
    one = si.custom_config("p1", 1, 1, 1100, 700, 5)
    q, k, v = si.make_all(one)
    want = run_forward(one, q, k, v, uos, pnq)
    many = si.custom_config("pm", 8, 80, 1100, 700, 5)
    rep = lambda x: np.ascontiguousarray(np.broadcast_to(x, (many.B, many.H) + x.shape[2:]))
    got = run_forward(many, rep(q), rep(k), rep(v), uos, pnq)
    assert torch.equal(got, want.expand_as(got))


@pytest.mark.parametrize("recipe", ["outlier", "wan", "hunyuan"])
def test_structured_inputs_small(recipe):
    cfg = si.custom_config("s", 2, 2, 384, 1536, 41, recipe)
    q, k, v = si.make_all(cfg)
    for uos, pnq in ((True, True), (False, False)):
        check(run_forward(cfg, q, k, v, uos, pnq), oracle_out(cfg, q, k, v, uos, pnq))


def test_bf16_output_is_rounded_fp32_output():
    cfg = si.custom_config("b", 1, 2, 256, 512, 51)
    q, k, v = si.make_all(cfg)
    o32 = run_forward(cfg, q, k, v, True, True, f32=True)
    o16 = run_forward(cfg, q, k, v, True, True, f32=False)
    assert torch.equal(o32.to(torch.bfloat16), o16)


# The bf16 output leaves through shared-memory boxes of 32 rows and tensor copies that clip at Nq; the fp32 output is
# stored from registers.  Ragged query counts (a box that ends, or lies entirely, beyond Nq; Nq smaller than a box),
# several heads (a row written past Nq would land in the next head), and the item-walking variant (last case).
@pytest.mark.parametrize("B,H,nq,nkv", [(1, 3, 1, 1), (1, 3, 31, 200), (1, 3, 77, 40), (1, 3, 130, 3000), (2, 2, 300, 1000),
                                        (1, 5, 257, 129), (4, 30, 1100, 300)])
def test_bf16_output_on_ragged_shapes(B, H, nq, nkv):
    cfg = si.custom_config("br", B, H, nq, nkv, 91 + nq)
    q, k, v = si.make_all(cfg)
    o32 = run_forward(cfg, q, k, v, True, True, f32=True)
    o16 = run_forward(cfg, q, k, v, True, True, f32=False)
    assert torch.equal(o32.to(torch.bfloat16), o16)


@pytest.mark.parametrize("uos,pnq", [(True, False), (False, True), (False, False)])
def test_bf16_output_of_the_other_variants_in_the_item_walking_kernel(uos, pnq):
    cfg = si.custom_config("bv", 3, 60, 520, 700, 17)         # 900 work items of 6 KV tiles, ragged query tail
    q, k, v = si.make_all(cfg)
    o32 = run_forward(cfg, q, k, v, uos, pnq, f32=True)
    o16 = run_forward(cfg, q, k, v, uos, pnq, f32=False)
    assert torch.equal(o32.to(torch.bfloat16), o16)
    sample = si.custom_config("bv1", 1, 2, 520, 700, 17)       # the first two heads against the oracle
    check(o32[:1, :2], oracle_out(sample, q[:1, :2], k[:1, :2], v[:1, :2], uos, pnq))


def test_constant_v_gives_exactly_normalized_rows_under_pnq():
    # Proposition 1 on the GPU, no oracle involved: V == 1 -> O == 1 under PNQ, != 1 under the direct placement
    cfg = si.custom_config("c", 1, 2, 256, 1024, 61)
    q, k, v = si.make_all(cfg)
    v[:] = si.f32_to_bf16_bits(np.ones(1, np.float32))[0]
    o = run_forward(cfg, q, k, v, True, True).cpu().numpy()
    assert np.abs(o - 1.0).max() < 1e-6
    o = run_forward(cfg, q, k, v, True, False).cpu().numpy()
    assert np.abs(o - 1.0).max() > 1e-3


def test_prequantized_entry_equals_full_forward():
    import paper_2607_24377_b200 as mx
    cfg = si.custom_config("p", 1, 2, 300, 700, 71)
    q, k, v = si.make_all(cfg)
    full = run_forward(cfg, q, k, v, True, True)
    bh, qt, kt = cfg.B * cfg.H, -(-cfg.Nq // 128), -(-cfg.Nkv // 128)
    bufs = []
    for x, n, nt, axis in ((q, cfg.Nq, qt, 1), (k, cfg.Nkv, kt, 1), (v, cfg.Nkv, kt, 0)):
        codes = torch.empty((bh, nt, 8192), dtype=torch.uint8, device="cuda")
        scales = torch.empty((bh, nt, 512), dtype=torch.uint8, device="cuda")
        mx.quantize_mxfp4_batched(util.to_dev_bf16(x), codes, scales, bh, n, 128, axis, mx.MODE_UOS, mx.LAYOUT_TILE)
        bufs += [codes, scales]
    out = torch.zeros((cfg.B, cfg.H, cfg.Nq, 128), dtype=torch.float32, device="cuda")
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    mx.forward_prequantized(*bufs, out, cfg.B, cfg.H, cfg.Nq, cfg.Nkv, 128, cfg.softmax_scale,
                            mx.FLAG_UOS | mx.FLAG_PNQ | mx.FLAG_OUT_FP32, status)
    torch.cuda.synchronize()
    assert int(status[0]) == 0
    assert torch.equal(out, full)


@pytest.mark.parametrize("B,H", [(1, 2), (1, 13), (2, 7)])
def test_host_buffer_entry_point(B, H):
    # 2 heads: one head per pipeline stage; 13 and 14 heads of a single query-tile pair: several heads per stage
    # (a stage should fill the SMs), with a shorter last stage
    import paper_2607_24377_b200 as mx
    cfg = si.custom_config("h", B, H, 256, 512, 81)
    q, k, v = si.make_all(cfg)
    want = run_forward(cfg, q, k, v, True, True).cpu()
    hq, hk, hv = (torch.from_numpy(x.view(np.int16)).pin_memory() for x in (q, k, v))
    ho = torch.empty((cfg.B, cfg.H, cfg.Nq, 128), dtype=torch.float32).pin_memory()
    flags = mx.FLAG_UOS | mx.FLAG_PNQ | mx.FLAG_OUT_FP32
    arena = torch.empty(mx.forward_host_arena_bytes(cfg.B, cfg.H, cfg.Nq, cfg.Nkv, 128, flags), dtype=torch.uint8, device="cuda")
    mx.forward_host(hq, hk, hv, ho, cfg.B, cfg.H, cfg.Nq, cfg.Nkv, 128, cfg.softmax_scale, flags, arena)
    assert torch.equal(ho, want)
    assert mx.last_launch_count() % 4 == 0 and mx.last_launch_count() <= 4 * B * H
    if B * H >= 12:
        assert mx.last_launch_count() < 4 * B * H          # heads were grouped into stages


@pytest.mark.parametrize("recipe", ["iid", "outlier", "wan"])
def test_full_algorithm_with_hadamard_rotation(recipe):
    # Algorithm 2 complete: lines 1-2 (rotation of Q and K) fused into the quantize launches
    cfg = si.custom_config("rot", 1, 2, 300, 1000, 91, recipe)
    q, k, v = si.make_all(cfg)
    got = run_forward(cfg, q, k, v, True, True, rotate=True)
    want = oracle_out(cfg, q, k, v, True, True, rotate=True)
    check(got, want)
    if recipe != "iid":     # and it is the better approximation of float64 dense attention on outlier data
        f = util.bits_to_f64
        dense = np.stack([attention.dense_attention_head(f(q[0, h]), f(k[0, h]), f(v[0, h]), cfg.softmax_scale) for h in range(2)])[None]
        plain = run_forward(cfg, q, k, v, True, True).double().cpu().numpy()
        e_rot = np.linalg.norm(got.double().cpu().numpy() - dense) / np.linalg.norm(dense)
        e_plain = np.linalg.norm(plain - dense) / np.linalg.norm(dense)
        assert e_rot < e_plain


@pytest.mark.parametrize("nq,nkv", [(1024, 1024), (300, 1000), (77, 40), (640, 1296)])
def test_bf16_variant_of_the_kernel(nq, nkv):
    # the unquantized reference point: same recurrence, bf16 operands, P rounded to bf16, l from fp32 P
    import paper_2607_24377_b200 as mx
    cfg = si.custom_config("bf", 1, 2, nq, nkv, 300 + nq)
    q, k, v = si.make_all(cfg)
    out = torch.full((1, 2, nq, 128), float("nan"), dtype=torch.float32, device="cuda")
    ws = torch.empty(mx.forward_bf16_workspace_bytes(1, 2, nq, nkv, 128), dtype=torch.uint8, device="cuda")
    mx.forward_bf16(util.to_dev_bf16(q), util.to_dev_bf16(k), util.to_dev_bf16(v), out, 1, 2, nq, nkv, 128,
                    cfg.softmax_scale, mx.FLAG_OUT_FP32, ws)
    assert mx.device_status(ws) == 0
    f = util.bits_to_f64
    want = np.stack([attention.forward_head_bf16(f(q[0, h]), f(k[0, h]), f(v[0, h]), cfg.softmax_scale) for h in range(2)])[None]
    check(out, want)
    # and it is close to float64 dense attention (bf16 rounding of P only)
    dense = np.stack([attention.dense_attention_head(f(q[0, h]), f(k[0, h]), f(v[0, h]), cfg.softmax_scale) for h in range(2)])[None]
    got = out.double().cpu().numpy()
    assert np.linalg.norm(got - dense) / np.linalg.norm(dense) < 5e-3


def test_bounded_wait_gives_up_and_reports_without_disturbing_the_device():
    # failure detection without a fault: a wait that nothing satisfies runs out after a short limit,
    # records its code, the kernel ends normally and the next forward on the same context is correct
    import paper_2607_24377_b200 as mx
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    mx.selftest_bounded_wait(status, 2_000_000)          # about a millisecond of SM cycles
    t1.record(); torch.cuda.synchronize()
    assert int(status[0]) == 77
    assert t0.elapsed_time(t1) < 200.0
    cfg = si.custom_config("after", 1, 1, 130, 260, 5)
    q, k, v = si.make_all(cfg)
    check(run_forward(cfg, q, k, v, True, True), oracle_out(cfg, q, k, v, True, True))
    with pytest.raises(mx.MxAttnError):
        mx.selftest_bounded_wait(status, 0)


def test_paired_warps_stay_in_step_when_one_gives_up():
    # the two softmax warps of a row pair meet at a named barrier in every tile; a warp that gives up keeps the
    # remaining appointments so that its partner is never stranded.  A dedicated kernel makes one warp's short-limit
    # wait run out (no fault involved) and counts the meetings the healthy warp gets through.
    import paper_2607_24377_b200 as mx
    for meetings in (1, 7, 600):
        status = torch.zeros(4, dtype=torch.int32, device="cuda")
        t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
        t0.record()
        mx.selftest_pair_abandon(status, 2_000_000, meetings)
        t1.record(); torch.cuda.synchronize()
        assert status.tolist()[:2] == [77, meetings]
        assert t0.elapsed_time(t1) < 200.0
    cfg = si.custom_config("after2", 1, 1, 130, 260, 6)
    q, k, v = si.make_all(cfg)
    check(run_forward(cfg, q, k, v, True, False), oracle_out(cfg, q, k, v, True, False))


@pytest.mark.parametrize("uos,pnq", [(True, True), (False, False)])
def test_registered_workspace_entry_point(uos, pnq):
    """The two-call form of the interface: mxattn_set_workspace registers caller-owned scratch, mxattn_forward (the
    signature without a workspace argument) uses it.  Compared with the oracle like every other forward."""
    import paper_2607_24377_b200 as mx
    cfg = si.custom_config("reg", 1, 3, 300, 1000, 71)
    q, k, v = si.make_all(cfg)
    dq, dk, dv = util.to_dev_bf16(q), util.to_dev_bf16(k), util.to_dev_bf16(v)
    g_out = util.guarded((cfg.B, cfg.H, cfg.Nq, cfg.d), torch.float32, float("nan"))
    g_ws = util.guarded(mx.forward_workspace_bytes(cfg.B, cfg.H, cfg.Nq, cfg.Nkv, cfg.d), torch.uint8)
    flags = (mx.FLAG_UOS if uos else 0) | (mx.FLAG_PNQ if pnq else 0) | mx.FLAG_OUT_FP32
    mx.set_workspace(g_ws.t)
    try:
        mx.forward(dq, dk, dv, g_out.t, cfg.B, cfg.H, cfg.Nq, cfg.Nkv, cfg.d, cfg.softmax_scale, flags)
        assert mx.device_status(g_ws.t) == 0 and mx.last_launch_count() == 4
        g_out.check(); g_ws.check()
        check(g_out.t, oracle_out(cfg, q, k, v, uos, pnq))
        # a registered workspace that is too small is refused before anything is launched
        mx.set_workspace(g_ws.t, nbytes=1024)
        with pytest.raises(mx.MxAttnError) as ei:
            mx.forward(dq, dk, dv, g_out.t, cfg.B, cfg.H, cfg.Nq, cfg.Nkv, cfg.d, cfg.softmax_scale, flags)
        assert ei.value.code == -4
    finally:
        mx.set_workspace(None)


@pytest.mark.parametrize("B,H,nq,nkv", [(1, 3, 300, 1000), (4, 60, 520, 700)])
def test_cycle_profile_build_gives_the_same_output_and_fills_its_counters(B, H, nq, nkv):
    """The kernel compiled with cycle counters (a performance-analysis aid) computes exactly what the timed kernel
    computes; its counters account for every tile.  Second case: the item-walking variant."""
    import paper_2607_24377_b200 as mx
    cfg = si.custom_config("prof", B, H, nq, nkv, 81)
    q, k, v = si.make_all(cfg)
    dq, dk, dv = util.to_dev_bf16(q), util.to_dev_bf16(k), util.to_dev_bf16(v)
    flags = mx.FLAG_UOS | mx.FLAG_PNQ
    ws = torch.empty(mx.forward_workspace_bytes(B, H, nq, nkv, 128), dtype=torch.uint8, device="cuda")
    want = torch.empty((B, H, nq, 128), dtype=torch.bfloat16, device="cuda")
    mx.forward_ws(dq, dk, dv, want, B, H, nq, nkv, 128, cfg.softmax_scale, flags, ws)
    g_out = util.guarded((B, H, nq, 128), torch.bfloat16, float("nan"))
    g_prof = util.guarded((mx.forward_cycle_profile_bytes(B, H, nq, nkv, 128) // 8,), torch.int64, 0)
    mx.forward_cycle_profile(dq, dk, dv, g_out.t, B, H, nq, nkv, 128, cfg.softmax_scale, flags, ws, g_prof.t)
    assert mx.device_status(ws) == 0
    g_out.check(); g_prof.check()
    assert torch.equal(g_out.t, want)
    p = g_prof.t.view(-1, 18, 16).cpu().numpy()
    ran = p[p[:, 17, 9] > 0]
    items = B * H * -(-(-(-nq // 128)) // 2)
    tiles = -(-nkv // 128)
    assert ran[:, 17, 9].sum() == items * tiles                        # the issuer saw every tile of every item
    assert (ran[:, :16, 9].sum(axis=0) == items * tiles).all()         # and so did each of the 16 softmax warps
    assert (ran[:, :16, 6] > 0).all() and (ran[:, 17, 8] > 0).all()
