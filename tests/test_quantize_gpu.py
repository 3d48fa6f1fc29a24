"""Bit-exact parity of the CUDA quantizer with the oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import synth_inputs as si
from oracle import mxfp4
from tests import util

pytestmark = pytest.mark.gpu

RULE = {0: mxfp4.OCP, 1: mxfp4.UOS}


def run_gpu(bits, rows, cols, axis, mode):
    import paper_2607_24377_b200 as mx
    x = util.to_dev_bf16(bits)
    # outputs sit between canary bands and are pre-filled, so unwritten bytes and stray writes both show
    if axis == 1:
        gc = util.guarded((rows, cols // 2), torch.uint8, 0xAA)
        gs = util.guarded((rows, cols // 32), torch.uint8, 0xAA)
    else:
        rp = -(-rows // 128) * 128
        gc = util.guarded((cols, rp // 2), torch.uint8, 0xAA)
        gs = util.guarded((cols, rp // 32), torch.uint8, 0xAA)
    mx.quantize_mxfp4(x, gc.t, gs.t, rows, cols, axis, mode)
    gc.check(); gs.check()
    return gc.t.cpu().numpy(), gs.t.cpu().numpy()


def gaussian_bits(rows, cols, seed, spread=True):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((rows, cols)).astype(np.float32)
    if spread:   # vary magnitudes over many binades so every exponent path is hit
        x *= np.exp2(rng.integers(-12, 12, size=(rows, 1))).astype(np.float32)
    return si.f32_to_bf16_bits(x)


@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("rows,cols", [(1, 32), (3, 32), (7, 96), (1024, 128), (1000, 128), (333, 256), (4099, 128), (65, 4096)])
def test_axis1_matches_oracle_bit_exact(rows, cols, mode):
    bits = gaussian_bits(rows, cols, rows * 7 + cols + mode)
    want_c, want_s = mxfp4.quantize_matrix_canonical(util.bits_to_f64(bits), 1, RULE[mode])
    got_c, got_s = run_gpu(bits, rows, cols, 1, mode)
    assert np.array_equal(got_s, want_s)
    assert np.array_equal(got_c, want_c)


@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("rows,cols", [(1, 128), (31, 128), (128, 128), (200, 128), (1024, 128), (1000, 128), (75600 % 4096 + 4096, 128), (300, 64), (260, 264)])
def test_axis0_matches_oracle_bit_exact(rows, cols, mode):
    bits = gaussian_bits(rows, cols, rows * 3 + cols + mode)
    want_c, want_s = mxfp4.quantize_matrix_canonical(util.bits_to_f64(bits), 0, RULE[mode])
    got_c, got_s = run_gpu(bits, rows, cols, 0, mode)
    assert np.array_equal(got_s, want_s)
    assert np.array_equal(got_c, want_c)


@pytest.mark.parametrize("mode", [0, 1])
def test_every_bf16_bit_pattern(mode):
    # all 65536 patterns except Inf/NaN, once alone in a block and once with companions
    pats = np.array([p for p in range(65536) if (p & 0x7F80) != 0x7F80], dtype=np.uint16)
    n = pats.size
    alone = np.zeros((n, 32), np.uint16); alone[:, 5] = pats
    rng = np.random.default_rng(5)
    mixed = pats[rng.integers(0, n, size=(4096, 128))]
    # keep binades close so companions are not all flushed
    mixed = (mixed & 0x807F) | (np.uint16(0x3F00) + (rng.integers(0, 6, size=mixed.shape).astype(np.uint16) << 7))
    for bits, cols in ((alone, 32), (mixed, 128)):
        want_c, want_s = mxfp4.quantize_matrix_canonical(util.bits_to_f64(bits), 1, RULE[mode])
        got_c, got_s = run_gpu(bits, bits.shape[0], cols, 1, mode)
        assert np.array_equal(got_s, want_s)
        assert np.array_equal(got_c, want_c)


def test_special_blocks():
    bits = np.zeros((8, 128), np.uint16)
    bits[1, :] = 0x8000                               # all -0.0 : zero block, sign kept
    bits[2, 0] = 0x0001                               # smallest subnormal
    bits[2, 1] = 0x8040
    bits[3, 3] = 0x7F7F                               # largest finite
    bits[3, 4] = 0xFF7F
    bits[4, :] = si.f32_to_bf16_bits(np.full(128, 7.25, np.float32))      # exact UOS boundary
    bits[5, :] = si.f32_to_bf16_bits(np.full(128, 7.28125, np.float32))   # one bf16 ulp above
    bits[6, :32] = si.f32_to_bf16_bits(np.array([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0, 4.0] * 4, np.float32))  # ties at e = 0
    bits[7, 64:96] = si.f32_to_bf16_bits(np.linspace(-6, 6, 32).astype(np.float32))
    for mode in (0, 1):
        want_c, want_s = mxfp4.quantize_matrix_canonical(util.bits_to_f64(bits), 1, RULE[mode])
        got_c, got_s = run_gpu(bits, 8, 128, 1, mode)
        assert np.array_equal(got_s, want_s), mode
        assert np.array_equal(got_c, want_c), mode
        want_c, want_s = mxfp4.quantize_matrix_canonical(util.bits_to_f64(bits), 0, RULE[mode])
        got_c, got_s = run_gpu(bits, 8, 128, 0, mode)
        assert np.array_equal(got_s, want_s), mode
        assert np.array_equal(got_c, want_c), mode


@pytest.mark.parametrize("axis", [0, 1])
@pytest.mark.parametrize("rows", [128, 1000, 75600 % 1024 + 1024])
def test_tile_layout_is_a_permutation_of_the_canonical_one(axis, rows):
    import paper_2607_24377_b200 as mx
    batch = 3
    bits = np.stack([gaussian_bits(rows, 128, 100 + b + rows) for b in range(batch)])
    x = util.to_dev_bf16(bits)
    nt = -(-rows // 128)
    codes = torch.full((batch, nt, 8192), 0xAA, dtype=torch.uint8, device="cuda")
    scales = torch.full((batch, nt, 512), 0xAA, dtype=torch.uint8, device="cuda")
    mx.quantize_mxfp4_batched(x, codes, scales, batch, rows, 128, axis, mx.MODE_UOS, mx.LAYOUT_TILE)
    torch.cuda.synchronize()
    for b in range(batch):
        want_c, want_s = mxfp4.quantize_matrix_canonical(util.bits_to_f64(bits[b]), axis, mxfp4.UOS)
        tc, ts = (util.canonical_to_tile_axis1 if axis == 1 else util.canonical_to_tile_axis0)(want_c, want_s)
        assert np.array_equal(scales[b].cpu().numpy(), ts)
        assert np.array_equal(codes[b].cpu().numpy(), tc)


def test_batched_canonical_equals_per_matrix_calls():
    import paper_2607_24377_b200 as mx
    batch, rows = 4, 300
    bits = np.stack([gaussian_bits(rows, 128, 200 + b) for b in range(batch)])
    x = util.to_dev_bf16(bits)
    for axis in (0, 1):
        rp = rows if axis == 1 else 384
        shape_c = (batch, rows, 64) if axis == 1 else (batch, 128, rp // 2)
        shape_s = (batch, rows, 4) if axis == 1 else (batch, 128, rp // 32)
        codes = torch.zeros(shape_c, dtype=torch.uint8, device="cuda")
        scales = torch.zeros(shape_s, dtype=torch.uint8, device="cuda")
        mx.quantize_mxfp4_batched(x, codes, scales, batch, rows, 128, axis, mx.MODE_OCP, mx.LAYOUT_CANONICAL)
        torch.cuda.synchronize()
        for b in range(batch):
            want_c, want_s = mxfp4.quantize_matrix_canonical(util.bits_to_f64(bits[b]), axis, mxfp4.OCP)
            assert np.array_equal(codes[b].cpu().numpy(), want_c)
            assert np.array_equal(scales[b].cpu().numpy(), want_s)


def test_power_of_two_scaling_shifts_scale_bytes_only():
    bits = gaussian_bits(512, 128, 9, spread=False)
    x = si.bf16_bits_to_f32(bits)
    c0, s0 = run_gpu(bits, 512, 128, 1, 1)
    c1, s1 = run_gpu(si.f32_to_bf16_bits(x * np.float32(2.0 ** 9)), 512, 128, 1, 1)
    assert np.array_equal(c0, c1) and np.array_equal(s0.astype(np.int32) + 9, s1.astype(np.int32))


def _rotated_gpu(bits, rows, mode, layout_tile=False):
    import paper_2607_24377_b200 as mx
    if layout_tile:
        nt = -(-rows // 128)
        codes = torch.zeros((1, nt, 8192), dtype=torch.uint8, device="cuda"); scales = torch.zeros((1, nt, 512), dtype=torch.uint8, device="cuda")
    else:
        codes = torch.zeros((rows, 64), dtype=torch.uint8, device="cuda"); scales = torch.zeros((rows, 4), dtype=torch.uint8, device="cuda")
    mx.quantize_mxfp4_batched(util.to_dev_bf16(bits), codes, scales, 1, rows, 128, 1, mode | mx.MODE_HADAMARD,
                              mx.LAYOUT_TILE if layout_tile else mx.LAYOUT_CANONICAL)
    torch.cuda.synchronize()
    return codes.cpu().numpy(), scales.cpu().numpy()


# Flip-rate bound of the rotated quantizer against the paper's definition of the rotation (x H_128 / sqrt(128) in
# exact arithmetic, rounded once to fp32).  The kernel evaluates the rotation in fp32 (about 1e-7 relative noise), which can
# move a code or a scale byte only where a rotated value sits that close to a rounding boundary.
ROT_FLIP_BOUND = 1e-5


@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("recipe,rows", [("iid", 1), ("iid", 100), ("iid", 4099), ("outlier", 20000), ("wan", 20000), ("hunyuan", 8192)])
def test_hadamard_rotated_quantization_against_the_plain_definition(recipe, rows, mode):
    # Algorithm 2: rotate (plain definition, the oracle's `hadamard_rotate`), then quantize
    cfg = si.custom_config("rq", 1, 1, rows, rows, 300 + rows + mode, recipe)
    qbits, kbits, _ = si.make_head(cfg, 0, 0)
    for bits in (qbits, kbits):
        x = si.bf16_bits_to_f32(bits)
        want_c, want_s = mxfp4.quantize_matrix_canonical(mxfp4.hadamard_rotate(x).astype(np.float64), 1, RULE[mode])
        got_c, got_s = _rotated_gpu(bits, rows, mode)
        nib = lambda c: np.stack([c & 15, c >> 4], axis=-1)
        code_flips = int((nib(got_c) != nib(want_c)).sum()); scale_flips = int((got_s != want_s).sum())
        n_codes = rows * 128; n_scales = rows * 4
        print(f"rotation flips vs plain definition [{recipe}, rows={rows}, mode={mode}]: codes {code_flips}/{n_codes}, scales {scale_flips}/{n_scales}")
        assert code_flips <= max(1, ROT_FLIP_BOUND * n_codes) and scale_flips <= max(1, ROT_FLIP_BOUND * n_scales)
        if rows < 64:
            assert code_flips == 0 and scale_flips == 0
        # a flipped code is a neighbouring code, a flipped scale byte differs by one
        assert np.all(np.abs(got_s.astype(np.int32) - want_s.astype(np.int32)) <= 1)


@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("batch,rows", [(1, 1), (3, 100), (2, 1024), (1, 4099), (5, 300)])
def test_hadamard_rotated_quantization_tile_layout_is_a_permutation_of_the_canonical_one(batch, rows, mode):
    import paper_2607_24377_b200 as mx
    bits = np.stack([gaussian_bits(rows, 128, 300 + rows + mode + b) for b in range(batch)])
    bits[:, ::5, 7] = si.f32_to_bf16_bits(np.full(bits[:, ::5, 7].shape, 37.5, np.float32))      # a channel outlier
    nt = -(-rows // 128)
    gc = util.guarded((batch, rows, 64), torch.uint8, 0xAA); gs = util.guarded((batch, rows, 4), torch.uint8, 0xAA)
    mx.quantize_mxfp4_batched(util.to_dev_bf16(bits), gc.t, gs.t, batch, rows, 128, 1, mode | mx.MODE_HADAMARD, mx.LAYOUT_CANONICAL)
    tc = util.guarded((batch, nt, 8192), torch.uint8, 0xAA); ts = util.guarded((batch, nt, 512), torch.uint8, 0xAA)
    mx.quantize_mxfp4_batched(util.to_dev_bf16(bits), tc.t, ts.t, batch, rows, 128, 1, mode | mx.MODE_HADAMARD, mx.LAYOUT_TILE)
    for g in (gc, gs, tc, ts):
        g.check()
    assert mx.quantizer_status() == 0
    for b in range(batch):
        wc, ws = util.canonical_to_tile_axis1(gc.t[b].cpu().numpy(), gs.t[b].cpu().numpy())
        assert np.array_equal(ts.t[b].cpu().numpy(), ws) and np.array_equal(tc.t[b].cpu().numpy(), wc)
        # and the canonical output is the plain-definition oracle's (these sizes are far too small for a boundary case)
        x = si.bf16_bits_to_f32(bits[b])
        want_c, want_s = mxfp4.quantize_matrix_canonical(mxfp4.hadamard_rotate(x).astype(np.float64), 1, RULE[mode])
        assert np.array_equal(gs.t[b].cpu().numpy(), want_s) and np.array_equal(gc.t[b].cpu().numpy(), want_c)


def test_rotation_is_refused_where_it_is_not_defined():
    import paper_2607_24377_b200 as mx
    x = torch.zeros((128, 256), dtype=torch.bfloat16, device="cuda")
    out = torch.zeros(128 * 256, dtype=torch.uint8, device="cuda")
    for axis, cols in ((1, 256), (0, 128)):
        with pytest.raises(mx.MxAttnError) as ei:
            mx.quantize_mxfp4_batched(x, out, out, 1, 128, cols, axis, mx.MODE_UOS | mx.MODE_HADAMARD, mx.LAYOUT_CANONICAL)
        assert ei.value.code == -2


@pytest.mark.parametrize("qmax", [6.0, 7.0, 7.25, 6.55, 8.0, 4.0, 15.5])
def test_generic_ceiling_boundary_matches_oracle(qmax):
    # Eq. 7: the ceiling family; TFS (6), OAS at block 32 (7), UOS (7.25)
    import paper_2607_24377_b200 as mx
    rows = 777
    bits = gaussian_bits(rows, 128, 400 + int(qmax * 100))
    bits[0, :32] = si.f32_to_bf16_bits(np.full(32, qmax, np.float32))           # the endpoint q maps to exactly q
    rule = mxfp4.ScaleRule("ceil", float(np.float32(qmax)))
    for axis in (1, 0):
        want_c, want_s = mxfp4.quantize_matrix_canonical(util.bits_to_f64(bits), axis, rule)
        codes = torch.zeros(want_c.shape, dtype=torch.uint8, device="cuda")
        scales = torch.zeros(want_s.shape, dtype=torch.uint8, device="cuda")
        mx.quantize_mxfp4_qmax(util.to_dev_bf16(bits), codes, scales, 1, rows, 128, axis, qmax, mx.LAYOUT_CANONICAL)
        torch.cuda.synchronize()
        assert np.array_equal(scales.cpu().numpy(), want_s)
        assert np.array_equal(codes.cpu().numpy(), want_c)


def test_qmax_sweep_of_tensor_error_bottoms_near_7_25():
    # the setting of the paper's Q_max study (Section 5.4.1) on a synthetic N(0,1) tensor: sweep 6.00 .. 8.00
    import paper_2607_24377_b200 as mx
    rows = 8192
    bits = gaussian_bits(rows, 128, 500, spread=False)
    x = util.bits_to_f64(bits)
    dev = util.to_dev_bf16(bits)
    codes = torch.zeros((rows, 64), dtype=torch.uint8, device="cuda"); scales = torch.zeros((rows, 4), dtype=torch.uint8, device="cuda")
    mse = {}
    for q in np.round(np.arange(6.0, 8.0001, 0.25), 2):
        mx.quantize_mxfp4_qmax(dev, codes, scales, 1, rows, 128, 1, float(q), mx.LAYOUT_CANONICAL)
        torch.cuda.synchronize()
        c = codes.cpu().numpy(); s = scales.cpu().numpy().astype(np.int32) - 127
        nib = np.stack([c & 15, c >> 4], axis=-1).reshape(rows, 4, 32)
        deq = mxfp4.dequantize_blocks(nib, s).reshape(rows, 128)
        mse[float(q)] = float(((deq - x) ** 2).mean())
    best = min(mse, key=mse.get)
    assert best in (7.0, 7.25, 7.5), mse
    assert mse[7.25] < mse[6.0] and mse[7.25] < mse[8.0]
