"""Bit-exact parity of the CUDA NVFP4 quantizer (the paper's comparison format, Section 5.2) with the oracle, through
the C ABI: tensor maxima, block scales (E4M3 codes), element codes and the tensor decode scale."""
import numpy as np
import pytest
import torch

import synth_inputs as si
from oracle import nvfp4
from tests import util

pytestmark = pytest.mark.gpu


def gaussian_bits(rows, cols, seed, spread=True):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((rows, cols)).astype(np.float32)
    if spread:                                  # block maxima over many binades below the tensor maximum: subnormal and zero scales too
        x *= np.exp2(rng.integers(-14, 3, size=(rows, 1))).astype(np.float32)
    return si.f32_to_bf16_bits(x)


def run_gpu(bits, batch, rows, cols, axis, layout=0):
    import paper_2607_24377_b200 as mx
    x = util.to_dev_bf16(bits)
    g_amax = util.guarded((batch,), torch.float32, float("nan"))
    g_ts = util.guarded((batch,), torch.float32, float("nan"))
    mx.tensor_amax(x, g_amax.t, batch, rows, cols)
    rp = -(-rows // 128) * 128
    if layout == mx.LAYOUT_TILE:
        gc = util.guarded((batch, rp // 128, 8192), torch.uint8, 0xAA); gs = util.guarded((batch, rp // 128, 1024), torch.uint8, 0xAA)
    elif axis == 1:
        gc = util.guarded((batch, rows, cols // 2), torch.uint8, 0xAA); gs = util.guarded((batch, rows, cols // 16), torch.uint8, 0xAA)
    else:
        gc = util.guarded((batch, cols, rp // 2), torch.uint8, 0xAA); gs = util.guarded((batch, cols, rp // 16), torch.uint8, 0xAA)
    mx.quantize_nvfp4(x, gc.t, gs.t, g_amax.t, g_ts.t, batch, rows, cols, axis, layout)
    for g in (g_amax, g_ts, gc, gs):
        g.check()
    return gc.t.cpu().numpy(), gs.t.cpu().numpy(), g_amax.t.cpu().numpy(), g_ts.t.cpu().numpy()


@pytest.mark.parametrize("batch,rows,cols", [(1, 1, 16), (1, 3, 32), (2, 7, 96), (3, 1000, 128), (1, 4099, 128), (2, 65, 4096)])
def test_axis1_matches_oracle_bit_exact(batch, rows, cols):
    bits = np.stack([gaussian_bits(rows, cols, 11 * rows + cols + b) for b in range(batch)])
    got_c, got_s, got_a, got_t = run_gpu(bits, batch, rows, cols, 1)
    for b in range(batch):
        x = util.bits_to_f64(bits[b])
        assert float(got_a[b]) == float(np.abs(x).max())
        want_c, want_s, want_t = nvfp4.quantize_matrix_canonical(x, 1)
        assert float(got_t[b]) == float(want_t)
        assert np.array_equal(got_s[b], want_s)
        assert np.array_equal(got_c[b], want_c)


@pytest.mark.parametrize("batch,rows,cols", [(1, 1, 128), (2, 31, 128), (1, 128, 128), (3, 200, 128), (1, 1000, 128), (1, 4500, 128), (2, 300, 64), (1, 260, 264)])
def test_axis0_matches_oracle_bit_exact(batch, rows, cols):
    bits = np.stack([gaussian_bits(rows, cols, 5 * rows + cols + b) for b in range(batch)])
    got_c, got_s, got_a, got_t = run_gpu(bits, batch, rows, cols, 0)
    for b in range(batch):
        x = util.bits_to_f64(bits[b])
        want_c, want_s, want_t = nvfp4.quantize_matrix_canonical(x, 0)
        assert float(got_a[b]) == float(np.abs(x).max()) and float(got_t[b]) == float(want_t)
        assert np.array_equal(got_s[b], want_s)
        assert np.array_equal(got_c[b], want_c)


def nv_tile_scales(scales8: np.ndarray) -> np.ndarray:
    """[n_tiles*128, 8] block scales (rows zero-padded) -> [n_tiles, 1024] two scale-factor atoms per tile."""
    nt = scales8.shape[0] // 128
    out = np.zeros((nt, 1024), np.uint8)
    r = np.arange(128)
    for t in range(nt):
        for c in range(8):
            out[t, (c // 4) * 512 + util.tile_scale_offset(r, c % 4)] = scales8[t * 128 + r, c]
    return out


@pytest.mark.parametrize("rows", [1, 100, 128, 1000])
def test_tile_layout_is_a_permutation_of_the_canonical_one(rows):
    import paper_2607_24377_b200 as mx
    bits = np.stack([gaussian_bits(rows, 128, 900 + rows + b) for b in range(2)])
    rp = -(-rows // 128) * 128
    for axis in (1, 0):
        can_c, can_s, _, _ = run_gpu(bits, 2, rows, 128, axis)
        til_c, til_s, _, _ = run_gpu(bits, 2, rows, 128, axis, mx.LAYOUT_TILE)
        for b in range(2):
            if axis == 1:
                sc = np.zeros((rp, 8), np.uint8); sc[:rows] = can_s[b]
                wc, _ = util.canonical_to_tile_axis1(can_c[b], np.zeros((rows, 4), np.uint8))
                ws = nv_tile_scales(sc)
            else:
                wc, _ = util.canonical_to_tile_axis0(can_c[b], np.zeros((128, rp // 32), np.uint8))
                # channel n, block c of the tile t: canonical [n, t*8 + c]
                ws = np.concatenate([nv_tile_scales(can_s[b][:, t * 8:t * 8 + 8]) for t in range(rp // 128)])
            assert np.array_equal(til_c[b], wc)
            assert np.array_equal(til_s[b], ws)


def test_every_block_maximum_rounds_like_the_oracle():
    # block maxima on a fine logarithmic grid under a fixed tensor maximum: every E4M3 code, its subnormals, the
    # saturating top and the rounding boundaries between them
    rows = 4096
    rng = np.random.default_rng(77)
    x = np.zeros((rows, 16), np.float32)
    x[:, 0] = np.exp2(np.linspace(-24, 0, rows)).astype(np.float32) * np.float32(3.0)
    x[:, 1:] = x[:, :1] * rng.uniform(-1, 1, (rows, 15)).astype(np.float32)
    x[0, 0] = 3.0
    bits = si.f32_to_bf16_bits(x)[None]
    got_c, got_s, got_a, got_t = run_gpu(bits, 1, rows, 16, 1)
    want_c, want_s, want_t = nvfp4.quantize_matrix_canonical(util.bits_to_f64(bits[0]), 1)
    assert np.array_equal(got_s[0], want_s) and np.array_equal(got_c[0], want_c)
    assert len(np.unique(want_s)) > 100                    # the sweep really covers the code range


def test_argument_errors():
    import paper_2607_24377_b200 as mx
    L = mx.lib()
    assert L.mxattn_quantize_nvfp4(None, 16, 16, 16, None, 1, 4, 32, 1, 0, None) == -1
    assert L.mxattn_quantize_nvfp4(16, 16, 16, 16, None, 1, 4, 24, 1, 0, None) == -2       # cols % 16
    assert L.mxattn_quantize_nvfp4(16, 16, 16, 16, None, 1, 4, 64, 1, 1, None) == -2       # tile layout needs cols 128
    assert L.mxattn_quantize_nvfp4(24, 16, 16, 16, None, 1, 4, 32, 1, 0, None) == -3
    assert L.mxattn_quantize_nvfp4(16, 16, 16, 16, None, 1, 4, 32, 2, 0, None) == -1
    assert L.mxattn_tensor_amax(16, None, 1, 4, 32, None) == -1
    assert L.mxattn_tensor_amax(16, 16, 1, 3, 9, None) == -2
