"""The dense FP4 GEMM probe (the measuring stick of the roofline) computes what it says: its result on operands
quantized by the library equals the float64 product of the oracle's dequantized operands."""
import numpy as np
import pytest
import torch

import synth_inputs as si
from oracle import mxfp4
from tests import util

pytestmark = pytest.mark.gpu


def quantized_operand(x_bits, rows, K):
    """bf16 bit patterns [rows, K] -> tile images ordered [K/128][rows/128] on the device (UOS rule)."""
    import paper_2607_24377_b200 as mx
    kb = K // 128
    arranged = np.ascontiguousarray(x_bits.reshape(rows, kb, 128).transpose(1, 0, 2))        # [K/128][rows][128]
    codes = torch.zeros((kb, rows // 128, 8192), dtype=torch.uint8, device="cuda")
    scales = torch.zeros((kb, rows // 128, 512), dtype=torch.uint8, device="cuda")
    mx.quantize_mxfp4_batched(util.to_dev_bf16(arranged), codes, scales, kb, rows, 128, 1, mx.MODE_UOS, mx.LAYOUT_TILE)
    return codes, scales


@pytest.mark.parametrize("tile_n", [256, 128])
@pytest.mark.parametrize("M,N,K", [(128, 256, 128), (256, 512, 1024), (384, 256, 2048)])
def test_streaming_gemm_equals_the_product_of_the_dequantized_operands(M, N, K, tile_n):
    import paper_2607_24377_b200 as mx
    rng = np.random.default_rng(M + N + K)
    a = si.f32_to_bf16_bits(rng.standard_normal((M, K)).astype(np.float32) * np.exp2(rng.integers(-3, 4, (M, 1))).astype(np.float32))
    b = si.f32_to_bf16_bits(rng.standard_normal((N, K)).astype(np.float32))
    ac, asc = quantized_operand(a, M, K)
    bc, bsc = quantized_operand(b, N, K)
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    ad = mxfp4.quantize_dequantize(util.bits_to_f64(a), 1, mxfp4.UOS)
    bd = mxfp4.quantize_dequantize(util.bits_to_f64(b), 1, mxfp4.UOS)
    want = ad @ bd.T
    g = util.guarded((M, N), torch.float32, float("nan"))
    mx.probe_fp4_gemm(ac, asc, bc, bsc, g.t, M, N, K, K // 128, False, True, status, tile_n)
    g.check()
    assert int(status[0].item()) == 0
    got = g.t.double().cpu().numpy()
    assert np.linalg.norm(got - want) / np.linalg.norm(want) < 1e-6 and np.abs(got - want).max() < 1e-4 * np.abs(want).max()
    # bf16 output: the same values rounded
    g16 = util.guarded((M, N), torch.bfloat16, float("nan"))
    mx.probe_fp4_gemm(ac, asc, bc, bsc, g16.t, M, N, K, K // 128, False, False, status, tile_n)
    g16.check()
    assert torch.equal(g16.t, g.t.to(torch.bfloat16))


@pytest.mark.parametrize("tile_n", [256, 128])
def test_resident_mode_cycles_over_the_first_six_k_blocks(tile_n):
    import paper_2607_24377_b200 as mx
    M, N, K = 128, 256, 1024
    rng = np.random.default_rng(5)
    a = si.f32_to_bf16_bits(rng.standard_normal((M, K)).astype(np.float32))
    b = si.f32_to_bf16_bits(rng.standard_normal((N, K)).astype(np.float32))
    ac, asc = quantized_operand(a, M, K)
    bc, bsc = quantized_operand(b, N, K)
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    ad = mxfp4.quantize_dequantize(util.bits_to_f64(a), 1, mxfp4.UOS)[:, :768]
    bd = mxfp4.quantize_dequantize(util.bits_to_f64(b), 1, mxfp4.UOS)[:, :768]
    out = torch.zeros((M, N), dtype=torch.float32, device="cuda")
    mx.probe_fp4_gemm(ac, asc, bc, bsc, out, M, N, K, 18, True, True, status, tile_n)
    torch.cuda.synchronize()
    assert int(status[0].item()) == 0
    want = 3.0 * (ad @ bd.T)                                  # 18 steps = three rounds over blocks 0..5
    got = out.double().cpu().numpy()
    assert np.linalg.norm(got - want) / np.linalg.norm(want) < 1e-6


def test_argument_errors():
    import paper_2607_24377_b200 as mx
    L = mx.lib()
    assert L.mxattn_probe_fp4_gemm(16, 16, 16, 16, 16, 128, 256, 128, 1, 0, 1, 256, None, None) == -1
    assert L.mxattn_probe_fp4_gemm(16, 16, 16, 16, 16, 128, 128, 128, 1, 0, 1, 256, 16, None) == -2      # N % tile_n
    assert L.mxattn_probe_fp4_gemm(16, 16, 16, 16, 16, 128, 256, 256, 1, 0, 1, 256, 16, None) == -1      # streaming: k_steps == K/128
    assert L.mxattn_probe_fp4_gemm(16, 16, 16, 16, 16, 128, 256, 1024, 8, 1, 1, 256, 16, None) == -1     # resident: k_steps % 6
    assert L.mxattn_probe_fp4_gemm(16, 16, 16, 16, 16, 128, 256, 128, 1, 0, 1, 192, 16, None) == -1      # tile_n
    assert L.mxattn_probe_fp4_gemm(16, 16, 16, 16, 24, 128, 256, 128, 1, 0, 1, 256, 16, None) == -3
