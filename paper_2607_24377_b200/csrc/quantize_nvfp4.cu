// NVFP4 block quantization for sm_100a: the comparison format of the paper (named in its Introduction; Section 5.2,
// baseline "NVFP4"): E2M1 elements in blocks of 16 with an E4M3 block scale and one fp32 tensor-level scale.
//
// Two-level recipe, every step in IEEE fp32 (the order is part of the definition because the results are codes):
//   g   = fl32(2688 / A)       A = largest magnitude of the tensor (one per matrix of the batch), 2688 = 448 * 6
//   s_T = fl32(1 / g)          decode scale of the tensor
//   y_b = fl32(fl32(M_b * g) * fl32(1/6))          M_b = largest magnitude of the block
//   d_b = E4M3(y_b), round-to-nearest-even, saturating at 448
//   r_b = fl32(g / d_b)        (0 when d_b = 0)
//   code = sign | E2M1(fl32(|x| * r_b))
// Three HBM-bound passes: the tensor maximum (2 B/element read), then the quantizer (2 B read, 0.5 + 1/16 B written).
#include <cuda_fp16.h>

#include "common.cuh"

namespace mxattn {
namespace nv {

constexpr int kThreads = 256;
constexpr float kOneSixth = 0.16666667163372040f;      // fl32(1/6)
constexpr int kNvTileScaleBytes = 2 * kTileScaleBytes;   // two scale-factor atoms per 128 x 128 tile (8 blocks of 16 per row)

__device__ __forceinline__ uint32_t absmax_bf16x8(const uint4& v) {
  const uint32_t m = 0x7FFF7FFFu;
  uint32_t a = __vmaxu2(__vmaxu2(v.x & m, v.y & m), __vmaxu2(v.z & m, v.w & m));
  return max(a & 0xFFFFu, a >> 16);
}

// fp32 -> E4M3 code (round-to-nearest-even, saturating to 448) and back
__device__ __forceinline__ uint32_t e4m3_encode(float y) {
  uint16_t r;
  asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(0.0f), "f"(y));     // second source -> low byte
  return (uint32_t)(r & 0xFFu);
}
__device__ __forceinline__ float e4m3_decode(uint32_t code) {
  uint32_t h2;
  asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"((uint16_t)code));
  return __half2float(__ushort_as_half((unsigned short)(h2 & 0xFFFFu)));
}

__device__ __forceinline__ float encode_scale(float amax) { return amax == 0.0f ? 1.0f : __fdiv_rn(2688.0f, amax); }

// Block scale code and element multiplier of a block whose maximum magnitude is `m` (fp32, >= 0).
__device__ __forceinline__ float block_scale(float m, float g, uint32_t* code_out) {
  const float y = __fmul_rn(__fmul_rn(m, g), kOneSixth);
  const uint32_t code = e4m3_encode(y);
  *code_out = code;
  const float d = e4m3_decode(code);
  return d == 0.0f ? 0.0f : __fdiv_rn(g, d);
}

__device__ __forceinline__ uint32_t quantize_bf16x8(const uint4& v, float r) {
  return pack_e2m1x8(__fmul_rn(bf16lo(v.x), r), __fmul_rn(bf16hi(v.x), r), __fmul_rn(bf16lo(v.y), r), __fmul_rn(bf16hi(v.y), r),
                     __fmul_rn(bf16lo(v.z), r), __fmul_rn(bf16hi(v.z), r), __fmul_rn(bf16lo(v.w), r), __fmul_rn(bf16hi(v.w), r));
}

// ------------------------------------------------------------------------------------------
// Largest magnitude of each matrix of the batch: amax[b] (fp32; must be zero on entry).  grid = (chunks, batch).
__global__ void __launch_bounds__(kThreads) tensor_amax_kernel(const uint4* __restrict__ in, uint32_t* __restrict__ amax,
                                                               int64_t chunks_per_matrix) {
  const uint4* src = in + (int64_t)blockIdx.y * chunks_per_matrix;
  uint32_t m = 0;
  for (int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x; i < chunks_per_matrix; i += (int64_t)gridDim.x * kThreads)
    m = max(m, absmax_bf16x8(__ldg(src + i)));
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
  __shared__ uint32_t s[kThreads / 32];
  if ((threadIdx.x & 31) == 0) s[threadIdx.x >> 5] = m;
  __syncthreads();
  if (threadIdx.x == 0) {
#pragma unroll
    for (int w = 1; w < kThreads / 32; ++w) m = max(m, s[w]);
    atomicMax(amax + blockIdx.y, m << 16);          // non-negative floats order like their bit patterns
  }
}

// ------------------------------------------------------------------------------------------
// Axis 1 (Q, K: blocks of 16 along the row).  The CTA's 1024 chunks of 16 bytes (16 KiB) arrive in shared memory by
// asynchronous copies (chunk c at position c ^ ((c >> 3) & 7) within its group of eight: copies and reads both touch
// every bank group once per quarter warp); a thread then owns four consecutive chunks = two blocks: block maxima
// without shuffles, one division per block, one 16-byte store of codes and one 2-byte store of scales.
// grid = (ceil(chunks / 1024), batch); canonical layout: chunks = rows * cols / 8 per matrix; tile layout
// (cols == 128): chunks = rows_pad * 16, rows beyond `rows` read as zero.
constexpr int kA1ChunksPerCta = kThreads * 4;
template <bool kTileLayout>
__global__ void __launch_bounds__(kThreads)
quantize_nvfp4_axis1_kernel(const uint4* __restrict__ in, uint8_t* __restrict__ codes, uint8_t* __restrict__ scales,
                            const float* __restrict__ amax, float* __restrict__ tensor_scale, int64_t rows, int64_t cols,
                            int64_t rows_pad) {
  __shared__ uint4 s_v[kA1ChunksPerCta];
  const int tid = threadIdx.x;
  const int64_t b = blockIdx.y;
  const int64_t chunks_per_row = cols / 8;
  const int64_t n_valid = rows * chunks_per_row;                                  // chunks that exist in the input
  const int64_t n_out = (kTileLayout ? rows_pad : rows) * chunks_per_row;         // chunks that are written
  const uint4* src = in + b * n_valid;
  const int64_t base = (int64_t)blockIdx.x * kA1ChunksPerCta;
  auto pos = [](int c) { return c ^ ((c >> 3) & 7); };
#pragma unroll
  for (int u = 0; u < 4; ++u) {
    const int c = u * kThreads + tid;
    const bool inside = base + c < n_valid;
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"((uint32_t)__cvta_generic_to_shared(&s_v[pos(c)])),
                 "l"(inside ? src + base + c : in), "r"(inside ? 16 : 0) : "memory");
  }
  const float g = encode_scale(amax[b]);
  if (blockIdx.x == 0 && tid == 0 && tensor_scale) tensor_scale[b] = __fdiv_rn(1.0f, g);
  asm volatile("cp.async.wait_all;" ::: "memory");
  __syncthreads();
  const int64_t i = base + 4 * tid;                 // first of this thread's four chunks (n_out is even: whole blocks only)
  if (i >= n_out) return;
  uint4 v[4];
#pragma unroll
  for (int k = 0; k < 4; ++k) v[k] = s_v[pos(4 * tid + k)];
  uint32_t sc[2], w[4];
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const uint32_t m = max(absmax_bf16x8(v[2 * h]), absmax_bf16x8(v[2 * h + 1]));
    const float r = block_scale(__uint_as_float(m << 16), g, &sc[h]);
    w[2 * h] = quantize_bf16x8(v[2 * h], r);
    w[2 * h + 1] = quantize_bf16x8(v[2 * h + 1], r);
  }
  const bool both = i + 2 < n_out;                  // the matrix may end after this thread's first block
  if (kTileLayout) {                                // 16 chunks per row: the four chunks are one 32-column group of one row
    const int64_t row = i >> 4;
    const int q = (int)(i & 15) >> 2;
    const int64_t tile = b * (rows_pad / kTile) + row / kTile;
    const int rr = (int)(row % kTile);
    *reinterpret_cast<uint4*>(codes + tile * kTileCodeBytes + tile_code_offset(rr, q)) = make_uint4(w[0], w[1], w[2], w[3]);
    // blocks 2q and 2q + 1 of the row: adjacent bytes of one scale-factor atom
    *reinterpret_cast<uint16_t*>(scales + tile * kNvTileScaleBytes + (q >> 1) * kTileScaleBytes + tile_scale_offset(rr, (2 * q) & 3)) =
        (uint16_t)(sc[0] | (sc[1] << 8));
  } else {
    uint32_t* cdst = reinterpret_cast<uint32_t*>(codes) + b * n_out + i;
    uint8_t* sdst = scales + b * (n_out / 2) + (i >> 1);
    if (both && (((b * n_out) & 3) == 0)) {
      *reinterpret_cast<uint4*>(cdst) = make_uint4(w[0], w[1], w[2], w[3]);
    } else {
      *reinterpret_cast<uint2*>(cdst) = make_uint2(w[0], w[1]);
      if (both) *reinterpret_cast<uint2*>(cdst + 2) = make_uint2(w[2], w[3]);
    }
    if (both && (((b * (n_out / 2)) & 1) == 0)) {
      *reinterpret_cast<uint16_t*>(sdst) = (uint16_t)(sc[0] | (sc[1] << 8));
    } else {
      sdst[0] = (uint8_t)sc[0];
      if (both) sdst[1] = (uint8_t)sc[1];
    }
  }
}

// ------------------------------------------------------------------------------------------
// Axis 0 (V: blocks of 16 along the rows = tokens), outputs transposed (column-major, token-contiguous).
// A CTA stages a 128-token x 128-column slab; thread -> (column pair, chunk of 32 tokens = two blocks).
// grid = (ceil(cols / 128), rows_pad / 128, batch).
template <bool kTileLayout>
__global__ void __launch_bounds__(kThreads)
quantize_nvfp4_axis0_kernel(const uint16_t* __restrict__ in, uint8_t* __restrict__ codes, uint8_t* __restrict__ scales,
                            const float* __restrict__ amax, float* __restrict__ tensor_scale, int64_t rows, int64_t cols,
                            int64_t rows_pad) {
  __shared__ __align__(16) uint16_t s_in[kTile][kTile];
  __shared__ __align__(16) uint8_t s_codes[kTileCodeBytes];
  __shared__ __align__(16) uint8_t s_scales[kNvTileScaleBytes];
  const int tid = threadIdx.x;
  const int64_t col0 = (int64_t)blockIdx.x * kTile, row0 = (int64_t)blockIdx.y * kTile, b = blockIdx.z;
  const float g = encode_scale(amax[b]);
  if (blockIdx.x == 0 && blockIdx.y == 0 && tid == 0 && tensor_scale) tensor_scale[b] = __fdiv_rn(1.0f, g);
  const uint16_t* src = in + b * rows * cols;
#pragma unroll
  for (int k = 0; k < (kTile * kTile / 8) / kThreads; ++k) {
    const int chunk = k * kThreads + tid;
    const int t = chunk >> 4, cc = (chunk & 15) << 3;
    // asynchronous 16-byte copy straight into shared memory; nothing is read (and zeros are written) beyond the edges
    const bool inside = row0 + t < rows && col0 + cc < cols;
    const uint16_t* gsrc = inside ? src + (row0 + t) * cols + col0 + cc : src;
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"((uint32_t)__cvta_generic_to_shared(&s_in[t][cc])), "l"(gsrc), "r"(inside ? 16 : 0) : "memory");
  }
  asm volatile("cp.async.wait_all;" ::: "memory");
  __syncthreads();
  {
    const int np = tid & 63, c = tid >> 6;              // column pair, chunk of 32 tokens
    const uint32_t* s32 = reinterpret_cast<const uint32_t*>(&s_in[0][0]);
    uint32_t w[32], m2[2] = {0u, 0u};
#pragma unroll
    for (int i = 0; i < 32; ++i) {
      w[i] = s32[(c * 32 + i) * (kTile / 2) + np];
      m2[i >> 4] = __vmaxu2(m2[i >> 4], w[i] & 0x7FFF7FFFu);
    }
#pragma unroll
    for (int side = 0; side < 2; ++side) {
      const int n = 2 * np + side;
      uint32_t o[4];
#pragma unroll
      for (int hb = 0; hb < 2; ++hb) {                  // the two blocks of 16 tokens
        const uint32_t m = side ? (m2[hb] >> 16) : (m2[hb] & 0xFFFFu);
        uint32_t sc;
        const float r = block_scale(__uint_as_float(m << 16), g, &sc);
#pragma unroll
        for (int q = 0; q < 2; ++q) {
          float f[8];
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const uint32_t ww = w[16 * hb + 8 * q + i];
            f[i] = __fmul_rn(side ? bf16hi(ww) : bf16lo(ww), r);
          }
          o[2 * hb + q] = pack_e2m1x8(f[0], f[1], f[2], f[3], f[4], f[5], f[6], f[7]);
        }
        const int blk = 2 * c + hb;                      // block of 16 tokens within the slab, 0..7
        s_scales[kTileLayout ? ((blk >> 2) * kTileScaleBytes + tile_scale_offset(n, blk & 3)) : (n * 8 + blk)] = (uint8_t)sc;
      }
      *reinterpret_cast<uint4*>(&s_codes[tile_code_offset(n, c)]) = make_uint4(o[0], o[1], o[2], o[3]);
    }
  }
  __syncthreads();
  if (kTileLayout) {
    const int64_t tile = b * gridDim.y + blockIdx.y;
    uint4* dst = reinterpret_cast<uint4*>(codes + tile * kTileCodeBytes);
#pragma unroll
    for (int k = 0; k < kTileCodeBytes / 16 / kThreads; ++k)
      dst[k * kThreads + tid] = reinterpret_cast<const uint4*>(s_codes)[k * kThreads + tid];
    if (tid < kNvTileScaleBytes / 16)
      reinterpret_cast<uint4*>(scales + tile * kNvTileScaleBytes)[tid] = reinterpret_cast<const uint4*>(s_scales)[tid];
  } else {
    uint8_t* cdst = codes + b * cols * (rows_pad / 2);
    uint8_t* sdst = scales + b * cols * (rows_pad / 16);
#pragma unroll
    for (int k = 0; k < kTileCodeBytes / 16 / kThreads; ++k) {
      const int chunk = k * kThreads + tid;
      const int n = chunk >> 2, q = chunk & 3;
      if (col0 + n < cols)
        *reinterpret_cast<uint4*>(cdst + (col0 + n) * (rows_pad / 2) + row0 / 2 + q * 16) =
            *reinterpret_cast<const uint4*>(&s_codes[tile_code_offset(n, q)]);
    }
    if (tid < kTile && col0 + tid < cols)
      *reinterpret_cast<uint2*>(sdst + (col0 + tid) * (rows_pad / 16) + row0 / 16) = reinterpret_cast<const uint2*>(s_scales)[tid];
  }
}

}  // namespace nv

int launch_tensor_amax(const void* in, float* amax, int64_t batch, int64_t rows, int64_t cols, cudaStream_t stream) {
  if (!in || !amax) return MXATTN_EINVAL;
  if (batch <= 0 || rows <= 0 || cols <= 0) return MXATTN_EINVAL;
  if ((rows * cols) % 8 != 0) return MXATTN_EUNSUPPORTED;
  if (!aligned16(in) || (reinterpret_cast<uintptr_t>(amax) & 3u)) return MXATTN_EALIGN;
  if (batch > 65535) return MXATTN_EUNSUPPORTED;
  const int64_t chunks = rows * cols / 8;
  int64_t blocks = (chunks + nv::kThreads * 8 - 1) / (nv::kThreads * 8);
  if (blocks > 1184) blocks = 1184;                 // 8 CTAs per SM at most: the loop strides over the rest
  if (cudaMemsetAsync(amax, 0, (size_t)batch * sizeof(float), stream) != cudaSuccess) return MXATTN_ECUDA;
  nv::tensor_amax_kernel<<<dim3((unsigned)blocks, (unsigned)batch), nv::kThreads, 0, stream>>>(
      (const uint4*)in, reinterpret_cast<uint32_t*>(amax), chunks);
  count_launch(1);
  return cudaGetLastError() == cudaSuccess ? MXATTN_OK : MXATTN_ECUDA;
}

int launch_quantize_nvfp4(const void* in, void* codes, void* scales, const float* amax, float* tensor_scale, int64_t batch,
                          int64_t rows, int64_t cols, int block_axis, int layout, cudaStream_t stream) {
  if (!in || !codes || !scales || !amax) return MXATTN_EINVAL;
  if (batch <= 0 || rows <= 0 || cols <= 0) return MXATTN_EINVAL;
  if (block_axis != 0 && block_axis != 1) return MXATTN_EINVAL;
  if (layout != MXATTN_LAYOUT_CANONICAL && layout != MXATTN_LAYOUT_TILE) return MXATTN_EINVAL;
  if (layout == MXATTN_LAYOUT_TILE && cols != kHeadDim) return MXATTN_EUNSUPPORTED;
  if (block_axis == 1 && cols % 16 != 0) return MXATTN_EUNSUPPORTED;
  if (block_axis == 0 && cols % 8 != 0) return MXATTN_EUNSUPPORTED;
  if (!aligned16(in) || !aligned16(codes) || !aligned16(scales)) return MXATTN_EALIGN;
  if ((reinterpret_cast<uintptr_t>(amax) & 3u) || (reinterpret_cast<uintptr_t>(tensor_scale) & 3u)) return MXATTN_EALIGN;
  if (batch > 65535) return MXATTN_EUNSUPPORTED;
  const int64_t rows_pad = (rows + kTile - 1) / kTile * kTile;
  const bool tile = (layout == MXATTN_LAYOUT_TILE);
  if (block_axis == 1) {
    const int64_t n_out = (tile ? rows_pad : rows) * (cols / 8);
    const int64_t blocks = (n_out + nv::kA1ChunksPerCta - 1) / nv::kA1ChunksPerCta;
    if (blocks > 0x7FFFFFFF) return MXATTN_EUNSUPPORTED;
    dim3 grid((unsigned)blocks, (unsigned)batch);
    if (tile)
      nv::quantize_nvfp4_axis1_kernel<true><<<grid, nv::kThreads, 0, stream>>>((const uint4*)in, (uint8_t*)codes, (uint8_t*)scales,
                                                                               amax, tensor_scale, rows, cols, rows_pad);
    else
      nv::quantize_nvfp4_axis1_kernel<false><<<grid, nv::kThreads, 0, stream>>>((const uint4*)in, (uint8_t*)codes, (uint8_t*)scales,
                                                                                amax, tensor_scale, rows, cols, rows_pad);
  } else {
    const int64_t ct = (cols + kTile - 1) / kTile, rt = rows_pad / kTile;
    if (ct > 0x7FFFFFFF || rt > 65535) return MXATTN_EUNSUPPORTED;
    dim3 grid((unsigned)ct, (unsigned)rt, (unsigned)batch);
    if (tile)
      nv::quantize_nvfp4_axis0_kernel<true><<<grid, nv::kThreads, 0, stream>>>((const uint16_t*)in, (uint8_t*)codes, (uint8_t*)scales,
                                                                               amax, tensor_scale, rows, cols, rows_pad);
    else
      nv::quantize_nvfp4_axis0_kernel<false><<<grid, nv::kThreads, 0, stream>>>((const uint16_t*)in, (uint8_t*)codes, (uint8_t*)scales,
                                                                                amax, tensor_scale, rows, cols, rows_pad);
  }
  count_launch(1);
  return cudaGetLastError() == cudaSuccess ? MXATTN_OK : MXATTN_ECUDA;
}

}  // namespace mxattn

extern "C" int mxattn_tensor_amax(const void* in, void* amax, int64_t batch, int64_t rows, int64_t cols, void* stream) {
  return mxattn::launch_tensor_amax(in, static_cast<float*>(amax), batch, rows, cols, (cudaStream_t)stream);
}

extern "C" int mxattn_quantize_nvfp4(const void* in, void* codes, void* e4m3_scales, const void* tensor_amax,
                                     void* tensor_scale, int64_t batch, int64_t rows, int64_t cols, int block_axis,
                                     int layout, void* stream) {
  return mxattn::launch_quantize_nvfp4(in, codes, e4m3_scales, static_cast<const float*>(tensor_amax),
                                       static_cast<float*>(tensor_scale), batch, rows, cols, block_axis, layout,
                                       (cudaStream_t)stream);
}
