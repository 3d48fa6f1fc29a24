// MXFP4 block quantization kernels (paper Section 2, Eq. 4-7; Algorithm 1) for sm_100a.
//
// Both kernels are HBM-bound streaming passes: 2 bytes read, 0.5 + 1/32 bytes written per element.
//   axis 1 (Q, K): a block is 32 consecutive bf16 of one row.  One thread owns 8 elements (one
//     128-bit load); the 4 threads of a block combine their maxima with two shuffles.
//   axis 0 (V): a block is 32 consecutive rows (tokens) of one column.  A CTA stages a
//     128-token x 128-column slab in shared memory with coalesced 128-bit loads, quantizes down
//     the columns, and writes the transposed codes through a shared-memory staging tile so that
//     the global stores stay 128-bit.
#include <string.h>

#include "common.cuh"

namespace mxattn {

// ------------------------------------------------------------------------------------------
// max |x| over the eight bf16 in a uint4, as a bf16 bit pattern (compare as unsigned integers:
// monotone for non-negative floats).
__device__ __forceinline__ uint32_t absmax_bf16x8(const uint4& v) {
  const uint32_t m = 0x7FFF7FFFu;
  uint32_t a = __vmaxu2(__vmaxu2(v.x & m, v.y & m), __vmaxu2(v.z & m, v.w & m));
  return max(a & 0xFFFFu, a >> 16);
}

// Quantize the eight bf16 of `v` with scale 2^-e.
__device__ __forceinline__ uint32_t quantize_bf16x8(const uint4& v, float inv) {
  return pack_e2m1x8(bf16lo(v.x) * inv, bf16hi(v.x) * inv, bf16lo(v.y) * inv, bf16hi(v.y) * inv,
                     bf16lo(v.z) * inv, bf16hi(v.z) * inv, bf16lo(v.w) * inv, bf16hi(v.w) * inv);
}

// Packed fp32x2 arithmetic (two IEEE round-to-nearest fp32 operations per instruction; each half gives
// exactly the result of the scalar instruction).
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ uint64_t sub2(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t r;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
  return r;
}
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}

// One 16-byte chunk (8 bf16) -> packed codes and the block's shared exponent; the four lanes of a
// 32-element block combine their maxima with two shuffles.
__device__ __forceinline__ uint32_t quantize_chunk(const uint4& v, uint32_t rule, int* e_out) {
  uint32_t m = absmax_bf16x8(v);
  m = max(m, __shfl_xor_sync(0xFFFFFFFFu, m, 1));
  m = max(m, __shfl_xor_sync(0xFFFFFFFFu, m, 2));
  const int e = shared_exponent_rule(m << 16, rule);
  *e_out = e;
  return quantize_bf16x8(v, pow2_neg(e));
}

constexpr int kQThreads = 256;

// ------------------------------------------------------------------------------------------
// Axis 1, canonical layout: a linear streaming pass.  Work unit = one 16-byte chunk (8 elements);
// chunk i yields code word i and (with its three neighbours) scale byte i / 4.  A CTA owns 2048
// consecutive chunks (32 KiB) and issues all of its loads before it quantizes anything.
constexpr int kQChunksPerThread = 8;

__global__ void __launch_bounds__(kQThreads)
quantize_axis1_kernel(const uint4* __restrict__ in, uint32_t* __restrict__ codes,
                      uint8_t* __restrict__ scales, int64_t n_chunks, uint32_t rule) {
  const int lane = threadIdx.x & 31;
  const int64_t base = (int64_t)blockIdx.x * (kQThreads * kQChunksPerThread) + threadIdx.x;
  uint4 v[kQChunksPerThread];
#pragma unroll
  for (int u = 0; u < kQChunksPerThread; ++u) {
    const int64_t i = base + u * kQThreads;
    v[u] = i < n_chunks ? __ldg(in + i) : make_uint4(0u, 0u, 0u, 0u);
  }
#pragma unroll
  for (int u = 0; u < kQChunksPerThread; ++u) {
    const int64_t i = base + u * kQThreads;
    int e;
    const uint32_t packed = quantize_chunk(v[u], rule, &e);
    // four consecutive blocks (16 lanes) -> one 32-bit scale word
    const uint32_t eb = (uint32_t)(e + 127);
    const uint32_t b1 = __shfl_down_sync(0xFFFFFFFFu, eb, 4);
    const uint32_t b2 = __shfl_down_sync(0xFFFFFFFFu, eb, 8);
    const uint32_t b3 = __shfl_down_sync(0xFFFFFFFFu, eb, 12);
    if (i >= n_chunks) continue;
    codes[i] = packed;
    if ((lane & 15) == 0) {
      const int64_t g = i >> 2;                      // block index, multiple of 4 here
      if (i + 16 <= n_chunks) {
        *reinterpret_cast<uint32_t*>(scales + g) = eb | (b1 << 8) | (b2 << 16) | (b3 << 24);
      } else {                                       // ragged end: fewer than 4 blocks left
        scales[g] = (uint8_t)eb;
        if (i + 4 < n_chunks) scales[g + 1] = (uint8_t)b1;
        if (i + 8 < n_chunks) scales[g + 2] = (uint8_t)b2;
      }
    }
  }
}

// ------------------------------------------------------------------------------------------
// Axis 1, tile layout (cols == 128).  grid = (row tiles, batch); one CTA quantizes one 128-row
// tile: 32 KiB in, 8.5 KiB out.  A thread issues its eight 16-byte loads up front (the whole
// tile is in flight at once), then quantizes them; a warp covers two full rows per step, so the
// four lanes of a block and the sixteen lanes of a row are always in the same warp.
__global__ void __launch_bounds__(kQThreads)
quantize_axis1_tile_kernel(const uint4* __restrict__ in, uint8_t* __restrict__ codes,
                           uint8_t* __restrict__ scales, int64_t rows, uint32_t rule) {
  const int tid = threadIdx.x, lane = tid & 31;
  const int64_t tile = (int64_t)blockIdx.y * gridDim.x + blockIdx.x;
  const int64_t row0 = (int64_t)blockIdx.x * kTile;
  const uint4* src = in + ((int64_t)blockIdx.y * rows + row0) * 16;     // 16 chunks per row
  const int rows_here = (int)min((int64_t)kTile, rows - row0);
  uint4 v[8];
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    const int chunk = k * kQThreads + tid;           // row = chunk >> 4
    v[k] = (chunk >> 4) < rows_here ? __ldg(src + chunk) : make_uint4(0u, 0u, 0u, 0u);
  }
  uint32_t* ctile = reinterpret_cast<uint32_t*>(codes + tile * kTileCodeBytes);
  uint8_t* stile = scales + tile * kTileScaleBytes;
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    const int chunk = k * kQThreads + tid;
    const int r = chunk >> 4, c = (chunk >> 2) & 3;
    int e;
    const uint32_t packed = quantize_chunk(v[k], rule, &e);
    const uint32_t eb = (uint32_t)(e + 127);
    const uint32_t b1 = __shfl_down_sync(0xFFFFFFFFu, eb, 4);
    const uint32_t b2 = __shfl_down_sync(0xFFFFFFFFu, eb, 8);
    const uint32_t b3 = __shfl_down_sync(0xFFFFFFFFu, eb, 12);
    ctile[tile_code_offset(r, c) / 4 + (chunk & 3)] = packed;
    if ((lane & 15) == 0)
      *reinterpret_cast<uint32_t*>(stile + tile_scale_offset(r, 0)) = eb | (b1 << 8) | (b2 << 16) | (b3 << 24);
  }
}

// ------------------------------------------------------------------------------------------
// Axis 1 with the Hadamard rotation (cols == 128), both layouts.  A CTA takes 128 consecutive rows;
// FOUR lanes share a row and each holds 32 of its elements: lane q (0..3) loads the 16-byte chunks
// q, q + 4, q + 8, q + 12, so element index = 32 u + 8 q + i with u = 0..3 the chunk number within the
// lane and i = 0..7.  The butterfly stages of strides 1, 2, 4 (bits of i) and 32, 64 (bits of u) stay
// inside the thread; only strides 8 and 16 (bits of q) cross lanes -- two shuffle stages per row
// instead of the four that an 8-elements-per-lane split needs.  Stage order (ascending strides) and
// the fp32 arithmetic (every stage (a, b) -> (a + b, a - b) with a the lower index, then one multiply by
// fl32(1/sqrt(128))) are part of the definition, because the result feeds a rounding decision.  The MX block
// u is the chunk u of the four lanes: its maximum takes two more shuffles, its codes are one word per
// lane, its scale byte is written (with the row's other three) by lane 0.
// kRuleKind: 0 = OCP floor rule, 1 = UOS (boundary 7.25, the mantissa compare of shared_exponent), 2 = the
// boundary passed in `rule` (this kernel is bound by instruction issue, so the common rules are compiled in).
template <bool kTileLayout, int kRuleKind>
__global__ void __launch_bounds__(kQThreads)
quantize_axis1_rot_kernel(const uint4* __restrict__ in, uint8_t* __restrict__ codes,
                          uint8_t* __restrict__ scales, int64_t rows, uint32_t rule) {
  const int tid = threadIdx.x;
  const int q = tid & 3, rr = tid >> 2;              // lane within the row's quad; row within a 64-row pass
  // tile layout: grid = (row tiles, batch), `rows` per batch entry; canonical: grid = row groups, `rows` in total
  const int64_t row0 = (int64_t)blockIdx.x * kTile;
  const uint4* src = in + ((kTileLayout ? (int64_t)blockIdx.y * rows : 0) + row0) * 16;     // 16 chunks per row
  const int rows_here = (int)min((int64_t)kTile, rows - row0);
  uint4 v[2][4];
#pragma unroll
  for (int k = 0; k < 2; ++k)
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int r = k * 64 + rr;
      v[k][u] = r < rows_here ? __ldg(src + r * 16 + 4 * u + q) : make_uint4(0u, 0u, 0u, 0u);
    }
  const int64_t tile = (int64_t)blockIdx.y * gridDim.x + blockIdx.x;
  const uint64_t sgn1 = (q & 1) ? pack2(-1.0f, -1.0f) : pack2(1.0f, 1.0f);
  const uint64_t sgn2 = (q & 2) ? pack2(-1.0f, -1.0f) : pack2(1.0f, 1.0f);
#pragma unroll
  for (int k = 0; k < 2; ++k) {
    const int r = k * 64 + rr;
    // the 32 values as 16 packed pairs: pair j = elements (2j, 2j + 1) of the thread
    uint64_t pr[16];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const uint4& w = v[k][u];
      const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        // stride 1 on the way in: (a, b) -> (a + b, a - b)
        const float a = bf16lo(ww[j]), b = bf16hi(ww[j]);
        pr[4 * u + j] = pack2(__fadd_rn(a, b), __fsub_rn(a, b));
      }
    }
    // strides 2, 4 (pair strides 1, 2): inside each chunk, two elements per instruction
#pragma unroll
    for (int st = 1; st < 4; st <<= 1)
#pragma unroll
      for (int j = 0; j < 16; ++j)
        if ((j & st) == 0) {
          const uint64_t a = pr[j], b = pr[j + st];
          pr[j] = add2(a, b);
          pr[j + st] = sub2(a, b);
        }
    // strides 8, 16: across the quad.  The lower lane gets a + b = own * 1 + other, the upper one
    // a - b = own * (-1) + other (the product is exact, so the fma rounds like the add / subtract).
#pragma unroll
    for (int j = 0; j < 16; ++j) pr[j] = fma2(pr[j], sgn1, __shfl_xor_sync(0xFFFFFFFFu, pr[j], 1));
#pragma unroll
    for (int j = 0; j < 16; ++j) pr[j] = fma2(pr[j], sgn2, __shfl_xor_sync(0xFFFFFFFFu, pr[j], 2));
    // strides 32, 64 (pair strides 4, 8): across the thread's chunks
#pragma unroll
    for (int st = 4; st < 16; st <<= 1)
#pragma unroll
      for (int j = 0; j < 16; ++j)
        if ((j & st) == 0) {
          const uint64_t a = pr[j], b = pr[j + st];
          pr[j] = add2(a, b);
          pr[j + st] = sub2(a, b);
        }
    uint32_t word[4], sf = 0;
    const uint64_t norm2 = pack2(0.08838834764831845f, 0.08838834764831845f);
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      float mf = 0.0f;                               // max |.| as a float: the operand modifiers make |x| free
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        pr[4 * u + j] = mul2(pr[4 * u + j], norm2);
        float lo, hi;
        unpack2(pr[4 * u + j], lo, hi);
        mf = fmaxf(fmaxf(mf, fabsf(lo)), fabsf(hi));
      }
      mf = fmaxf(mf, __shfl_xor_sync(0xFFFFFFFFu, mf, 1));
      mf = fmaxf(mf, __shfl_xor_sync(0xFFFFFFFFu, mf, 2));
      const int e = kRuleKind == 2 ? shared_exponent_ceil(__float_as_uint(mf), rule)
                                   : shared_exponent(__float_as_uint(mf), kRuleKind == 1);
      const float inv = pow2_neg(e);
      const uint64_t inv2 = pack2(inv, inv);
      float x[8];
#pragma unroll
      for (int j = 0; j < 4; ++j) unpack2(mul2(pr[4 * u + j], inv2), x[2 * j], x[2 * j + 1]);
      word[u] = pack_e2m1x8(x[0], x[1], x[2], x[3], x[4], x[5], x[6], x[7]);
      sf |= (uint32_t)(e + 127) << (8 * u);
    }
    if (kTileLayout) {
      uint32_t* ctile = reinterpret_cast<uint32_t*>(codes + tile * kTileCodeBytes);
#pragma unroll
      for (int u = 0; u < 4; ++u) ctile[tile_code_offset(r, u) / 4 + q] = word[u];
      if (q == 0) *reinterpret_cast<uint32_t*>(scales + tile * kTileScaleBytes + tile_scale_offset(r, 0)) = sf;
    } else if (r < rows_here) {
      uint32_t* crow = reinterpret_cast<uint32_t*>(codes) + (row0 + r) * 16;
#pragma unroll
      for (int u = 0; u < 4; ++u) crow[4 * u + q] = word[u];
      if (q == 0) *reinterpret_cast<uint32_t*>(scales + (row0 + r) * 4) = sf;
    }
  }
}

// ------------------------------------------------------------------------------------------
// Axis 0.  256 threads; a CTA stages a 32 KiB slab of the input in shared memory:
//   tile layout:  128 tokens x 128 columns -> one 8.5 KiB tile image, written contiguously;
//                 grid = (1, ceil(rows/128), batch)
//   canonical:    256 tokens x 64 columns, so that every column leaves as ONE 128-byte segment of codes
//                 (and 8 scale bytes) instead of two 64-byte ones; grid = (ceil(cols/64), ceil(rows_pad/256), batch)
constexpr int kVThreads = 256;

template <bool kTileLayout>
__global__ void __launch_bounds__(kVThreads)
quantize_axis0_kernel(const uint16_t* __restrict__ in, uint8_t* __restrict__ codes,
                      uint8_t* __restrict__ scales, int64_t rows, int64_t cols, int64_t rows_pad,
                      uint32_t rule) {
  constexpr int kTok = kTileLayout ? 128 : 256;                   // tokens per slab
  constexpr int kCol = kTileLayout ? 128 : 64;                    // columns per slab
  constexpr int kColBytes = kTok / 2;                             // code bytes per column of the slab
  constexpr int kColBlocks = kTok / kBlock;                       // blocks (scale bytes) per column of the slab
  __shared__ __align__(16) uint16_t s_in[kTok][kCol];             // [token][column] raw bf16
  __shared__ __align__(16) uint8_t s_codes[kTileCodeBytes];       // [column][kColBytes], 16-byte chunks swizzled
  __shared__ __align__(16) uint8_t s_scales[kTileScaleBytes];

  const int tid = threadIdx.x;
  const int64_t col0 = (int64_t)blockIdx.x * kCol;
  const int64_t row0 = (int64_t)blockIdx.y * kTok;
  const int64_t b = blockIdx.z;
  const uint16_t* src = in + b * rows * cols;
  // staging offset of the 16-byte chunk c of column n: the tile image's own swizzle, or (canonical) the
  // chunk index XORed with the column pair so that the 8 threads of a store phase hit 8 different bank groups
  auto code_off = [](int n, int c) { return kTileLayout ? tile_code_offset(n, c) : n * kColBytes + ((c ^ ((n >> 1) & 7)) << 4); };

  // phase 1: slab -> shared, 16 B per thread per step, zero beyond the edges
#pragma unroll
  for (int k = 0; k < (kTok * kCol / 8) / kVThreads; ++k) {
    const int chunk = k * kVThreads + tid;
    const int t = chunk / (kCol / 8), cc = (chunk % (kCol / 8)) << 3;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (row0 + t < rows && col0 + cc < cols)
      v = __ldg(reinterpret_cast<const uint4*>(src + (row0 + t) * cols + col0 + cc));
    *reinterpret_cast<uint4*>(&s_in[t][cc]) = v;
  }
  __syncthreads();

  // phase 2: thread -> (column pair 2np, 2np+1; token block c).  One 32-bit shared load brings both
  // columns of a token, so the packed maximum and the two conversions share the 32 loads.
  {
    const int np = tid % (kCol / 2), c = tid / (kCol / 2);
    const uint32_t* s32 = reinterpret_cast<const uint32_t*>(&s_in[0][0]);
    uint32_t w[32];
    uint32_t m2 = 0;
#pragma unroll
    for (int i = 0; i < 32; ++i) {
      w[i] = s32[(c * 32 + i) * (kCol / 2) + np];
      m2 = __vmaxu2(m2, w[i] & 0x7FFF7FFFu);
    }
#pragma unroll
    for (int side = 0; side < 2; ++side) {          // side 0: column 2np (low halves), side 1: column 2np+1
      const int n = 2 * np + side;
      const uint32_t m = side ? (m2 >> 16) : (m2 & 0xFFFFu);
      const int e = shared_exponent_rule(m << 16, rule);
      const float inv = pow2_neg(e);
      uint32_t o[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        float f[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) f[i] = (side ? bf16hi(w[8 * q + i]) : bf16lo(w[8 * q + i])) * inv;
        o[q] = pack_e2m1x8(f[0], f[1], f[2], f[3], f[4], f[5], f[6], f[7]);
      }
      *reinterpret_cast<uint4*>(&s_codes[code_off(n, c)]) = make_uint4(o[0], o[1], o[2], o[3]);
      s_scales[kTileLayout ? tile_scale_offset(n, c) : (n * kColBlocks + c)] = (uint8_t)(e + 127);
    }
  }
  __syncthreads();

  // phase 3: staged slab -> global
  if (kTileLayout) {
    const int64_t tile = b * gridDim.y + blockIdx.y;            // cols == 128: one column tile
    uint4* dst = reinterpret_cast<uint4*>(codes + tile * kTileCodeBytes);
#pragma unroll
    for (int k = 0; k < kTileCodeBytes / 16 / kVThreads; ++k)
      dst[k * kVThreads + tid] = reinterpret_cast<const uint4*>(s_codes)[k * kVThreads + tid];
    if (tid < kTileScaleBytes / 16)
      reinterpret_cast<uint4*>(scales + tile * kTileScaleBytes)[tid] =
          reinterpret_cast<const uint4*>(s_scales)[tid];
  } else {
    // codes [cols, rows_pad/2]: column n owns kColBytes contiguous bytes of this slab (the second 128 tokens
    // only if they are inside rows_pad, which is a multiple of 128, not of 256)
    uint8_t* cdst = codes + b * cols * (rows_pad / 2);
    uint8_t* sdst = scales + b * cols * (rows_pad / 32);
    const bool second = row0 + 128 < rows_pad;
#pragma unroll
    for (int k = 0; k < kTileCodeBytes / 16 / kVThreads; ++k) {
      const int chunk = k * kVThreads + tid;
      const int n = chunk / (kColBytes / 16), q = chunk % (kColBytes / 16);
      if (col0 + n < cols && (q < 4 || second))
        *reinterpret_cast<uint4*>(cdst + (col0 + n) * (rows_pad / 2) + row0 / 2 + q * 16) =
            *reinterpret_cast<const uint4*>(&s_codes[code_off(n, q)]);
    }
    if (tid < 2 * kCol) {
      const int n = tid >> 1, half = tid & 1;
      if (col0 + n < cols && (half == 0 || second))
        *reinterpret_cast<uint32_t*>(sdst + (col0 + n) * (rows_pad / 32) + row0 / 32 + 4 * half) =
            reinterpret_cast<const uint32_t*>(s_scales)[n * 2 + half];
    }
  }
}

// ------------------------------------------------------------------------------------------
int launch_quantize(const void* in, void* codes, void* scales, int64_t batch, int64_t rows,
                    int64_t cols, int block_axis, int mode, int layout, cudaStream_t stream,
                    uint32_t rule_override) {
  if (!in || !codes || !scales) return MXATTN_EINVAL;
  if (batch <= 0 || rows <= 0 || cols <= 0) return MXATTN_EINVAL;
  if (block_axis != 0 && block_axis != 1) return MXATTN_EINVAL;
  const bool rotate = (mode & MXATTN_MODE_HADAMARD) != 0;
  mode &= ~MXATTN_MODE_HADAMARD;
  if (mode != MXATTN_MODE_OCP && mode != MXATTN_MODE_UOS) return MXATTN_EINVAL;
  if (rotate && (block_axis != 1 || cols != kHeadDim)) return MXATTN_EUNSUPPORTED;
  if (layout != MXATTN_LAYOUT_CANONICAL && layout != MXATTN_LAYOUT_TILE) return MXATTN_EINVAL;
  if (layout == MXATTN_LAYOUT_TILE && cols != kHeadDim) return MXATTN_EUNSUPPORTED;
  if (block_axis == 1 && cols % kBlock != 0) return MXATTN_EUNSUPPORTED;
  if (block_axis == 0 && cols % 8 != 0) return MXATTN_EUNSUPPORTED;
  if (!aligned16(in) || !aligned16(codes) || !aligned16(scales)) return MXATTN_EALIGN;
  const uint32_t rule = rule_override != 0xFFFFFFFFu ? rule_override : (mode == MXATTN_MODE_UOS ? kRuleUos : kRuleOcp);
  const int64_t rows_pad = (rows + kTile - 1) / kTile * kTile;

  if (block_axis == 1) {
    const bool tile = (layout == MXATTN_LAYOUT_TILE);
    const int64_t n_chunks = tile ? batch * rows_pad * 16 : batch * rows * (cols / 8);
    const int64_t blocks = (n_chunks + kQThreads * kQChunksPerThread - 1) / (kQThreads * kQChunksPerThread);
    if (!tile && blocks > 0x7FFFFFFF) return MXATTN_EUNSUPPORTED;
    if (tile) {
      if (rows_pad / kTile > 0x7FFFFFFF || batch > 65535) return MXATTN_EUNSUPPORTED;
      dim3 grid((unsigned)(rows_pad / kTile), (unsigned)batch);
      if (rotate) {
        auto kern = rule == kRuleOcp ? quantize_axis1_rot_kernel<true, 0>
                  : rule == kRuleUos ? quantize_axis1_rot_kernel<true, 1> : quantize_axis1_rot_kernel<true, 2>;
        kern<<<grid, kQThreads, 0, stream>>>((const uint4*)in, (uint8_t*)codes, (uint8_t*)scales, rows, rule);
      } else
        quantize_axis1_tile_kernel<<<grid, kQThreads, 0, stream>>>((const uint4*)in, (uint8_t*)codes,
                                                                          (uint8_t*)scales, rows, rule);
    } else {
      if (rotate) {                                  // cols == 128 here: batch * rows rows of 16 chunks
        const int64_t groups = (batch * rows + kTile - 1) / kTile;
        if (groups > 0x7FFFFFFF) return MXATTN_EUNSUPPORTED;
        auto kern = rule == kRuleOcp ? quantize_axis1_rot_kernel<false, 0>
                  : rule == kRuleUos ? quantize_axis1_rot_kernel<false, 1> : quantize_axis1_rot_kernel<false, 2>;
        kern<<<(unsigned)groups, kQThreads, 0, stream>>>((const uint4*)in, (uint8_t*)codes, (uint8_t*)scales,
                                                         batch * rows, rule);
      } else
        quantize_axis1_kernel<<<(unsigned)blocks, kQThreads, 0, stream>>>(
            (const uint4*)in, (uint32_t*)codes, (uint8_t*)scales, n_chunks, rule);
    }
  } else {
    const bool tile = (layout == MXATTN_LAYOUT_TILE);
    const int64_t ct = tile ? 1 : (cols + 63) / 64, rt = tile ? rows_pad / kTile : (rows_pad + 255) / 256;
    if (ct > 0x7FFFFFFF || rt > 65535 || batch > 65535) return MXATTN_EUNSUPPORTED;
    dim3 grid((unsigned)ct, (unsigned)rt, (unsigned)batch);
    if (tile)
      quantize_axis0_kernel<true><<<grid, kVThreads, 0, stream>>>(
          (const uint16_t*)in, (uint8_t*)codes, (uint8_t*)scales, rows, cols, rows_pad, rule);
    else
      quantize_axis0_kernel<false><<<grid, kVThreads, 0, stream>>>(
          (const uint16_t*)in, (uint8_t*)codes, (uint8_t*)scales, rows, cols, rows_pad, rule);
  }
  count_launch(1);
  return cudaGetLastError() == cudaSuccess ? MXATTN_OK : MXATTN_ECUDA;
}

}  // namespace mxattn

extern "C" int mxattn_quantize_mxfp4(const void* in, void* codes, void* e8m0_scales, int64_t rows,
                                     int64_t cols, int block_axis, int mode, void* stream) {
  return mxattn::launch_quantize(in, codes, e8m0_scales, 1, rows, cols, block_axis, mode,
                                 MXATTN_LAYOUT_CANONICAL, (cudaStream_t)stream);
}

extern "C" int mxattn_quantize_mxfp4_batched(const void* in, void* codes, void* e8m0_scales,
                                             int64_t batch, int64_t rows, int64_t cols,
                                             int block_axis, int mode, int layout, void* stream) {
  return mxattn::launch_quantize(in, codes, e8m0_scales, batch, rows, cols, block_axis, mode, layout,
                                 (cudaStream_t)stream);
}

extern "C" int mxattn_quantize_mxfp4_qmax(const void* in, void* codes, void* e8m0_scales, int64_t batch,
                                          int64_t rows, int64_t cols, int block_axis, float qmax,
                                          int layout, void* stream) {
  if (!(qmax >= 4.0f) || !(qmax < 16.0f)) return MXATTN_EINVAL;
  uint32_t bits;
  memcpy(&bits, &qmax, sizeof bits);
  return mxattn::launch_quantize(in, codes, e8m0_scales, batch, rows, cols, block_axis, MXATTN_MODE_UOS, layout,
                                 (cudaStream_t)stream, bits);
}
