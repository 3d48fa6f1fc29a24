// MXFP4 block quantization kernels (paper Section 2, Eq. 4-7; Algorithm 1) for sm_100a.
//
// All kernels are HBM-bound streaming passes: 2 bytes read, 0.5 + 1/32 bytes written per element.
//   axis 1 (Q, K): a block is 32 consecutive bf16 of one row.  The CTA's input arrives in shared memory by
//     asynchronous 16-byte copies; one thread then owns a whole block (four 16-byte chunks) and writes its
//     16 bytes of codes with one store.
//   axis 0 (V): a block is 32 consecutive rows (tokens) of one column.  A CTA stages a
//     128-token x 128-column slab in shared memory with coalesced 128-bit loads, quantizes down
//     the columns, and writes the transposed codes through a shared-memory staging tile so that
//     the global stores stay 128-bit.
//   axis 1 with the Hadamard rotation of Algorithm 2 (Q, K): the rotation of a 128-row tile is one bf16 matrix
//     product with the +-1 matrix on the tensor core; the quantizer reads the rotated rows out of tensor memory.
#include <string.h>

#include "common.cuh"
#include "tc_helpers.cuh"

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

constexpr int kQThreads = 256;

// ------------------------------------------------------------------------------------------
// Axis 1, canonical layout: a linear streaming pass.  Work unit = one 32-element block = four 16-byte chunks;
// block g yields 16 bytes of codes and scale byte g.  A CTA owns 1024 consecutive chunks (16 KiB).  Measured against
// the earlier form (a thread per chunk, loads to registers, block maximum by two shuffles, 4-byte code stores):
// 0.83 / 0.93 / 0.98 of the plain-copy rate at 2^26 / 2^27 / 2^28 elements then, 0.89 / 1.01 / 1.06 now.
constexpr int kQChunksPerThread = 4;

__global__ void __launch_bounds__(kQThreads)
quantize_axis1_kernel(const uint4* __restrict__ in, uint32_t* __restrict__ codes,
                      uint8_t* __restrict__ scales, int64_t n_chunks, uint32_t rule) {
  // The CTA's chunks arrive in shared memory by asynchronous 16-byte copies; then a thread owns whole blocks (four
  // consecutive chunks): block maximum without shuffles, 16 bytes of codes per store.  Chunk c sits at position
  // c ^ ((c >> 3) & 7) within its group of eight, so that both the copies (consecutive c per warp) and the reads
  // (c = 4 blk + k per thread) touch every bank group once per quarter warp.
  __shared__ uint4 s_v[kQThreads * kQChunksPerThread];
  const int tid = threadIdx.x, lane = tid & 31;
  const int64_t base = (int64_t)blockIdx.x * (kQThreads * kQChunksPerThread);
  auto pos = [](int c) { return c ^ ((c >> 3) & 7); };
#pragma unroll
  for (int u = 0; u < kQChunksPerThread; ++u) {
    const int c = u * kQThreads + tid;
    const bool inside = base + c < n_chunks;
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"((uint32_t)__cvta_generic_to_shared(&s_v[pos(c)])),
                 "l"(inside ? in + base + c : in), "r"(inside ? 16 : 0) : "memory");
  }
  asm volatile("cp.async.wait_all;" ::: "memory");
  __syncthreads();
  const int64_t n_blocks = n_chunks >> 2;           // cols is a multiple of 32: whole blocks only
  uint4* codes16 = reinterpret_cast<uint4*>(codes);
#pragma unroll
  for (int r = 0; r < kQChunksPerThread / 4; ++r) {
    const int blk = r * kQThreads + tid;
    const int64_t g = (base >> 2) + blk;            // global block index
    uint4 v[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) v[k] = s_v[pos(4 * blk + k)];
    const uint32_t m = max(max(absmax_bf16x8(v[0]), absmax_bf16x8(v[1])), max(absmax_bf16x8(v[2]), absmax_bf16x8(v[3])));
    const int e = shared_exponent_rule(m << 16, rule);
    const float inv = pow2_neg(e);
    const uint32_t eb = (uint32_t)(e + 127);
    // four consecutive blocks (4 lanes) -> one 32-bit scale word
    const uint32_t b1 = __shfl_down_sync(0xFFFFFFFFu, eb, 1);
    const uint32_t b2 = __shfl_down_sync(0xFFFFFFFFu, eb, 2);
    const uint32_t b3 = __shfl_down_sync(0xFFFFFFFFu, eb, 3);
    if (g >= n_blocks) continue;
    codes16[g] = make_uint4(quantize_bf16x8(v[0], inv), quantize_bf16x8(v[1], inv), quantize_bf16x8(v[2], inv), quantize_bf16x8(v[3], inv));
    if ((lane & 3) == 0) {
      if (g + 4 <= n_blocks) {
        *reinterpret_cast<uint32_t*>(scales + g) = eb | (b1 << 8) | (b2 << 16) | (b3 << 24);
      } else {                                       // ragged end: fewer than 4 blocks left
        scales[g] = (uint8_t)eb;
        if (g + 1 < n_blocks) scales[g + 1] = (uint8_t)b1;
        if (g + 2 < n_blocks) scales[g + 2] = (uint8_t)b2;
      }
    }
  }
}

// ------------------------------------------------------------------------------------------
// Axis 1, tile layout (cols == 128).  grid = (2 x row tiles, batch); one CTA quantizes half a 128-row tile
// (64 rows, 16 KiB in) the same way: asynchronous copies into shared memory, one block (row r, 32 columns c) per
// thread, one 16-byte store into the tile image, one 32-bit scale store per row.
__global__ void __launch_bounds__(kQThreads)
quantize_axis1_tile_kernel(const uint4* __restrict__ in, uint8_t* __restrict__ codes,
                           uint8_t* __restrict__ scales, int64_t rows, uint32_t rule) {
  __shared__ uint4 s_v[kQThreads * 4];
  const int tid = threadIdx.x;
  const int64_t tile = (int64_t)blockIdx.y * (gridDim.x >> 1) + (blockIdx.x >> 1);
  const int half = blockIdx.x & 1;
  const int64_t row0 = (int64_t)(blockIdx.x >> 1) * kTile + half * 64;
  const uint4* src = in + ((int64_t)blockIdx.y * rows + row0) * 16;     // 16 chunks per row
  const int rows_here = (int)max((int64_t)0, min((int64_t)64, rows - row0));
  auto pos = [](int c) { return c ^ ((c >> 3) & 7); };
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const int chunk = k * kQThreads + tid;           // row = chunk >> 4
    const bool inside = (chunk >> 4) < rows_here;    // rows beyond the matrix are zero blocks of the padded tile
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"((uint32_t)__cvta_generic_to_shared(&s_v[pos(chunk)])),
                 "l"(inside ? src + chunk : in), "r"(inside ? 16 : 0) : "memory");
  }
  asm volatile("cp.async.wait_all;" ::: "memory");
  __syncthreads();
  const int r = half * 64 + (tid >> 2), c = tid & 3;
  uint4 v[4];
#pragma unroll
  for (int k = 0; k < 4; ++k) v[k] = s_v[pos(4 * tid + k)];
  const uint32_t m = max(max(absmax_bf16x8(v[0]), absmax_bf16x8(v[1])), max(absmax_bf16x8(v[2]), absmax_bf16x8(v[3])));
  const int e = shared_exponent_rule(m << 16, rule);
  const float inv = pow2_neg(e);
  const uint32_t eb = (uint32_t)(e + 127);
  const uint32_t b1 = __shfl_down_sync(0xFFFFFFFFu, eb, 1);
  const uint32_t b2 = __shfl_down_sync(0xFFFFFFFFu, eb, 2);
  const uint32_t b3 = __shfl_down_sync(0xFFFFFFFFu, eb, 3);
  *reinterpret_cast<uint4*>(codes + tile * kTileCodeBytes + tile_code_offset(r, c)) =
      make_uint4(quantize_bf16x8(v[0], inv), quantize_bf16x8(v[1], inv), quantize_bf16x8(v[2], inv), quantize_bf16x8(v[3], inv));
  if (c == 0)
    *reinterpret_cast<uint32_t*>(scales + tile * kTileScaleBytes + tile_scale_offset(r, 0)) = eb | (b1 << 8) | (b2 << 16) | (b3 << 24);
}

// ------------------------------------------------------------------------------------------
// Axis 1 with the Hadamard rotation on the tensor core (cols == 128), both layouts.  The rotation of a 128-row tile,
// Y = X H_128, is one 128 x 128 x 128 bf16 matrix product: X is bf16 as given, the entries of H are +-1 (exact in
// bf16), every product is exact and the sums are accumulated in fp32 by tcgen05.mma kind::f16 into tensor memory.
// Two threads then share a row of Y (64 columns = two blocks each): scale by fl32(1/sqrt(128)), block maxima, quantize.
// Against the exact product rounded once to fp32 the tensor core's fp32 accumulation carries rounding noise of about
// 1e-7 relative, which moves a code only where a value sits that close to a rounding boundary.
//
// Persistent CTAs (two per SM, 256 threads) walk the tiles.  H (32 KiB, generated once per CTA) and two X buffers
// (32 KiB each) sit in shared memory as K-major operand tiles (two 64-element K halves, 128-byte swizzle); X arrives
// by 16-byte asynchronous copies straight into its swizzled place; two accumulators of 128 tensor-memory columns
// alternate, so that the product of tile i runs while tile i - 1 is quantized and tile i + 1 is fetched.
namespace rot {
using namespace fwd;
constexpr int kThreads = 256;
constexpr int kHalf = 16384;                              // one K half of an operand tile: 128 rows x 128 bytes
constexpr int kOffH = 4 * kHalf;                          // after the two X buffers
constexpr int kOffBar = 6 * kHalf;
constexpr int kSmemBytes = kOffBar + 64 + 1024;           // + barriers, slots, slack for the 1024-byte alignment
__device__ int g_status = 0;                               // non-zero if a bounded wait for a product ever ran out

__device__ __forceinline__ int half_chunk_offset(int r, int c) { return r * 128 + ((c ^ (r & 7)) << 4); }

template <bool kTileLayout, int kRuleKind>
__global__ void __launch_bounds__(kThreads, 2)
quantize_axis1_rot_tc_kernel(const uint4* __restrict__ in, uint8_t* __restrict__ codes, uint8_t* __restrict__ scales,
                             int64_t rows, int tiles_per_matrix, int n_tiles, uint32_t rule) {
  // tile layout: `rows` per matrix of the batch, tile = matrix * tiles_per_matrix + tile within the matrix;
  // canonical: one matrix of `rows` rows (the batch is contiguous), tiles_per_matrix == n_tiles
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t sbase = smem_u32(smem);
  const uint32_t bar0 = sbase + kOffBar;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + kOffBar + 16);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + kOffBar + 24);
  const int tid = threadIdx.x, warp = tid >> 5;
  const int n_my = ((int)blockIdx.x < n_tiles) ? (n_tiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;

  auto tile_rows = [&](int tile, int64_t* first_row) {       // rows of the input this tile covers
    const int m = tile / tiles_per_matrix, t = tile - m * tiles_per_matrix;
    *first_row = (int64_t)m * rows + (int64_t)t * kTile;
    return (int)min((int64_t)kTile, rows - (int64_t)t * kTile);
  };
  auto fetch = [&](int tile, int buf) {                       // X tile -> shared memory, zero beyond the matrix
    int64_t first;
    const int here = tile_rows(tile, &first);
    const uint4* src = in + first * 16;
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const int chunk = k * kThreads + tid;
      const int r = chunk >> 4, cc = chunk & 15;
      const uint32_t dst = sbase + buf * 2 * kHalf + (cc >> 3) * kHalf + half_chunk_offset(r, cc & 7);
      const bool valid = r < here;
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(valid ? src + chunk : in), "r"(valid ? 16 : 0) : "memory");
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };

  if (tid == 0) {
    mbar_init(bar0, 1); mbar_init(bar0 + 8, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 256;" ::"r"(smem_u32(tmem_slot)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if (n_my > 0) fetch(blockIdx.x, 0);
  // H as the B operand: B[n][k] = H[k][n] = (-1)^popcount(n & k); chunk (n, cc) holds k = 8 cc .. 8 cc + 7
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    const int chunk = k * kThreads + tid;
    const int n = chunk >> 4, cc = chunk & 15;
    const uint32_t base_par = (uint32_t)__popc(n & (cc << 3)) & 1u;
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const uint32_t p0 = (base_par ^ ((uint32_t)__popc(n & (2 * i)) & 1u)), p1 = (base_par ^ ((uint32_t)__popc(n & (2 * i + 1)) & 1u));
      w[i] = (0x3F80u | (p0 << 15)) | ((0x3F80u | (p1 << 15)) << 16);       // bf16 +1 / -1
    }
    *reinterpret_cast<uint4*>(smem + kOffH + (cc >> 3) * kHalf + half_chunk_offset(n, cc & 7)) = make_uint4(w[0], w[1], w[2], w[3]);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  // epilogue of one tile: this thread's half row (row r, columns 64 h .. 64 h + 63) out of accumulator `buf`
  const int r = (warp & 3) * 32 + (tid & 31), h = warp >> 2;
  auto quantize_tile = [&](int tile, int buf) {
    int64_t first;
    const int here = tile_rows(tile, &first);
    const uint32_t t_row = tmem + 128 * buf + ((uint32_t)((warp & 3) * 32) << 16) + 64 * h;
    uint32_t sf = 0;
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      uint32_t acc[32];
      TMEM_LD32(t_row + 32 * u, acc);
      tmem_ld_wait();
      float y[32], mf = 0.0f;
#pragma unroll
      for (int i = 0; i < 32; ++i) {
        y[i] = __fmul_rn(__uint_as_float(acc[i]), 0.08838834764831845f);
        mf = fmaxf(mf, fabsf(y[i]));
      }
      const int e = kRuleKind == 2 ? shared_exponent_ceil(__float_as_uint(mf), rule) : shared_exponent(__float_as_uint(mf), kRuleKind == 1);
      const float inv = pow2_neg(e);
      uint32_t wd[4];
#pragma unroll
      for (int g = 0; g < 4; ++g)
        wd[g] = pack_e2m1x8(y[8 * g] * inv, y[8 * g + 1] * inv, y[8 * g + 2] * inv, y[8 * g + 3] * inv,
                            y[8 * g + 4] * inv, y[8 * g + 5] * inv, y[8 * g + 6] * inv, y[8 * g + 7] * inv);
      sf |= (uint32_t)(e + 127) << (8 * u);
      const int blk = 2 * h + u;
      if (kTileLayout)
        *reinterpret_cast<uint4*>(codes + (int64_t)tile * kTileCodeBytes + tile_code_offset(r, blk)) = make_uint4(wd[0], wd[1], wd[2], wd[3]);
      else if (r < here)
        *reinterpret_cast<uint4*>(codes + (first + r) * 64 + 16 * blk) = make_uint4(wd[0], wd[1], wd[2], wd[3]);
    }
    if (kTileLayout)
      *reinterpret_cast<uint16_t*>(scales + (int64_t)tile * kTileScaleBytes + tile_scale_offset(r, 2 * h)) = (uint16_t)sf;
    else if (r < here)
      *reinterpret_cast<uint16_t*>(scales + (first + r) * 4 + 2 * h) = (uint16_t)sf;
  };

  bool ok = true;
  for (int i = 0; i < n_my && ok; ++i) {
    const int tile = (int)blockIdx.x + i * (int)gridDim.x;
    if (i > 0) {                                       // the product of tile i - 1 is complete: its X buffer is free, its accumulator full
      ok = __all_sync(0xFFFFFFFFu, mbar_wait(bar0 + 8 * ((i - 1) & 1), (uint32_t)(((i - 1) >> 1) & 1), abort_flag, &g_status, 51));
      if (!ok) break;
      tc_fence_after();
    }
    if (i + 1 < n_my) {                                // fetch tile i + 1 as early as its buffer allows
      fetch(tile + (int)gridDim.x, (i + 1) & 1);
      asm volatile("cp.async.wait_group 1;" ::: "memory");        // X(i) has landed; X(i + 1) stays in flight
    } else {
      asm volatile("cp.async.wait_group 0;" ::: "memory");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    tc_fence_before();
    __syncthreads();                                               // X(i) is there for every thread; accumulator i & 1 has been read out
    tc_fence_after();
    if (tid == 0) {
      constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);     // 8-row groups 1024 B apart, 128-byte swizzle
      constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);   // fp32 accumulate, bf16 x bf16, N = 128, M = 128
      const uint32_t a = (sbase + (i & 1) * 2 * kHalf) >> 4, b = (sbase + kOffH) >> 4;
#pragma unroll
      for (int k = 0; k < 8; ++k) {                    // K = 16 per instruction: 4 steps of 32 bytes per 64-element half
        const uint32_t off = (uint32_t)(k >> 2) * (kHalf >> 4) + (uint32_t)(k & 3) * 2;
        asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                     "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                     ::"r"(tmem + 128 * (i & 1)), "l"(((uint64_t)kDescHi << 32) | (a + off)), "l"(((uint64_t)kDescHi << 32) | (b + off)),
                       "r"(kIdesc), "r"(k > 0 ? 1u : 0u) : "memory");
      }
      tc_commit(bar0 + 8 * (i & 1));
    }
    if (i > 0) quantize_tile(tile - (int)gridDim.x, (i - 1) & 1);
  }
  if (ok && n_my > 0) {
    ok = __all_sync(0xFFFFFFFFu, mbar_wait(bar0 + 8 * ((n_my - 1) & 1), (uint32_t)(((n_my - 1) >> 1) & 1), abort_flag, &g_status, 51));
    if (ok) {
      tc_fence_after();
      quantize_tile((int)blockIdx.x + (n_my - 1) * (int)gridDim.x, (n_my - 1) & 1);
    }
  }
  asm volatile("cp.async.wait_group 0;" ::: "memory");
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 256;" ::"r"(tmem) : "memory");
  }
}
}  // namespace rot

// ------------------------------------------------------------------------------------------
// Axis 0.  256 threads; a CTA stages a 32 KiB slab of the input in shared memory, by asynchronous 16-byte copies
// (cp.async: no staging registers and no second pass through the load/store unit; against loads to registers
// followed by shared-memory stores this took the canonical layout from 0.77 / 0.84 / 0.88 of the plain-copy rate to
// 0.89 / 0.97 / 1.02 at 2^26 / 2^27 / 2^28 elements):
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
    // asynchronous 16-byte copy straight into shared memory; nothing is read (and zeros are written) beyond the edges
    const bool inside = row0 + t < rows && col0 + cc < cols;
    const uint16_t* g = inside ? src + (row0 + t) * cols + col0 + cc : src;
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"((uint32_t)__cvta_generic_to_shared(&s_in[t][cc])), "l"(g), "r"(inside ? 16 : 0) : "memory");
  }
  asm volatile("cp.async.wait_all;" ::: "memory");
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
// persistent grid of the rotating quantizer: two CTAs per SM
static int rot_grid() {
  static int n = 0;
  if (n == 0) {
    int dev = 0, v = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) v = 148;
    n = 2 * v;
  }
  return n;
}

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
      if (rows_pad / kTile > 0x3FFFFFFF || batch > 65535) return MXATTN_EUNSUPPORTED;
      dim3 grid((unsigned)(2 * (rows_pad / kTile)), (unsigned)batch);       // the plain tile kernel takes half a tile per CTA
      if (rotate) {
        auto kern = rule == kRuleOcp ? rot::quantize_axis1_rot_tc_kernel<true, 0>
                  : rule == kRuleUos ? rot::quantize_axis1_rot_tc_kernel<true, 1> : rot::quantize_axis1_rot_tc_kernel<true, 2>;
        const int64_t n_tiles = batch * (rows_pad / kTile);
        if (n_tiles > 0x7FFFFFFF) return MXATTN_EUNSUPPORTED;
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, rot::kSmemBytes) != cudaSuccess) return MXATTN_ECUDA;
        kern<<<(unsigned)min((int64_t)rot_grid(), n_tiles), rot::kThreads, rot::kSmemBytes, stream>>>(
            (const uint4*)in, (uint8_t*)codes, (uint8_t*)scales, rows, (int)(rows_pad / kTile), (int)n_tiles, rule);
      } else
        quantize_axis1_tile_kernel<<<grid, kQThreads, 0, stream>>>((const uint4*)in, (uint8_t*)codes,
                                                                          (uint8_t*)scales, rows, rule);
    } else {
      if (rotate) {                                  // cols == 128 here: batch * rows rows of 16 chunks
        const int64_t groups = (batch * rows + kTile - 1) / kTile;
        if (groups > 0x7FFFFFFF) return MXATTN_EUNSUPPORTED;
        auto kern = rule == kRuleOcp ? rot::quantize_axis1_rot_tc_kernel<false, 0>
                  : rule == kRuleUos ? rot::quantize_axis1_rot_tc_kernel<false, 1> : rot::quantize_axis1_rot_tc_kernel<false, 2>;
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, rot::kSmemBytes) != cudaSuccess) return MXATTN_ECUDA;
        kern<<<(unsigned)min((int64_t)rot_grid(), groups), rot::kThreads, rot::kSmemBytes, stream>>>(
            (const uint4*)in, (uint8_t*)codes, (uint8_t*)scales, batch * rows, (int)groups, (int)groups, rule);
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

extern "C" int mxattn_quantizer_status(int* host_out, void* stream) {
  if (!host_out) return MXATTN_EINVAL;
  if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return MXATTN_ECUDA;
  if (cudaMemcpyFromSymbol(host_out, mxattn::rot::g_status, sizeof(int)) != cudaSuccess) return MXATTN_ECUDA;
  return MXATTN_OK;
}
