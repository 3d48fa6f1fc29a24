// bf16 variant of the fused attention forward: the same CTA structure, pipeline and online-softmax
// recurrence (paper Section 2, the FlashAttention-2 form: Eq. 2-3) as the MXFP4 kernel in forward.cu,
// with NO quantization: Q, K, V stay bf16, the exponentials are rounded to bf16 for the second GEMM,
// and the row sum is taken from the fp32 exponentials.  It is the "high precision" reference point
// the MXFP4 variants are reported against (paper Section 5.2, "FP16" baseline; bf16 here).
//
//   GEMM 1  S   = Q_t K_j^T          tcgen05.mma kind::f16, M=128, N=128, 8 instructions of K=16
//   GEMM 2  O_t += P_t V_j           same shape; V is staged transposed (K-major), like the FP4 path
//
// Operands are K-major tiles of two 64-element K halves, each half [128 rows x 128 bytes] with the
// 128-byte swizzle; a tile image is 32 KiB and is produced by pack_bf16_tiles_kernel so that one bulk
// copy brings it into shared memory.  Shared memory: Q 2 x 32, K 2 x 32, V 1 x 32, P 2 x 32 KiB.
// Tensor memory: S [0,128) shared by both softmax groups, O_0 [128,256), O_1 [256,384).
#include <type_traits>

#include "common.cuh"
#include "tc_helpers.cuh"

namespace mxattn {
namespace fwd16 {

using namespace fwd;

constexpr int kThreads = 576;
constexpr int kSoftmaxWarps = 16;
constexpr int kKStages = 2;
constexpr int kTileBytes = 32768;                          // 128 x 128 bf16
constexpr int kHalfBytes = 16384;

constexpr int kOffQ = 0;                                   // 2 tiles
constexpr int kOffK = kOffQ + 2 * kTileBytes;              // 2 stages
constexpr int kOffV = kOffK + kKStages * kTileBytes;       // 1 stage
constexpr int kOffP = kOffV + kTileBytes;                  // 2 tiles
constexpr int kOffBar = kOffP + 2 * kTileBytes;
enum Bar { BAR_Q = 0, BAR_KFULL = 1, BAR_KEMPTY = 3, BAR_VFULL = 5, BAR_VEMPTY = 6, BAR_SFULL = 7, BAR_SFREE = 9,
           BAR_PFULL = 10, BAR_ODONE = 12, kNumBars = 14 };
constexpr int kOffMisc = kOffBar + kNumBars * 8;
constexpr int kOffMax = kOffMisc + 32;                     // half-row maxima [parity 2][tile 2][half 2][128]... halved: see below
constexpr int kSmemBytes = kOffMax + 2 * 2 * 128 * 4;      // single-buffered exchange (2 tiles x 2 halves x 128 floats)
static_assert(kSmemBytes <= 232448, "shared memory budget");

constexpr uint32_t kColS = 0, kColO0 = 128, kColO1 = 256;

__device__ __forceinline__ void tc_mma_f16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
               "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
               ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}

// byte offset of the 16-byte chunk c (0..7) of row r inside a 16 KiB half tile (128-byte swizzle)
__device__ __forceinline__ int half_chunk_offset(int r, int c) { return r * 128 + ((c ^ (r & 7)) << 4); }

struct Params {
  const uint8_t* q_tiles; const uint8_t* k_tiles; const uint8_t* v_tiles;
  void* out;
  int* status;
  int64_t Nq, Nkv;
  int q_tiles_n, kv_tiles, q_pairs;
  float scale_log2e;
};

// ---------------------------------------------------------------------------------------------
// bf16 [batch][rows,128] -> tile images.  axis 1: rows stay rows (Q, K).  axis 0: transposed, the
// 128 columns become the tile's rows and 128 consecutive input rows its K extent (V).
template <int kAxis>
__global__ void __launch_bounds__(256) pack_bf16_tiles_kernel(const uint16_t* __restrict__ in, uint8_t* __restrict__ tiles,
                                                              int64_t rows) {
  const int tid = threadIdx.x;
  const int64_t tile = (int64_t)blockIdx.y * gridDim.x + blockIdx.x;
  const int64_t row0 = (int64_t)blockIdx.x * kTile;
  const uint16_t* src = in + ((int64_t)blockIdx.y * rows + row0) * kHeadDim;
  const int rows_here = (int)min((int64_t)kTile, rows - row0);
  uint8_t* dst = tiles + tile * kTileBytes;
  if (kAxis == 1) {
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const int chunk = k * 256 + tid;                 // 16 chunks of 8 bf16 per row
      const int r = chunk >> 4, cc = chunk & 15;
      uint4 v = make_uint4(0u, 0u, 0u, 0u);
      if (r < rows_here) v = __ldg(reinterpret_cast<const uint4*>(src + (int64_t)r * kHeadDim) + cc);
      *reinterpret_cast<uint4*>(dst + (cc >> 3) * kHalfBytes + half_chunk_offset(r, cc & 7)) = v;
    }
  } else {
    __shared__ __align__(16) uint16_t s_in[kTile][kTile + 8];     // [token][channel], padded rows
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const int chunk = k * 256 + tid;
      const int t = chunk >> 4, cc = (chunk & 15) << 3;
      uint4 v = make_uint4(0u, 0u, 0u, 0u);
      if (t < rows_here) v = __ldg(reinterpret_cast<const uint4*>(src + (int64_t)t * kHeadDim + cc));
      *reinterpret_cast<uint4*>(&s_in[t][cc]) = v;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const int job = k * 256 + tid;                   // (channel n, token chunk tc of 8 tokens)
      const int n = job & 127, tc = job >> 7;
      uint32_t w[4];
#pragma unroll
      for (int i = 0; i < 4; ++i)
        w[i] = (uint32_t)s_in[tc * 8 + 2 * i][n] | ((uint32_t)s_in[tc * 8 + 2 * i + 1][n] << 16);
      *reinterpret_cast<uint4*>(dst + (tc >> 3) * kHalfBytes + half_chunk_offset(n, tc & 7)) = make_uint4(w[0], w[1], w[2], w[3]);
    }
  }
}

// ---------------------------------------------------------------------------------------------
template <bool kOutF32>
__global__ void __launch_bounds__(kThreads, 1) attention_bf16_kernel(const Params p) {
  extern __shared__ __align__(1024) uint8_t smem[];
  const uint32_t sbase = smem_u32(smem);
  const uint32_t bar0 = sbase + kOffBar;
  auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + kOffMisc);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + kOffMisc + 8);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (*reinterpret_cast<volatile int*>(p.status) != 0) return;
  if ((sbase & 1023u) != 0u) {                       // the swizzled tiles need a 1024-byte aligned base
    if (tid == 0) atomicCAS(p.status, 0, 41);
    return;
  }
  const int bh = blockIdx.x / p.q_pairs;
  const int pair = blockIdx.x - bh * p.q_pairs;
  const int T = p.kv_tiles;

  if (tid == 0) {
    mbar_init(bar(BAR_Q), 1);
    for (int s = 0; s < kKStages; ++s) { mbar_init(bar(BAR_KFULL + s), 1); mbar_init(bar(BAR_KEMPTY + s), 1); }
    mbar_init(bar(BAR_VFULL), 1); mbar_init(bar(BAR_VEMPTY), 1);
    mbar_init(bar(BAR_SFULL + 0), 1); mbar_init(bar(BAR_SFULL + 1), 1);
    mbar_init(bar(BAR_SFREE), 8);
    mbar_init(bar(BAR_PFULL + 0), 8); mbar_init(bar(BAR_PFULL + 1), 8);
    mbar_init(bar(BAR_ODONE + 0), 1); mbar_init(bar(BAR_ODONE + 1), 1);
    abort_flag[0] = 0;
    abort_flag[1] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == kSoftmaxWarps + 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(tmem_slot)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  if (warp == kSoftmaxWarps) {
    // =============================== producer ===============================================
    if (lane == 0) {
      const int64_t qt0 = (int64_t)bh * p.q_tiles_n + 2 * pair;
      const int64_t qt1 = (2 * pair + 1 < p.q_tiles_n) ? qt0 + 1 : qt0;
      mbar_expect_tx(bar(BAR_Q), 2 * kTileBytes);
      bulk_g2s(sbase + kOffQ, p.q_tiles + qt0 * kTileBytes, kTileBytes, bar(BAR_Q));
      bulk_g2s(sbase + kOffQ + kTileBytes, p.q_tiles + qt1 * kTileBytes, kTileBytes, bar(BAR_Q));
      const int64_t kv0 = (int64_t)bh * T;
      int k_issued = 0, v_issued = 0;
      bool ok = true;
      auto issue_k = [&](int j) {
        const int s = j % kKStages;
        mbar_expect_tx(bar(BAR_KFULL + s), kTileBytes);
        bulk_g2s(sbase + kOffK + s * kTileBytes, p.k_tiles + (kv0 + j) * kTileBytes, kTileBytes, bar(BAR_KFULL + s));
        k_issued = j + 1;
      };
      issue_k(0);
      if (T > 1) issue_k(1);
      for (int j = 0; j < T && ok; ++j) {              // order K0 K1 V0 K2 V1 K3 ...: K never queues behind V
        if (j >= 1) ok = mbar_wait(bar(BAR_VEMPTY), (uint32_t)((j - 1) & 1), abort_flag, p.status, 12);
        if (!ok) break;
        mbar_expect_tx(bar(BAR_VFULL), kTileBytes);
        bulk_g2s(sbase + kOffV, p.v_tiles + (kv0 + j) * kTileBytes, kTileBytes, bar(BAR_VFULL));
        v_issued = j + 1;
        if (j + 2 < T) {
          ok = mbar_wait(bar(BAR_KEMPTY + j % kKStages), (uint32_t)((j / kKStages) & 1), abort_flag, p.status, 11);
          if (!ok) break;
          issue_k(j + 2);
        }
      }
      if (!ok || *abort_flag) {                       // let copies in flight land before shared memory is released
        const long long t0 = clock64();
        for (int j = (k_issued > kKStages ? k_issued - kKStages : 0); j < k_issued; ++j)
          while (!mbar_try(bar(BAR_KFULL + j % kKStages), (uint32_t)((j / kKStages) & 1)) && clock64() - t0 < 400000000LL) {}
        if (v_issued > 0)
          while (!mbar_try(bar(BAR_VFULL), (uint32_t)((v_issued - 1) & 1)) && clock64() - t0 < 400000000LL) {}
        while (!mbar_try(bar(BAR_Q), 0) && clock64() - t0 < 400000000LL) {}
      }
    }
  } else if (warp == kSoftmaxWarps + 1) {
    // =============================== MMA issuer =============================================
    if (lane == 0) {
      bool ok = mbar_wait(bar(BAR_Q), 0, abort_flag, p.status, 21);
      uint32_t sfree_n = 0;
      constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);     // 8-row groups 1024 B apart, 128-byte swizzle
      constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);  // f32 accum, bf16 x bf16, N=128, M=128
      const uint32_t q_lo = (sbase + kOffQ) >> 4, k_lo = (sbase + kOffK) >> 4, v_lo = (sbase + kOffV) >> 4, p_lo = (sbase + kOffP) >> 4;
      auto gemm = [&](uint32_t d, uint32_t a, uint32_t b, bool accumulate) {
#pragma unroll
        for (int k = 0; k < 8; ++k) {                  // K = 16 per instruction: 4 steps of 32 bytes per 64-element half
          const uint32_t off = (uint32_t)(k >> 2) * (kHalfBytes >> 4) + (uint32_t)(k & 3) * 2;
          tc_mma_f16(d, ((uint64_t)kDescHi << 32) | (a + off), ((uint64_t)kDescHi << 32) | (b + off), kIdesc,
                     (accumulate || k > 0) ? 1u : 0u);
        }
      };
      auto gemm1 = [&](int t, int j) {
        gemm(tmem + kColS, q_lo + (uint32_t)t * (kTileBytes >> 4), k_lo + (uint32_t)(j % kKStages) * (kTileBytes >> 4), false);
        tc_commit(bar(BAR_SFULL + t));
      };
      auto gemm2 = [&](int t, int j) {
        gemm(tmem + (t ? kColO1 : kColO0), p_lo + (uint32_t)t * (kTileBytes >> 4), v_lo, j > 0);
        tc_commit(bar(BAR_ODONE + t));
      };
      auto wait_k = [&](int j) {
        const bool r = mbar_wait(bar(BAR_KFULL + j % kKStages), (uint32_t)((j / kKStages) & 1), abort_flag, p.status, 22);
        tc_fence_after();
        return r;
      };
      auto wait_sfree = [&]() {
        const bool r = mbar_wait(bar(BAR_SFREE), sfree_n & 1u, abort_flag, p.status, 23);
        ++sfree_n;
        tc_fence_after();
        return r;
      };
      if (ok) tc_fence_after();
      ok = ok && wait_k(0);
      if (ok) gemm1(0, 0);
      ok = ok && wait_sfree();
      if (ok) { gemm1(1, 0); tc_commit(bar(BAR_KEMPTY + 0)); }
      if (T > 1) {
        ok = ok && wait_k(1);
        ok = ok && wait_sfree();
        if (ok) gemm1(0, 1);
      }
      for (int j = 0; j < T && ok; ++j) {
        ok = mbar_wait(bar(BAR_PFULL + 0), (uint32_t)(j & 1), abort_flag, p.status, 24);
        ok = ok && mbar_wait(bar(BAR_VFULL), (uint32_t)(j & 1), abort_flag, p.status, 25);
        if (!ok) break;
        tc_fence_after();
        gemm2(0, j);
        if (j + 1 < T) {
          ok = wait_sfree();
          if (!ok) break;
          gemm1(1, j + 1);
          tc_commit(bar(BAR_KEMPTY + (j + 1) % kKStages));
        }
        ok = mbar_wait(bar(BAR_PFULL + 1), (uint32_t)(j & 1), abort_flag, p.status, 26);
        if (!ok) break;
        tc_fence_after();
        gemm2(1, j);
        tc_commit(bar(BAR_VEMPTY));
        if (j + 2 < T) {
          ok = wait_k(j + 2);
          ok = ok && wait_sfree();
          if (!ok) break;
          gemm1(0, j + 2);
        }
      }
    }
  } else if (warp < kSoftmaxWarps) {
    // =============================== softmax groups =========================================
    const int t = warp >> 3;
    const int h = (warp >> 2) & 1;
    const int row = (warp & 3) * 32 + lane;
    const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t t_s = tmem + kColS + lane_addr + 64 * h;
    const uint32_t t_o = tmem + (t ? kColO1 : kColO0) + lane_addr;
    const float c = p.scale_log2e;
    float m_run = -INFINITY, l_run = 0.0f;
    uint8_t* sP = smem + kOffP + t * kTileBytes + h * kHalfBytes;       // this thread's keys are one K half of P
    float* sMax = reinterpret_cast<float*>(smem + kOffMax) + t * 256;
    const int pair_bar = 1 + (warp & 3) + 4 * t;
    // the two warps of a pair meet at named barriers (twice per tile, twice in the epilogue); a warp whose bounded wait
    // has run out keeps the remaining appointments (pair_keep_company) so that its partner is never stranded.  Their
    // waits give up only on their own cycle limit: they watch a flag that nothing sets and raise the CTA's
    volatile int* const own_limit_only = abort_flag + 1;
    bool ok = true;

    int j = 0;                                       // after the loop: the first tile whose two meetings have not been kept
    for (; j < T; ++j) {
      ok = __all_sync(0xFFFFFFFFu, mbar_wait(bar(BAR_SFULL + t), (uint32_t)(j & 1), own_limit_only, p.status, 31, kWaitLimitCycles, abort_flag));
      if (!ok) break;
      tc_fence_after();
      uint32_t sr[64];
      TMEM_LD32(t_s + 0, (sr + 0));
      TMEM_LD32(t_s + 32, (sr + 32));
      tmem_ld_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(BAR_SFREE));

      if (j == T - 1) {
        const int valid = (int)(p.Nkv - (int64_t)j * kTile) - 64 * h;
#pragma unroll
        for (int i = 0; i < 64; ++i)
          if (i >= valid) sr[i] = 0xFF800000u;
      }
      float q8[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const uint32_t* v = sr + 8 * u;
        float mx = max3(__uint_as_float(v[0]), __uint_as_float(v[1]), __uint_as_float(v[2]));
        mx = max3(mx, __uint_as_float(v[3]), __uint_as_float(v[4]));
        mx = max3(mx, __uint_as_float(v[5]), __uint_as_float(v[6]));
        q8[u] = fmaxf(mx, __uint_as_float(v[7]));
      }
      const float hmax = fmaxf(max3(q8[0], q8[1], q8[2]), max3(max3(q8[3], q8[4], q8[5]), q8[6], q8[7]));
      // exchange with the partner thread; the two barriers per tile make the single buffer safe
      asm volatile("bar.sync %0, 64;" ::"r"(pair_bar) : "memory");
      sMax[h * 128 + row] = hmax;
      const bool o_ready = (j == 0) || mbar_test(bar(BAR_ODONE + t), (uint32_t)((j - 1) & 1));
      asm volatile("bar.sync %0, 64;" ::"r"(pair_bar) : "memory");
      const float m_new = max3(m_run, hmax, sMax[(h ^ 1) * 128 + row]);
      const bool moved = (m_new != m_run) && (j > 0);
      const float m_old = m_run;
      m_run = m_new;
      const float nmc = -(m_new * c);
      if (!__all_sync(0xFFFFFFFFu, o_ready)) {
        ok = __all_sync(0xFFFFFFFFu, mbar_wait(bar(BAR_ODONE + t), (uint32_t)((j - 1) & 1), own_limit_only, p.status, 32, kWaitLimitCycles, abort_flag));
        if (!ok) { ++j; break; }
      }
      tc_fence_after();
      const bool rescale = __any_sync(0xFFFFFFFFu, moved);
      float alpha = 1.0f;
      float l_tile = 0.0f;
      auto tile_body = [&](auto resc_tag) {
        constexpr bool kResc = decltype(resc_tag)::value;
        if (kResc) alpha = ex2((m_old - m_new) * c);
#pragma unroll
        for (int g = 0; g < 8; ++g) {                  // 8 keys per step = one 16-byte chunk of bf16
          uint32_t oc[8];
          const uint32_t t_oc = t_o + 64 * h + 8 * g;
          if (kResc) TMEM_LD8(t_oc, oc);
          float x[8];
#pragma unroll
          for (int i = 0; i < 8; ++i) x[i] = ex2(fmaf(__uint_as_float(sr[8 * g + i]), c, nmc));
          l_tile += ((x[0] + x[1]) + (x[2] + x[3])) + ((x[4] + x[5]) + (x[6] + x[7]));
          uint32_t w[4];
#pragma unroll
          for (int i = 0; i < 4; ++i) asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(w[i]) : "f"(x[2 * i + 1]), "f"(x[2 * i]));
          *reinterpret_cast<uint4*>(sP + half_chunk_offset(row, g)) = make_uint4(w[0], w[1], w[2], w[3]);
          if (kResc) {
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 8; ++i) oc[i] = __float_as_uint(__uint_as_float(oc[i]) * alpha);
            TMEM_ST8(t_oc, oc);
          }
        }
        if (kResc) tmem_st_wait();
      };
      if (rescale) tile_body(std::true_type{}); else tile_body(std::false_type{});
      l_run = fmaf(alpha, l_run, l_tile);
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(BAR_PFULL + t));
    }

    if (!ok) pair_keep_company(pair_bar, 2 * (T - j));
    if (ok) ok = __all_sync(0xFFFFFFFFu, mbar_wait(bar(BAR_ODONE + t), (uint32_t)((T - 1) & 1), own_limit_only, p.status, 33, kWaitLimitCycles, abort_flag));
    asm volatile("bar.sync %0, 64;" ::"r"(pair_bar) : "memory");
    sMax[h * 128 + row] = l_run;
    asm volatile("bar.sync %0, 64;" ::"r"(pair_bar) : "memory");
    const float l = l_run + sMax[(h ^ 1) * 128 + row];
    if (ok) {
      tc_fence_after();
      const int qtile = 2 * pair + t;
      const int64_t grow = (int64_t)qtile * kTile + row;
      const bool store = (qtile < p.q_tiles_n) && (grow < p.Nq);
      const float inv_l = 1.0f / l;
      const int64_t obase = ((int64_t)bh * p.Nq + grow) * kHeadDim + 64 * h;
#pragma unroll 1
      for (int c0 = 0; c0 < 64; c0 += 32) {
        uint32_t r32[32];
        TMEM_LD32(t_o + 64 * h + c0, r32);
        tmem_ld_wait();
        if (store) {
          if (kOutF32) {
            float4* dst = reinterpret_cast<float4*>(static_cast<float*>(p.out) + obase + c0);
#pragma unroll
            for (int i = 0; i < 8; ++i)
              dst[i] = make_float4(__uint_as_float(r32[4 * i]) * inv_l, __uint_as_float(r32[4 * i + 1]) * inv_l,
                                   __uint_as_float(r32[4 * i + 2]) * inv_l, __uint_as_float(r32[4 * i + 3]) * inv_l);
          } else {
            uint4* dst = reinterpret_cast<uint4*>(static_cast<uint16_t*>(p.out) + obase + c0);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              uint32_t hh[4];
#pragma unroll
              for (int k = 0; k < 4; ++k) {
                const float a = __uint_as_float(r32[8 * i + 2 * k]) * inv_l, b2 = __uint_as_float(r32[8 * i + 2 * k + 1]) * inv_l;
                asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(hh[k]) : "f"(b2), "f"(a));
              }
              dst[i] = make_uint4(hh[0], hh[1], hh[2], hh[3]);
            }
          }
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == kSoftmaxWarps + 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");
  }
}

}  // namespace fwd16

size_t bf16_workspace_bytes(int B, int H, int64_t Nq, int64_t Nkv) {
  const size_t bh = (size_t)B * H;
  const size_t qt = (size_t)((Nq + kTile - 1) / kTile), kt = (size_t)((Nkv + kTile - 1) / kTile);
  return 256 + bh * (qt + 2 * kt) * fwd16::kTileBytes;
}

int launch_forward_bf16(const void* q, const void* k, const void* v, void* o, int B, int H, int64_t Nq, int64_t Nkv,
                        float softmax_scale, unsigned flags, void* workspace, size_t workspace_bytes, cudaStream_t stream) {
  using namespace fwd16;
  if (workspace_bytes < bf16_workspace_bytes(B, H, Nq, Nkv)) return MXATTN_EWORKSPACE;
  const int64_t bh = (int64_t)B * H;
  const int64_t qt = (Nq + kTile - 1) / kTile, kt = (Nkv + kTile - 1) / kTile;
  const int64_t pairs = (qt + 1) / 2, grid = bh * pairs;
  if (qt > 0x3FFFFFFF || kt > 65535 || qt > 0x7FFFFFFF || bh > 65535 || grid > 0x7FFFFFFF) return MXATTN_EUNSUPPORTED;
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  uint8_t* qtiles = ws + 256;
  uint8_t* ktiles = qtiles + (size_t)bh * qt * kTileBytes;
  uint8_t* vtiles = ktiles + (size_t)bh * kt * kTileBytes;
  if (cudaMemsetAsync(ws, 0, 16, stream) != cudaSuccess) return MXATTN_ECUDA;
  pack_bf16_tiles_kernel<1><<<dim3((unsigned)qt, (unsigned)bh), 256, 0, stream>>>((const uint16_t*)q, qtiles, Nq);
  pack_bf16_tiles_kernel<1><<<dim3((unsigned)kt, (unsigned)bh), 256, 0, stream>>>((const uint16_t*)k, ktiles, Nkv);
  pack_bf16_tiles_kernel<0><<<dim3((unsigned)kt, (unsigned)bh), 256, 0, stream>>>((const uint16_t*)v, vtiles, Nkv);
  Params p;
  p.q_tiles = qtiles; p.k_tiles = ktiles; p.v_tiles = vtiles; p.out = o; p.status = reinterpret_cast<int*>(ws);
  p.Nq = Nq; p.Nkv = Nkv; p.q_tiles_n = (int)qt; p.kv_tiles = (int)kt; p.q_pairs = (int)pairs;
  p.scale_log2e = softmax_scale * 1.4426950408889634f;
  void (*kern)(const Params) = (flags & MXATTN_FLAG_OUT_FP32) ? attention_bf16_kernel<true> : attention_bf16_kernel<false>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess) return MXATTN_ECUDA;
  kern<<<(unsigned)grid, kThreads, kSmemBytes, stream>>>(p);
  count_launch(4);
  return cudaGetLastError() == cudaSuccess ? MXATTN_OK : MXATTN_ECUDA;
}

}  // namespace mxattn
