// NVFP4 variant of the fused attention forward: the paper's comparison baseline "NVFP4" (Section 5.2) -- Q, K, V and
// the softmax tile in NVFP4 (E2M1 in blocks of 16, E4M3 block scale, fp32 tensor scale), nothing else changed -- run by
// the same CTA structure, pipeline and online-softmax recurrence as the MXFP4 kernel in forward.cu (Algorithm 2 with
// the quantizer exchanged), so that the two formats can be compared at equal kernel design.
//
//   GEMM 1  S_raw = Q-hat_t K-hat_j^T            tcgen05.mma kind::mxf4nvf4, block16, UE4M3 scales; M = 128, N = 128
//   GEMM 2  O_t  += P-hat_t [V-hat_j | 1]        N = 144: the 16 extra rows hold the constant 1 (code 2, scale 1.0),
//                                                so column 128 accumulates the row sum of the quantized probabilities
// The tensor-level scales are applied outside the tensor core: S = S_raw * s_T(Q) s_T(K) * softmax_scale (folded into
// the exponent's multiplier), O = O_raw * s_T(V) * s_T(P) / l with s_T(P) = fl32(1/2688) (the softmax tile's maximum
// is known to be 1); under PNQ l = l_raw * s_T(P) and s_T(P) cancels.
//
// Per KV tile a softmax thread (two threads per query row, 64 key columns = 4 blocks of 16 each):
//   per block: M = its largest p = exp2(s_max * c - m_new * c), d = E4M3(fl32(fl32(M * 2688) * fl32(1/6))), scale byte = d
//   per element: codes = E2M1(exp2(s_i * c - m_new * c + log2(2688 / d)))      half a packed fma + one ex2
// which is the library's NVFP4 recipe (include/mxattn.h) with the tensor maximum 1, the element multiplier
// r = 2688 / d folded into the exponent (the recipe's fl32(p_i * r) differs from this by about 2e-7 relative, the order
// of ex2.approx itself; a block with d = 0 keeps r = 1, its codes are 0 either way).
//
// One CTA per work item (two query tiles of one head); outputs are stored from registers.  Tensor-memory map:
// S [0,128), O_0 [128,272), O_1 [272,416), scale factors from 416 (8 columns per operand tile: two atoms).
// Every mbarrier wait is bounded; a softmax warp that gives up keeps its partner's appointments (tc_helpers.cuh).
#include <cuda_fp16.h>

#include <type_traits>

#include "common.cuh"
#include "tc_helpers.cuh"

namespace mxattn {
namespace fwdnv {
using namespace fwd;

constexpr int kCols = 64;                        // key columns per softmax thread
constexpr int kSoftmaxWarps = 16;
constexpr int kThreads = 32 * (kSoftmaxWarps + 2);
constexpr int kStages = 4;
constexpr int kNV = 144;
constexpr int kVStageBytes = kNV * 64;
constexpr int kSF = 2 * kTileScaleBytes;         // scale bytes per operand tile: two atoms (8 blocks of 16 per row)

constexpr int kOffQ = 0;                                   // 2 tiles
constexpr int kOffK = kOffQ + 2 * kTileCodeBytes;          // 4 stages
constexpr int kOffV = kOffK + kStages * kTileCodeBytes;    // 4 stages of 144 rows
constexpr int kOffP = kOffV + kStages * kVStageBytes;      // 2 tiles
constexpr int kOffSFQ = kOffP + 2 * kTileCodeBytes;        // 2 x 1024
constexpr int kOffSFK = kOffSFQ + 2 * kSF;                 // 4 x 1024
constexpr int kOffSFV = kOffSFK + kStages * kSF;           // 4 x 1024
constexpr int kOffSFOnes = kOffSFV + kStages * kSF;        // 512 (one atom serves both K halves)
constexpr int kOffSFP = kOffSFOnes + kTileScaleBytes;      // 2 x 1024
constexpr int kOffBar = kOffSFP + 2 * kSF;
enum Bar { BAR_Q = 0, BAR_KFULL = 1, BAR_KEMPTY = BAR_KFULL + kStages, BAR_SFULL = BAR_KEMPTY + kStages, BAR_SFREE = BAR_SFULL + 2,
           BAR_PFULL = BAR_SFREE + 1, BAR_ODONE = BAR_PFULL + 2, kNumBars = BAR_ODONE + 2 };
constexpr int kOffMisc = kOffBar + kNumBars * 8;
constexpr int kOffMax = kOffMisc + 64;                     // half-row exchange: [parity 2][tile 2][half 2][128] floats
constexpr int kSmemBytes = kOffMax + 2 * 2 * 2 * 128 * 4 + 1024;
static_assert(kSmemBytes <= 227 * 1024, "shared memory per CTA");

// tensor-memory columns: per operand tile 8 scale columns (atom of K half 0, atom of K half 1); a V slot interleaves
// the atoms of the ones rows: [V half 0][ones][V half 1][ones]
constexpr uint32_t kColS = 0, kColO0 = 128, kColO1 = 272, kColSFQ = 416, kColSFK = 432, kColSFV = 448, kColSFP = 480;

constexpr float kTensorRangeP = 2688.0f;                   // 448 * 6: encode scale of the softmax tile (tensor maximum 1)
constexpr float kOneSixth = 0.16666667163372040f;          // fl32(1/6)
constexpr float kInvTensorRangeP = 3.7202381e-4f;          // fl32(1/2688)

struct Params {
  const uint8_t* q_codes; const uint8_t* q_scales;
  const uint8_t* k_codes; const uint8_t* k_scales;
  const uint8_t* v_codes; const uint8_t* v_scales;
  const float* ts_q; const float* ts_k; const float* ts_v;   // tensor decode scales, one per head
  void* out;
  int* status;
  int64_t Nq, Nkv;
  int q_tiles, kv_tiles, q_pairs;
  float scale_log2e;
};

// instruction descriptor of kind::mxf4nvf4.block_scale.block16: A, B = E2M1 (K-major), scales UE4M3, M = 128
__device__ __forceinline__ constexpr uint32_t make_idesc_nv(int n) {
  return (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((128u >> 4) << 24);
}
__device__ __forceinline__ void tc_mma_nv(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t sfa, uint32_t sfb, uint32_t accumulate) {
  asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
               "tcgen05.mma.cta_group::1.kind::mxf4nvf4.block_scale.block16 [%0], %1, %2, %3, [%5], [%6], p;\n\t}"
               ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(sfa), "r"(sfb) : "memory");
}
__device__ __forceinline__ uint32_t e4m3_encode(float y) {
  uint16_t r;
  asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(0.0f), "f"(y));
  return (uint32_t)(r & 0xFFu);
}
__device__ __forceinline__ float e4m3_decode(uint32_t code) {
  uint32_t h2;
  asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"((uint16_t)code));
  return __half2float(__ushort_as_half((unsigned short)(h2 & 0xFFFFu)));
}

template <bool kPnq, bool kOutF32>
__global__ void __launch_bounds__(kThreads, 1) attention_nvfp4_kernel(const Params p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t sbase = smem_u32(smem);
  const uint32_t bar0 = sbase + kOffBar;
  auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + kOffMisc);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + kOffMisc + 8);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (*reinterpret_cast<volatile int*>(p.status) != 0) return;
  const int T = p.kv_tiles;
  const int bh = blockIdx.x / p.q_pairs, pair = blockIdx.x - bh * p.q_pairs;

  if (tid == 0) {
    mbar_init(bar(BAR_Q), 1);
    for (int s = 0; s < kStages; ++s) { mbar_init(bar(BAR_KFULL + s), 1); mbar_init(bar(BAR_KEMPTY + s), 1); }
    mbar_init(bar(BAR_SFULL + 0), 1); mbar_init(bar(BAR_SFULL + 1), 1);
    mbar_init(bar(BAR_SFREE), 8);
    mbar_init(bar(BAR_PFULL + 0), 8); mbar_init(bar(BAR_PFULL + 1), 8);
    mbar_init(bar(BAR_ODONE + 0), 1); mbar_init(bar(BAR_ODONE + 1), 1);
    abort_flag[0] = 0;
    abort_flag[1] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // rows of ones appended to every V stage (E2M1 code 2 = 1.0) and their scale atom (E4M3 1.0 = 0x38)
  for (int i = tid; i < kStages * 16 * 64 / 16; i += kThreads) {
    const int s = i / 64, c = i % 64;
    reinterpret_cast<uint4*>(smem + kOffV + s * kVStageBytes + kTileCodeBytes)[c] =
        make_uint4(0x22222222u, 0x22222222u, 0x22222222u, 0x22222222u);
  }
  for (int i = tid; i < kTileScaleBytes / 16; i += kThreads)
    reinterpret_cast<uint4*>(smem + kOffSFOnes)[i] = make_uint4(0x38383838u, 0x38383838u, 0x38383838u, 0x38383838u);
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
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
      const int64_t qt0 = (int64_t)bh * p.q_tiles + 2 * pair;
      const int64_t qt1 = (2 * pair + 1 < p.q_tiles) ? qt0 + 1 : qt0;
      mbar_expect_tx(bar(BAR_Q), 2 * (kTileCodeBytes + kSF));
      bulk_g2s(sbase + kOffQ, p.q_codes + qt0 * kTileCodeBytes, kTileCodeBytes, bar(BAR_Q));
      bulk_g2s(sbase + kOffQ + kTileCodeBytes, p.q_codes + qt1 * kTileCodeBytes, kTileCodeBytes, bar(BAR_Q));
      bulk_g2s(sbase + kOffSFQ, p.q_scales + qt0 * kSF, kSF, bar(BAR_Q));
      bulk_g2s(sbase + kOffSFQ + kSF, p.q_scales + qt1 * kSF, kSF, bar(BAR_Q));
      const int64_t kv0 = (int64_t)bh * T;
      bool ok = true;
      int j = 0;
      for (; j < T && ok; ++j) {
        const int s = j % kStages;
        if (j >= kStages) ok = mbar_wait(bar(BAR_KEMPTY + s), (uint32_t)(((j / kStages) & 1) ^ 1), abort_flag, p.status, 11);
        if (!ok) break;
        mbar_expect_tx(bar(BAR_KFULL + s), 2 * (kTileCodeBytes + kSF));
        bulk_g2s(sbase + kOffK + s * kTileCodeBytes, p.k_codes + (kv0 + j) * kTileCodeBytes, kTileCodeBytes, bar(BAR_KFULL + s));
        bulk_g2s(sbase + kOffSFK + s * kSF, p.k_scales + (kv0 + j) * kSF, kSF, bar(BAR_KFULL + s));
        bulk_g2s(sbase + kOffV + s * kVStageBytes, p.v_codes + (kv0 + j) * kTileCodeBytes, kTileCodeBytes, bar(BAR_KFULL + s));
        bulk_g2s(sbase + kOffSFV + s * kSF, p.v_scales + (kv0 + j) * kSF, kSF, bar(BAR_KFULL + s));
      }
      if (!ok || *abort_flag) {                        // gave up: let copies in flight land before shared memory is released
        const long long t0 = clock64();
        for (int f = (j > kStages ? j - kStages : 0); f < j; ++f)
          while (!mbar_try(bar(BAR_KFULL + f % kStages), (uint32_t)((f / kStages) & 1)) && clock64() - t0 < 200000000LL) {}
        while (!mbar_try(bar(BAR_Q), 0u) && clock64() - t0 < 200000000LL) {}
      }
    }
  } else if (warp == kSoftmaxWarps + 1) {
    // =============================== MMA issuer =============================================
    if (lane == 0) {
      bool ok = mbar_wait(bar(BAR_Q), 0, abort_flag, p.status, 21);
      uint32_t sfree_n = 0;
      constexpr uint32_t kDescHiTile = (512u >> 4) | (1u << 14) | (4u << 29);   // 64-byte swizzle, K-major
      const uint32_t q_lo = (sbase + kOffQ) >> 4, k_lo = (sbase + kOffK) >> 4;
      const uint32_t v_lo = (sbase + kOffV) >> 4, p_lo = (sbase + kOffP) >> 4;
      auto desc = [](uint32_t lo) { return ((uint64_t)kDescHiTile << 32) | lo; };
      auto gemm1 = [&](int t, int j) {                 // S = Q_t K_j^T
        const uint32_t a = q_lo + (uint32_t)t * (kTileCodeBytes >> 4);
        const uint32_t b = k_lo + (uint32_t)(j % kStages) * (kTileCodeBytes >> 4);
        const uint32_t sfa = tmem + kColSFQ + 8 * t, sfb = tmem + kColSFK + 8 * (j & 1);
        tc_mma_nv(tmem + kColS, desc(a), desc(b), make_idesc_nv(128), sfa, sfb, 0u);
        tc_mma_nv(tmem + kColS, desc(a + 2), desc(b + 2), make_idesc_nv(128), sfa + 4, sfb + 4, 1u);
        tc_commit(bar(BAR_SFULL + t));
      };
      auto gemm2 = [&](int t, int j) {                 // O_t += P_t [V_j | 1]
        tc_cp_sf(tmem + kColSFP + 8 * t, sbase + kOffSFP + t * kSF);
        tc_cp_sf(tmem + kColSFP + 8 * t + 4, sbase + kOffSFP + t * kSF + kTileScaleBytes);
        const uint32_t a = p_lo + (uint32_t)t * (kTileCodeBytes >> 4);
        const uint32_t b = v_lo + (uint32_t)(j % kStages) * (kVStageBytes >> 4);
        const uint32_t d = tmem + (t ? kColO1 : kColO0);
        const uint32_t sfa = tmem + kColSFP + 8 * t, sfb = tmem + kColSFV + 16 * (j & 1);
        tc_mma_nv(d, desc(a), desc(b), make_idesc_nv(kNV), sfa, sfb, j > 0 ? 1u : 0u);
        tc_mma_nv(d, desc(a + 2), desc(b + 2), make_idesc_nv(kNV), sfa + 4, sfb + 8, 1u);
        tc_commit(bar(BAR_ODONE + t));
      };
      auto wait_kv = [&](int j, bool first) {
        const int s = j % kStages;
        if (!mbar_wait(bar(BAR_KFULL + s), (uint32_t)((j / kStages) & 1), abort_flag, p.status, 22)) return false;
        if (!first) {
          if (!mbar_wait(bar(BAR_SFREE), sfree_n & 1u, abort_flag, p.status, 23)) return false;
          ++sfree_n;
        }
        tc_fence_after();
        tc_cp_sf(tmem + kColSFK + 8 * (j & 1), sbase + kOffSFK + s * kSF);
        tc_cp_sf(tmem + kColSFK + 8 * (j & 1) + 4, sbase + kOffSFK + s * kSF + kTileScaleBytes);
        tc_cp_sf(tmem + kColSFV + 16 * (j & 1), sbase + kOffSFV + s * kSF);
        tc_cp_sf(tmem + kColSFV + 16 * (j & 1) + 8, sbase + kOffSFV + s * kSF + kTileScaleBytes);
        return true;
      };
      auto wait_sfree = [&]() {
        const bool r = mbar_wait(bar(BAR_SFREE), sfree_n & 1u, abort_flag, p.status, 23);
        ++sfree_n;
        tc_fence_after();
        return r;
      };
      if (ok) {
        tc_fence_after();
        for (int t = 0; t < 2; ++t) {
          tc_cp_sf(tmem + kColSFQ + 8 * t, sbase + kOffSFQ + t * kSF);
          tc_cp_sf(tmem + kColSFQ + 8 * t + 4, sbase + kOffSFQ + t * kSF + kTileScaleBytes);
        }
        for (int slot = 0; slot < 2; ++slot) {           // scales of the ones rows, both slots and both K halves
          tc_cp_sf(tmem + kColSFV + 16 * slot + 4, sbase + kOffSFOnes);
          tc_cp_sf(tmem + kColSFV + 16 * slot + 12, sbase + kOffSFOnes);
        }
      }
      // the issue order of forward.cu: G2(0,j) G1(1,j+1) G2(1,j) G1(0,j+2)
      ok = ok && wait_kv(0, true);
      if (ok) gemm1(0, 0);
      ok = ok && wait_sfree();
      if (ok) gemm1(1, 0);
      if (T > 1) {
        ok = ok && wait_kv(1, false);
        if (ok) gemm1(0, 1);
      }
      for (int j = 0; j < T && ok; ++j) {
        ok = mbar_wait(bar(BAR_PFULL + 0), (uint32_t)(j & 1), abort_flag, p.status, 24);
        if (!ok) break;
        tc_fence_after();
        gemm2(0, j);
        if (j + 1 < T) {
          ok = wait_sfree();
          if (!ok) break;
          gemm1(1, j + 1);
        }
        ok = mbar_wait(bar(BAR_PFULL + 1), (uint32_t)(j & 1), abort_flag, p.status, 26);
        if (!ok) break;
        tc_fence_after();
        gemm2(1, j);
        tc_commit(bar(BAR_KEMPTY + j % kStages));
        if (j + 2 < T) {
          ok = wait_kv(j + 2, false);
          if (!ok) break;
          gemm1(0, j + 2);
        }
      }
    }
  } else {
    // =============================== softmax groups =========================================
    const int t = warp >> 3;
    const int h = (warp >> 2) & 1;
    const int row = (warp & 3) * 32 + lane;
    const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t t_s = tmem + kColS + lane_addr + kCols * h;
    const uint32_t t_o = tmem + (t ? kColO1 : kColO0) + lane_addr;
    // S_raw carries neither tensor scale: both go into the exponent's multiplier
    const float c = p.scale_log2e * p.ts_q[bh] * p.ts_k[bh];
    float m_run = -INFINITY, l_run = 0.0f;
    const uint32_t aP0 = sbase + kOffP + t * kTileCodeBytes + tile_code_offset(row, 2 * h);
    const uint32_t aP1 = sbase + kOffP + t * kTileCodeBytes + tile_code_offset(row, 2 * h + 1);
    const uint32_t aSF = sbase + kOffSFP + t * kSF + h * kTileScaleBytes + tile_scale_offset(row, 0);   // atom h: this thread's 4 blocks
    const uint32_t aMaxOwn = sbase + kOffMax + (t * 256 + h * 128 + row) * 4;
    const uint32_t aMaxPartner = sbase + kOffMax + (t * 256 + (h ^ 1) * 128 + row) * 4;
    const int pair_bar = 1 + (warp & 3) + 4 * t;
    volatile int* const own_limit_only = abort_flag + 1;
    bool ok = true;
    int j = 0;
    for (; j < T; ++j) {
      ok = __all_sync(0xFFFFFFFFu, mbar_wait(bar(BAR_SFULL + t), (uint32_t)(j & 1), own_limit_only, p.status, 31, kWaitLimitCycles, abort_flag));
      if (!ok) break;
      tc_fence_after();
      uint32_t sr[kCols];
      TMEM_LD64(t_s, sr);
      tmem_ld_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(BAR_SFREE));
      if (j == T - 1) {
        const int valid = (int)(p.Nkv - (int64_t)j * kTile) - kCols * h;
#pragma unroll
        for (int i = 0; i < kCols; ++i)
          if (i >= valid) sr[i] = 0xFF800000u;
      }
      float bmax[4];
#pragma unroll
      for (int b = 0; b < 4; ++b) {
        float q2[2];
#pragma unroll
        for (int u = 0; u < 2; ++u) {
          const uint32_t* v = sr + 16 * b + 8 * u;
          float mx = max3(__uint_as_float(v[0]), __uint_as_float(v[1]), __uint_as_float(v[2]));
          mx = max3(mx, __uint_as_float(v[3]), __uint_as_float(v[4]));
          mx = max3(mx, __uint_as_float(v[5]), __uint_as_float(v[6]));
          q2[u] = fmaxf(mx, __uint_as_float(v[7]));
        }
        bmax[b] = fmaxf(q2[0], q2[1]);
      }
      const float own_max = fmaxf(fmaxf(bmax[0], bmax[1]), fmaxf(bmax[2], bmax[3]));
      const uint32_t par = (uint32_t)(j & 1) * 2048u;
      sts32f(aMaxOwn + par, own_max);
      asm volatile("bar.sync %0, 64;" ::"r"(pair_bar) : "memory");
      const float partner_max = lds32f(aMaxPartner + par);
      const bool o_ready = (j == 0) || mbar_test(bar(BAR_ODONE + t), (uint32_t)((j - 1) & 1));
      const float m_new = max3(m_run, own_max, partner_max);
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
      // block scales: the block's largest probability by the elements' own expression, then the two-level recipe.
      // The element multiplier 2688 / d_b is folded into the exponent as its logarithm (one lg2.approx per block in
      // place of a division per block and a multiply per element; relative difference about 2e-7, the order of
      // ex2.approx itself).  A block whose scale rounds to zero keeps multiplier 1: its probabilities are below
      // 2.2e-6 and round to code 0 either way, and the direct placement still sums them.
      float nb[4], inv_r[4];
      uint32_t sf4 = 0;
#pragma unroll
      for (int b = 0; b < 4; ++b) {
        const float pm = ex2(fmaf(bmax[b], c, nmc));
        const float y = __fmul_rn(__fmul_rn(pm, kTensorRangeP), kOneSixth);
        const uint32_t code = e4m3_encode(y);
        const float d = e4m3_decode(code);
        // log2(2688 / d) from the code's fields: d = (1 + k/8) 2^(E-7), so only the mantissa's logarithm is approximated,
        // on an argument in [1, 2) where lg2.approx is good to 2^-22 absolute (on d itself its error is relative to
        // log2 d, about 2e-6 for the blocks that matter, which moves codes across rounding boundaries); the integer part
        // and log2(2688) = 11 + 0.39231742 are added exactly enough that the sum rounds once at its own magnitude
        const uint32_t fe = code >> 3, fk = code & 7u;
        float lgm;
        asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(lgm) : "f"(fe ? __uint_as_float(0x3F800000u | (fk << 20)) : d * 512.0f));
        const float fef = __uint_as_float(0x4B400000u + fe) - 12582912.0f;           // (float)E without a conversion instruction
        const float lr = (fe ? 18.0f - fef : 20.0f) + (0.39231742f - lgm);           // subnormal d = k 2^-9
        nb[b] = d == 0.0f ? nmc : fmaf(-m_new, c, lr);     // one rounding: -(m_new c) + log2(2688 / d)
        inv_r[b] = d == 0.0f ? 1.0f : d * kInvTensorRangeP;
        sf4 |= code << (8 * b);
      }
      asm volatile("st.shared.b32 [%0], %1;" ::"r"(aSF), "r"(sf4) : "memory");
      float l_tile = 0.0f;
      const uint64_t cc2 = dup2(c);
      auto tile_body = [&](auto resc_tag) {
        constexpr bool kResc = decltype(resc_tag)::value;
        if (kResc) alpha = ex2((m_old - m_new) * c);
#pragma unroll
        for (int b32 = 0; b32 < 2; ++b32) {           // one 16-byte chunk of codes = 32 elements = two blocks
          uint4 w;
#pragma unroll
          for (int g = 0; g < 4; ++g) {
            uint32_t oc[8];
            const uint32_t t_oc = t_o + kCols * h + 32 * b32 + 8 * g;
            if (kResc) TMEM_LD8(t_oc, oc);
            const uint64_t nb2 = dup2(nb[2 * b32 + (g >> 1)]);
            float x[8];
#pragma unroll
            for (int i = 0; i < 8; i += 2) {           // x = exp2(s * c + nb) = p~ * 2688 / d_b, two elements per multiply-add
              fma2(sr[32 * b32 + 8 * g + i], sr[32 * b32 + 8 * g + i + 1], cc2, nb2, x[i], x[i + 1]);
              x[i] = ex2(x[i]);
              x[i + 1] = ex2(x[i + 1]);
            }
            if (!kPnq) {
              float s0, s1;
              add2x2(x[0], x[1], x[2], x[3], x[4], x[5], x[6], x[7], s0, s1);
              l_tile = fmaf(s0 + s1, inv_r[2 * b32 + (g >> 1)], l_tile);
            }
            const uint32_t pk = pack_e2m1x8(x[0], x[1], x[2], x[3], x[4], x[5], x[6], x[7]);
            if (g == 0) w.x = pk; else if (g == 1) w.y = pk; else if (g == 2) w.z = pk; else w.w = pk;
            if (kResc) {
              tmem_ld_wait();
#pragma unroll
              for (int i = 0; i < 8; ++i) oc[i] = __float_as_uint(__uint_as_float(oc[i]) * alpha);
              TMEM_ST8(t_oc, oc);
            }
          }
          sts128(b32 == 0 ? aP0 : aP1, w);
        }
        if (kResc) {
          if (kPnq && h == 0) {                        // column 128: the running row sum of the quantized probabilities
            uint32_t lr;
            asm volatile("tcgen05.ld.sync.aligned.32x32b.x1.b32 {%0}, [%1];" : "=r"(lr) : "r"(t_o + 128) : "memory");
            tmem_ld_wait();
            lr = __float_as_uint(__uint_as_float(lr) * alpha);
            asm volatile("tcgen05.st.sync.aligned.32x32b.x1.b32 [%1], {%0};" ::"r"(lr), "r"(t_o + 128) : "memory");
          }
          tmem_st_wait();
        }
      };
      if (rescale) tile_body(std::true_type{}); else tile_body(std::false_type{});
      if (!kPnq) l_run = fmaf(alpha, l_run, l_tile);
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(BAR_PFULL + t));
    }
    if (!ok) pair_keep_company(pair_bar, T - j);

    // ---- epilogue ----
    if (ok) ok = __all_sync(0xFFFFFFFFu, mbar_wait(bar(BAR_ODONE + t), (uint32_t)((T - 1) & 1), own_limit_only, p.status, 33, kWaitLimitCycles, abort_flag));
    float l = l_run;
    if (!kPnq) {
      const uint32_t par = (uint32_t)(T & 1) * 2048u;
      sts32f(aMaxOwn + par, l_run);
      asm volatile("bar.sync %0, 64;" ::"r"(pair_bar) : "memory");
      l = l_run + lds32f(aMaxPartner + par);
    }
    if (ok) {
      tc_fence_after();
      float o_scale = p.ts_v[bh];                      // O = O_raw s_T(V) s_T(P) / l; under PNQ l = l_raw s_T(P)
      if (kPnq) {
        uint32_t lr;
        asm volatile("tcgen05.ld.sync.aligned.32x32b.x1.b32 {%0}, [%1];" : "=r"(lr) : "r"(t_o + 128) : "memory");
        tmem_ld_wait();
        l = __uint_as_float(lr);
      } else {
        o_scale *= __fdiv_rn(1.0f, kTensorRangeP);
      }
      const int qtile = 2 * pair + t;
      const int64_t grow = (int64_t)qtile * kTile + row;
      const bool store = (qtile < p.q_tiles) && (grow < p.Nq);
      const float inv_l = o_scale / l;
      const int64_t obase = ((int64_t)bh * p.Nq + grow) * kHeadDim + kCols * h;
#pragma unroll 1
      for (int c0 = 0; c0 < kCols; c0 += 32) {
        uint32_t r32[32];
        TMEM_LD32(t_o + kCols * h + c0, r32);
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

struct Layout { size_t status, amax, tscale, q_codes, q_scales, k_codes, k_scales, v_codes, v_scales, total; };

static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

static bool carve(int B, int H, int64_t Nq, int64_t Nkv, Layout* w) {
  if (B <= 0 || H <= 0 || Nq <= 0 || Nkv <= 0) return false;
  const size_t bh = (size_t)B * H;
  const size_t qt = (size_t)((Nq + kTile - 1) / kTile), kt = (size_t)((Nkv + kTile - 1) / kTile);
  size_t off = 0;
  w->status = off;   off += 256;
  w->amax = off;     off += align_up(3 * bh * sizeof(float), 256);
  w->tscale = off;   off += align_up(3 * bh * sizeof(float), 256);
  w->q_codes = off;  off += align_up(bh * qt * kTileCodeBytes, 256);
  w->q_scales = off; off += align_up(bh * qt * kSF, 256);
  w->k_codes = off;  off += align_up(bh * kt * kTileCodeBytes, 256);
  w->k_scales = off; off += align_up(bh * kt * kSF, 256);
  w->v_codes = off;  off += align_up(bh * kt * kTileCodeBytes, 256);
  w->v_scales = off; off += align_up(bh * kt * kSF, 256);
  w->total = off;
  return true;
}

}  // namespace fwdnv

size_t nvfp4_workspace_bytes(int B, int H, int64_t Nq, int64_t Nkv) {
  fwdnv::Layout w;
  return fwdnv::carve(B, H, Nq, Nkv, &w) ? w.total : 0;
}

int launch_forward_nvfp4(const void* q, const void* k, const void* v, void* o, int B, int H, int64_t Nq, int64_t Nkv,
                         float softmax_scale, unsigned flags, void* workspace, size_t workspace_bytes, cudaStream_t stream) {
  using namespace fwdnv;
  Layout w;
  if (!carve(B, H, Nq, Nkv, &w)) return MXATTN_EINVAL;
  if (workspace_bytes < w.total) return MXATTN_EWORKSPACE;
  const int64_t bh = (int64_t)B * H;
  const int64_t qt = (Nq + kTile - 1) / kTile, kt = (Nkv + kTile - 1) / kTile;
  const int64_t pairs = (qt + 1) / 2, grid = bh * pairs;
  if (qt > 0x3FFFFFFF || kt > 0x3FFFFFFF || grid > 0x7FFFFFFF) return MXATTN_EUNSUPPORTED;
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  float* amax = reinterpret_cast<float*>(ws + w.amax);
  float* ts = reinterpret_cast<float*>(ws + w.tscale);
  if (cudaMemsetAsync(ws + w.status, 0, 16, stream) != cudaSuccess) return MXATTN_ECUDA;
  int rc;
  // one tensor-level scale per head matrix (Q, K, V each), then the block quantizers
  if ((rc = launch_tensor_amax(q, amax, bh, Nq, kHeadDim, stream))) return rc;
  if ((rc = launch_tensor_amax(k, amax + bh, bh, Nkv, kHeadDim, stream))) return rc;
  if ((rc = launch_tensor_amax(v, amax + 2 * bh, bh, Nkv, kHeadDim, stream))) return rc;
  if ((rc = launch_quantize_nvfp4(q, ws + w.q_codes, ws + w.q_scales, amax, ts, bh, Nq, kHeadDim, 1, MXATTN_LAYOUT_TILE, stream))) return rc;
  if ((rc = launch_quantize_nvfp4(k, ws + w.k_codes, ws + w.k_scales, amax + bh, ts + bh, bh, Nkv, kHeadDim, 1, MXATTN_LAYOUT_TILE, stream))) return rc;
  if ((rc = launch_quantize_nvfp4(v, ws + w.v_codes, ws + w.v_scales, amax + 2 * bh, ts + 2 * bh, bh, Nkv, kHeadDim, 0, MXATTN_LAYOUT_TILE, stream))) return rc;
  Params p;
  p.q_codes = ws + w.q_codes; p.q_scales = ws + w.q_scales; p.k_codes = ws + w.k_codes; p.k_scales = ws + w.k_scales;
  p.v_codes = ws + w.v_codes; p.v_scales = ws + w.v_scales;
  p.ts_q = ts; p.ts_k = ts + bh; p.ts_v = ts + 2 * bh;
  p.out = o; p.status = reinterpret_cast<int*>(ws + w.status);
  p.Nq = Nq; p.Nkv = Nkv; p.q_tiles = (int)qt; p.kv_tiles = (int)kt; p.q_pairs = (int)pairs;
  p.scale_log2e = softmax_scale * 1.4426950408889634f;
  const bool pnq = flags & MXATTN_FLAG_PNQ, f32 = flags & MXATTN_FLAG_OUT_FP32;
  void (*kern)(const Params) = pnq ? (f32 ? attention_nvfp4_kernel<true, true> : attention_nvfp4_kernel<true, false>)
                                   : (f32 ? attention_nvfp4_kernel<false, true> : attention_nvfp4_kernel<false, false>);
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess) return MXATTN_ECUDA;
  kern<<<(unsigned)grid, kThreads, kSmemBytes, stream>>>(p);
  count_launch(1);
  return cudaGetLastError() == cudaSuccess ? MXATTN_OK : MXATTN_ECUDA;
}

}  // namespace mxattn
