// Row-sum diagnostic for MXFP4 quantization of attention probabilities (paper Section 5.3, figure
// "Row-sum diagnostics", panels A, B and D) for sm_100a.
//
// For every query row: the attention probabilities are formed as if materialized,
// P = softmax(Q-hat K-hat^T * softmax_scale), rounded to fp32, quantized in 32-blocks along the key
// axis with the OCP or the UOS rule, and the row sum of the quantized values is reported together
// with the split of its error by quantization outcome (zeroing, saturation, downward and upward
// rounding) and the row entropy.  Nothing is materialized: the scores are produced twice by the
// same block-scaled FP4 GEMM as in the attention kernel (tcgen05.mma kind::mxf4, fp32 scores in
// tensor memory) -- a first pass over the KV tiles takes the row maximum and the normalizer, a
// second one quantizes the normalized probabilities block by block in registers.
//
// One CTA = one query tile of 128 rows.  Roles (320 threads): warps 0-7 two threads per query row
// (64 key columns each, i.e. two blocks of every tile), warp 8 producer (bulk copies of the K-hat
// tile images, each tile twice), warp 9 MMA issuer (one thread).  Two score buffers in tensor
// memory.  Every mbarrier wait is bounded as in the attention kernel; the two named barriers that
// pair the half rows are reached by both warps on every path.
#include <cuda_fp16.h>

#include "common.cuh"
#include "tc_helpers.cuh"

namespace mxattn {
namespace diag {
using namespace fwd;

constexpr int kThreads = 320;
constexpr int kStages = 4;
constexpr int kOffQ = 0;                                   // 8192
constexpr int kOffK = kOffQ + kTileCodeBytes;              // 4 x 8192
constexpr int kOffSFQ = kOffK + kStages * kTileCodeBytes;  // 512
constexpr int kOffSFK = kOffSFQ + kTileScaleBytes;         // 4 x 512
constexpr int kOffBar = kOffSFK + kStages * kTileScaleBytes;
enum Bar { BAR_Q = 0, BAR_KFULL = 1, BAR_KEMPTY = BAR_KFULL + kStages, BAR_SFULL = BAR_KEMPTY + kStages,
           BAR_SFREE = BAR_SFULL + 2, kNumBars = BAR_SFREE + 2 };
constexpr int kOffMisc = kOffBar + kNumBars * 8;
constexpr int kOffEx = (kOffMisc + 64 + 15) & ~15;         // exchange between the half rows: [2][128][8] floats
constexpr int kSmemBytes = kOffEx + 2 * 128 * 8 * 4 + 1024;
constexpr uint32_t kColS = 0, kColSFQ = 256, kColSFK = 260;

struct Params {
  const uint8_t* q_codes; const uint8_t* q_scales;
  const uint8_t* k_codes; const uint8_t* k_scales;
  float* out;           // [B*H, Nq, 6]
  int* status;
  int64_t Nq, Nkv;
  int q_tiles, kv_tiles;
  float scale_log2e;
  uint32_t rule;        // kRuleOcp or the boundary's fp32 bit pattern
};

// two fp32 -> E2M1 (round to nearest even, saturating) and back: the values the format can hold
__device__ __forceinline__ void round_e2m1_pair(float x0, float x1, float& v0, float& v1) {
  uint32_t h2;
  asm("{\n\t.reg .b8 c;\n\tcvt.rn.satfinite.e2m1x2.f32 c, %2, %1;\n\tcvt.rn.f16x2.e2m1x2 %0, c;\n\t}" : "=r"(h2) : "f"(x0), "f"(x1));
  const __half2 h = *reinterpret_cast<const __half2*>(&h2);
  v0 = __low2float(h);
  v1 = __high2float(h);
}

__global__ void __launch_bounds__(kThreads, 1) rowsum_diag_kernel(const Params p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t sbase = smem_u32(smem);
  const uint32_t bar0 = sbase + kOffBar;
  auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + kOffMisc);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + kOffMisc + 8);
  float* ex = reinterpret_cast<float*>(smem + kOffEx);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (*reinterpret_cast<volatile int*>(p.status) != 0) return;
  const int bh = blockIdx.x / p.q_tiles;
  const int qtile = blockIdx.x - bh * p.q_tiles;
  const int T = p.kv_tiles;

  if (tid == 0) {
    mbar_init(bar(BAR_Q), 1);
    for (int s = 0; s < kStages; ++s) { mbar_init(bar(BAR_KFULL + s), 1); mbar_init(bar(BAR_KEMPTY + s), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(bar(BAR_SFULL + b), 1); mbar_init(bar(BAR_SFREE + b), 8); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 9) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(tmem_slot)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  if (warp == 8) {
    // ---- producer: every K-hat tile twice (pass 1: maximum and normalizer, pass 2: quantization) ----
    if (lane == 0) {
      const int64_t qt = (int64_t)bh * p.q_tiles + qtile;
      mbar_expect_tx(bar(BAR_Q), kTileCodeBytes + kTileScaleBytes);
      bulk_g2s(sbase + kOffQ, p.q_codes + qt * kTileCodeBytes, kTileCodeBytes, bar(BAR_Q));
      bulk_g2s(sbase + kOffSFQ, p.q_scales + qt * kTileScaleBytes, kTileScaleBytes, bar(BAR_Q));
      const int64_t kv0 = (int64_t)bh * T;
      int issued = 0;
      bool ok = true;
      for (int it = 0; it < 2 * T && ok; ++it) {
        const int s = it % kStages, j = it < T ? it : it - T;
        if (it >= kStages) ok = mbar_wait(bar(BAR_KEMPTY + s), (uint32_t)((it / kStages) & 1) ^ 1u, abort_flag, p.status, 11);
        if (!ok) break;
        mbar_expect_tx(bar(BAR_KFULL + s), kTileCodeBytes + kTileScaleBytes);
        bulk_g2s(sbase + kOffK + s * kTileCodeBytes, p.k_codes + (kv0 + j) * kTileCodeBytes, kTileCodeBytes, bar(BAR_KFULL + s));
        bulk_g2s(sbase + kOffSFK + s * kTileScaleBytes, p.k_scales + (kv0 + j) * kTileScaleBytes, kTileScaleBytes, bar(BAR_KFULL + s));
        issued = it + 1;
      }
      if (!ok || *abort_flag) {                    // gave up: let copies in flight land before the CTA ends
        const long long t0 = clock64();
        for (int it = (issued > kStages ? issued - kStages : 0); it < issued; ++it)
          while (!mbar_try(bar(BAR_KFULL + it % kStages), (uint32_t)((it / kStages) & 1)) && clock64() - t0 < 200000000LL) {}
        while (!mbar_try(bar(BAR_Q), 0) && clock64() - t0 < 200000000LL) {}
      }
    }
  } else if (warp == 9) {
    // ---- MMA issuer: S = Q-hat K-hat_j^T into the two score buffers alternately ----
    if (lane == 0) {
      bool ok = mbar_wait(bar(BAR_Q), 0, abort_flag, p.status, 21);
      constexpr uint32_t kDescHiTile = (512u >> 4) | (1u << 14) | (4u << 29);   // 64-byte swizzle, K-major
      auto desc = [](uint32_t lo) { return ((uint64_t)kDescHiTile << 32) | lo; };
      const uint32_t q_lo = (sbase + kOffQ) >> 4, k_lo = (sbase + kOffK) >> 4;
      if (ok) {
        tc_fence_after();
        tc_cp_sf(tmem + kColSFQ, sbase + kOffSFQ);
      }
      for (int it = 0; it < 2 * T && ok; ++it) {
        const int s = it % kStages, b = it & 1;
        ok = mbar_wait(bar(BAR_KFULL + s), (uint32_t)((it / kStages) & 1), abort_flag, p.status, 22);
        if (ok && it >= 2) ok = mbar_wait(bar(BAR_SFREE + b), (uint32_t)(((it - 2) >> 1) & 1), abort_flag, p.status, 23);
        if (!ok) break;
        tc_fence_after();
        const uint32_t sfb = tmem + kColSFK + 4 * b;
        tc_cp_sf(sfb, sbase + kOffSFK + s * kTileScaleBytes);
        const uint32_t kb = k_lo + (uint32_t)s * (kTileCodeBytes >> 4);
        tc_mma(tmem + kColS + 128 * b, desc(q_lo), desc(kb), make_idesc(128, 0), tmem + kColSFQ, sfb, 0u);
        tc_mma(tmem + kColS + 128 * b, desc(q_lo + 2), desc(kb + 2), make_idesc(128, 1), tmem + kColSFQ, sfb, 1u);
        tc_commit(bar(BAR_SFULL + b));
        tc_commit(bar(BAR_KEMPTY + s));
      }
    }
  } else {
    // ---- softmax / quantization warps ----
    const int h = warp >> 2, quad = warp & 3;
    const int row = quad * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
    const float c = p.scale_log2e;
    const int pair_bar = 1 + quad;
    const int last_valid = (int)(p.Nkv - (int64_t)(T - 1) * kTile) - 64 * h;   // valid columns of this half in the last tile
    bool ok = true;
    uint32_t sr[64];
    auto fetch = [&](int it) {                     // scores of tile `it` (0 .. 2T-1) -> registers, buffer released
      const int b = it & 1;
      ok = mbar_wait(bar(BAR_SFULL + b), (uint32_t)((it >> 1) & 1), abort_flag, p.status, 31);
      if (!ok) return;
      tc_fence_after();
      TMEM_LD64(tmem + kColS + 128 * b + lane_addr + 64 * h, sr);
      tmem_ld_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(BAR_SFREE + b));
      const int j = it < T ? it : it - T;
      if (j == T - 1) {
#pragma unroll
        for (int i = 0; i < 64; ++i)
          if (i >= last_valid) sr[i] = 0xFF800000u;   // keys beyond Nkv do not exist
      }
    };

    // pass 1: row maximum and normalizer of this half row (online, as in the softmax recurrence)
    float m = -INFINITY, z = 0.0f;
    for (int it = 0; it < T && ok; ++it) {
      fetch(it);
      if (!ok) break;
      float tmax = -INFINITY;
#pragma unroll
      for (int i = 0; i < 64; i += 2) tmax = max3(tmax, __uint_as_float(sr[i]), __uint_as_float(sr[i + 1]));
      const float m_new = fmaxf(m, tmax);
      if (m_new != -INFINITY) {
        const float nmc = -(m_new * c);
        float acc = 0.0f;
#pragma unroll
        for (int i = 0; i < 64; ++i) acc += ex2(fmaf(__uint_as_float(sr[i]), c, nmc));
        z = fmaf(z, ex2((m - m_new) * c), acc);
        m = m_new;
      }
    }
    ex[(h * 128 + row) * 8 + 0] = m;
    ex[(h * 128 + row) * 8 + 1] = z;
    asm volatile("bar.sync %0, 64;" ::"r"(pair_bar) : "memory");
    const float m_o = ex[((h ^ 1) * 128 + row) * 8 + 0], z_o = ex[((h ^ 1) * 128 + row) * 8 + 1];
    const float M = fmaxf(m, m_o);
    const float Z = (m == -INFINITY ? 0.0f : z * ex2((m - M) * c)) + (m_o == -INFINITY ? 0.0f : z_o * ex2((m_o - M) * c));
    const float inv_z = 1.0f / Z;
    const float ln_z = logf(Z);
    const float nMc = -(M * c);
    asm volatile("bar.sync %0, 64;" ::"r"(pair_bar) : "memory");      // the exchange slots are reused below

    // pass 2: normalized probabilities, quantized block by block
    float rs = 0.0f, zer = 0.0f, sat = 0.0f, dn = 0.0f, up = 0.0f, ent = 0.0f;
    for (int it = T; it < 2 * T && ok; ++it) {
      fetch(it);
      if (!ok) break;
#pragma unroll
      for (int b = 0; b < 2; ++b) {
        float pv[32];
        float bm = 0.0f;
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          const float y = fmaf(__uint_as_float(sr[32 * b + i]), c, nMc);     // log2 of the unnormalized weight
          pv[i] = ex2(y) * inv_z;                                            // -inf -> 0 for masked keys
          bm = fmaxf(bm, pv[i]);
          if (pv[i] > 0.0f) ent = fmaf(-pv[i], fmaf(y, 0.6931471805599453f, -ln_z), ent);
        }
        const int e = shared_exponent_rule(__float_as_uint(bm), p.rule);
        const float inv = pow2_neg(e);
        const float sigma = e > -127 ? __uint_as_float((uint32_t)(e + 127) << 23) : 5.877471754111438e-39f;   // 2^e
#pragma unroll
        for (int i = 0; i < 32; i += 2) {
          const float x0 = pv[i] * inv, x1 = pv[i + 1] * inv;
          float v0, v1;
          round_e2m1_pair(x0, x1, v0, v1);
          const float q0 = v0 * sigma, q1 = v1 * sigma;
          const float d0 = q0 - pv[i], d1 = q1 - pv[i + 1];
          rs += q0 + q1;
          if (x0 > 6.0f) sat += d0; else if (v0 == 0.0f) zer += d0; else if (d0 < 0.0f) dn += d0; else up += d0;
          if (x1 > 6.0f) sat += d1; else if (v1 == 0.0f) zer += d1; else if (d1 < 0.0f) dn += d1; else up += d1;
        }
      }
    }
    // combine the two half rows
    if (h == 1) {
      float* e8 = ex + row * 8;
      e8[0] = rs; e8[1] = zer; e8[2] = sat; e8[3] = dn; e8[4] = up; e8[5] = ent;
    }
    asm volatile("bar.sync %0, 64;" ::"r"(pair_bar) : "memory");
    const int64_t grow = (int64_t)qtile * kTile + row;
    if (h == 0 && ok && grow < p.Nq) {
      const float* e8 = ex + row * 8;
      float* o = p.out + ((int64_t)bh * p.Nq + grow) * 6;
      o[0] = rs + e8[0]; o[1] = zer + e8[1]; o[2] = sat + e8[2]; o[3] = dn + e8[3]; o[4] = up + e8[4]; o[5] = ent + e8[5];
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 9) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");
  }
}

}  // namespace diag

int launch_rowsum_diag(const void* q_codes, const void* q_scales, const void* k_codes, const void* k_scales,
                       void* out, int B, int H, int64_t Nq, int64_t Nkv, float softmax_scale, uint32_t rule,
                       int* status, cudaStream_t stream) {
  using namespace diag;
  Params p;
  p.q_codes = (const uint8_t*)q_codes; p.q_scales = (const uint8_t*)q_scales;
  p.k_codes = (const uint8_t*)k_codes; p.k_scales = (const uint8_t*)k_scales;
  p.out = (float*)out; p.status = status; p.Nq = Nq; p.Nkv = Nkv;
  const int64_t qt = (Nq + kTile - 1) / kTile, kt = (Nkv + kTile - 1) / kTile;
  const int64_t grid = (int64_t)B * H * qt;
  if (qt > 0x3FFFFFFF || kt > 0x3FFFFFFF || grid > 0x7FFFFFFF) return MXATTN_EUNSUPPORTED;
  p.q_tiles = (int)qt; p.kv_tiles = (int)kt;
  p.scale_log2e = softmax_scale * 1.4426950408889634f;
  p.rule = rule;
  if (cudaFuncSetAttribute(rowsum_diag_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess)
    return MXATTN_ECUDA;
  rowsum_diag_kernel<<<(unsigned)grid, kThreads, kSmemBytes, stream>>>(p);
  count_launch(1);
  return cudaGetLastError() == cudaSuccess ? MXATTN_OK : MXATTN_ECUDA;
}

}  // namespace mxattn
