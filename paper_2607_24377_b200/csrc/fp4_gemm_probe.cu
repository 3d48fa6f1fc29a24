// Dense block-scaled FP4 GEMM probe for sm_100a: C[M, N] = A[M, K] B[N, K]^T with MXFP4 operands (E2M1 codes,
// one E8M0 scale per 32 elements along K), fp32 accumulation in tensor memory -- the same
// tcgen05.mma kind::mxf4.block_scale instruction the attention kernel's two GEMMs use (paper Section 1: the two
// GEMMs are the dominant operations of the attention forward).  Its purpose is to MEASURE what the FP4 tensor pipe of
// the device delivers, as the denominator of the attention kernel's roofline fraction:
//   * streaming mode: a real GEMM, operand tiles streamed from global memory through a 6-stage shared-memory ring;
//   * resident mode:  the same instruction stream with the ring loaded once and reused for every K step, which takes
//                     global memory and L2 out of the picture and measures the issue rate of the tensor pipe itself.
//
// One CTA computes a 128 x 256 (or 128 x 128) tile of C.  Roles: warp 0 producer (bulk async copies), warp 1 MMA issuer (one
// thread), warps 2-5 epilogue (one thread per row of the tile: tensor memory -> registers -> global memory).
// Every barrier wait is bounded; on expiry the CTA records a code in `status` and exits normally.
#include "common.cuh"
#include "tc_helpers.cuh"

namespace mxattn {
namespace probe {
using namespace fwd;

constexpr int kStages = 6;
constexpr int kThreads = 32 * 6;
constexpr int kStageBytes = kTileCodeBytes * 3 + kTileScaleBytes * 3;    // A tile, two B tiles, their three scale atoms
constexpr int kOffBar = kStages * kStageBytes;
constexpr int kSmemBytes = kOffBar + 256 + 1024;
constexpr uint32_t kColAcc = 0, kColSF = 256;    // accumulator 256 columns; then scale-factor slots of 12 columns (A: 4, B: 8), one per stage

struct Params {
  const uint8_t* a_codes; const uint8_t* a_scales;     // [K/128][M/128][8192] / [K/128][M/128][512]
  const uint8_t* b_codes; const uint8_t* b_scales;     // [K/128][N/128][8192] / [K/128][N/128][512]
  void* c;                                             // [M, N] row-major, fp32 or bf16
  int* status;
  int m_tiles, n_tiles128;                             // M / 128, N / 128
  int k_blocks;                                        // K / 128 blocks that exist in memory
  int k_steps;                                         // K steps executed (= k_blocks when streaming)
  int resident;                                        // 1: load the first min(k_steps, kStages) blocks once and cycle over them
};

template <bool kOutF32, int kTileN>
__global__ void __launch_bounds__(kThreads, 1) fp4_gemm_probe_kernel(const Params p) {
  constexpr int kBTiles = kTileN / 128;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t sbase = smem_u32(smem);
  auto bar_full = [&](int s) { return sbase + kOffBar + 8u * (uint32_t)s; };
  auto bar_empty = [&](int s) { return sbase + kOffBar + 8u * (uint32_t)(kStages + s); };
  const uint32_t bar_acc = sbase + kOffBar + 8u * (2 * kStages);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + kOffBar + 8 * (2 * kStages + 1));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + kOffBar + 8 * (2 * kStages + 1) + 8);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (*reinterpret_cast<volatile int*>(p.status) != 0) return;
  const int mt = blockIdx.x % p.m_tiles, nt = blockIdx.x / p.m_tiles;     // consecutive CTAs share the B tiles

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(bar_full(s), 1); mbar_init(bar_empty(s), 1); }
    mbar_init(bar_acc, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(tmem_slot)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const int n_loads = p.resident ? (p.k_steps < kStages ? p.k_steps : kStages) : p.k_steps;

  if (warp == 0) {
    if (lane == 0) {
      bool ok = true;
      int i = 0;
      for (; i < n_loads && ok; ++i) {
        const int s = i % kStages;
        if (i >= kStages) ok = mbar_wait(bar_empty(s), (uint32_t)(((i / kStages) & 1) ^ 1), abort_flag, p.status, 41);
        if (!ok) break;
        const int kb = i % p.k_blocks;
        const uint32_t st = sbase + s * kStageBytes;
        const int64_t ta = (int64_t)kb * p.m_tiles + mt, tb = (int64_t)kb * p.n_tiles128 + kBTiles * nt;
        mbar_expect_tx(bar_full(s), (1 + kBTiles) * (kTileCodeBytes + kTileScaleBytes));
        bulk_g2s(st, p.a_codes + ta * kTileCodeBytes, kTileCodeBytes, bar_full(s));
        bulk_g2s(st + kTileCodeBytes, p.b_codes + tb * kTileCodeBytes, kBTiles * kTileCodeBytes, bar_full(s));     // the B tiles of a CTA are adjacent
        bulk_g2s(st + 3 * kTileCodeBytes, p.a_scales + ta * kTileScaleBytes, kTileScaleBytes, bar_full(s));
        bulk_g2s(st + 3 * kTileCodeBytes + kTileScaleBytes, p.b_scales + tb * kTileScaleBytes, kBTiles * kTileScaleBytes, bar_full(s));
      }
      if (!ok || *abort_flag) {                      // gave up: let the copies in flight land before shared memory is released
        const long long t0 = clock64();
        for (int f = (i > kStages ? i - kStages : 0); f < i; ++f)
          while (!mbar_try(bar_full(f % kStages), (uint32_t)((f / kStages) & 1)) && clock64() - t0 < 200000000LL) {}
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t kDescHi = (512u >> 4) | (1u << 14) | (4u << 29);       // 8-row groups 512 B apart, 64-byte swizzle, K-major
      auto desc = [](uint32_t lo) { return ((uint64_t)kDescHi << 32) | lo; };
      bool ok = true;
      // first pass over the ring (all steps when streaming): wait for the stage, copy its scale factors into the
      // stage's tensor-memory slot (slot s was last read by the multiplies of step i - kStages, issued long before),
      // two multiplies of K = 64
      for (int i = 0; i < n_loads && ok; ++i) {
        const int s = i % kStages;
        ok = mbar_wait(bar_full(s), (uint32_t)((i / kStages) & 1), abort_flag, p.status, 42);
        if (!ok) break;
        tc_fence_after();
        const uint32_t st = sbase + s * kStageBytes;
        const uint32_t sfa = tmem + kColSF + 12 * s, sfb = sfa + 4;
        tc_cp_sf(sfa, st + 3 * kTileCodeBytes);
        tc_cp_sf(sfb, st + 3 * kTileCodeBytes + kTileScaleBytes);
        if (kBTiles == 2) tc_cp_sf(sfb + 4, st + 3 * kTileCodeBytes + 2 * kTileScaleBytes);
        const uint32_t a = st >> 4, b = (st + kTileCodeBytes) >> 4;
        tc_mma(tmem + kColAcc, desc(a), desc(b), make_idesc(kTileN, 0), sfa, sfb, i > 0 ? 1u : 0u);
        tc_mma(tmem + kColAcc, desc(a + 2), desc(b + 2), make_idesc(kTileN, 1), sfa, sfb, 1u);
        if (!p.resident) tc_commit(bar_empty(s));
      }
      // resident mode: everything is in place; the loop that is timed issues multiplies and nothing else
      if (ok && p.resident && p.k_steps > n_loads) {
        const int rounds = (p.k_steps - n_loads) / kStages;       // k_steps is a multiple of kStages here (checked on the host)
        const uint32_t a0 = sbase >> 4, stride = (uint32_t)kStageBytes >> 4;
#pragma unroll 1
        for (int r = 0; r < rounds; ++r) {
#pragma unroll
          for (int s = 0; s < kStages; ++s) {
            const uint32_t a = a0 + s * stride, b = a + (kTileCodeBytes >> 4);
            const uint32_t sfa = tmem + kColSF + 12 * s, sfb = sfa + 4;
            tc_mma(tmem + kColAcc, desc(a), desc(b), make_idesc(kTileN, 0), sfa, sfb, 1u);
            tc_mma(tmem + kColAcc, desc(a + 2), desc(b + 2), make_idesc(kTileN, 1), sfa, sfb, 1u);
          }
        }
      }
      if (ok) tc_commit(bar_acc);
    }
  } else {
    // epilogue: warp w may touch the tensor-memory lanes 32 * (w % 4) .. + 31
    const int q = warp & 3;
    const int row = q * 32 + lane;
    bool ok = __all_sync(0xFFFFFFFFu, mbar_wait(bar_acc, 0u, abort_flag, p.status, 43));
    if (ok) {
      tc_fence_after();
      const int64_t n_total = (int64_t)p.n_tiles128 * 128;
      const int64_t off = ((int64_t)mt * 128 + row) * n_total + (int64_t)nt * kTileN;
#pragma unroll 1
      for (int c0 = 0; c0 < kTileN; c0 += 32) {
        uint32_t r[32];
        TMEM_LD32(tmem + kColAcc + ((uint32_t)(q * 32) << 16) + c0, r);
        tmem_ld_wait();
        if (kOutF32) {
          float4* dst = reinterpret_cast<float4*>(static_cast<float*>(p.c) + off + c0);
#pragma unroll
          for (int i = 0; i < 8; ++i)
            dst[i] = make_float4(__uint_as_float(r[4 * i]), __uint_as_float(r[4 * i + 1]), __uint_as_float(r[4 * i + 2]), __uint_as_float(r[4 * i + 3]));
        } else {
          uint4* dst = reinterpret_cast<uint4*>(static_cast<uint16_t*>(p.c) + off + c0);
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            uint32_t h[4];
#pragma unroll
            for (int k = 0; k < 4; ++k)
              asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(h[k]) : "f"(__uint_as_float(r[8 * i + 2 * k + 1])), "f"(__uint_as_float(r[8 * i + 2 * k])));
            dst[i] = make_uint4(h[0], h[1], h[2], h[3]);
          }
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");
  }
}

}  // namespace probe
}  // namespace mxattn

extern "C" int mxattn_probe_fp4_gemm(const void* a_codes, const void* a_scales, const void* b_codes, const void* b_scales,
                                     void* c, int64_t M, int64_t N, int64_t K, int64_t k_steps, int resident, int out_fp32,
                                     int tile_n, void* status, void* stream) {
  using namespace mxattn;
  using namespace mxattn::probe;
  if (!a_codes || !a_scales || !b_codes || !b_scales || !c || !status) return MXATTN_EINVAL;
  if (M <= 0 || N <= 0 || K <= 0 || k_steps <= 0) return MXATTN_EINVAL;
  if (tile_n != 128 && tile_n != 256) return MXATTN_EINVAL;
  if (M % 128 || N % tile_n || K % 128) return MXATTN_EUNSUPPORTED;
  if (M > 16384 || N > 16384 || K > 16384 || k_steps > (1 << 20)) return MXATTN_EUNSUPPORTED;
  if (!resident && k_steps != K / 128) return MXATTN_EINVAL;
  if (resident && k_steps > 6 && (k_steps % 6 != 0 || K / 128 < 6)) return MXATTN_EINVAL;
  if (!aligned16(a_codes) || !aligned16(a_scales) || !aligned16(b_codes) || !aligned16(b_scales) || !aligned16(c) || !aligned16(status))
    return MXATTN_EALIGN;
  Params p;
  p.a_codes = (const uint8_t*)a_codes; p.a_scales = (const uint8_t*)a_scales;
  p.b_codes = (const uint8_t*)b_codes; p.b_scales = (const uint8_t*)b_scales;
  p.c = c; p.status = (int*)status;
  p.m_tiles = (int)(M / 128); p.n_tiles128 = (int)(N / 128); p.k_blocks = (int)(K / 128); p.k_steps = (int)k_steps; p.resident = resident ? 1 : 0;
  auto kern = tile_n == 256 ? (out_fp32 ? fp4_gemm_probe_kernel<true, 256> : fp4_gemm_probe_kernel<false, 256>)
                            : (out_fp32 ? fp4_gemm_probe_kernel<true, 128> : fp4_gemm_probe_kernel<false, 128>);
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess) return MXATTN_ECUDA;
  const unsigned grid = (unsigned)(p.m_tiles * (N / tile_n));
  kern<<<grid, kThreads, kSmemBytes, (cudaStream_t)stream>>>(p);
  count_launch(1);
  return cudaGetLastError() == cudaSuccess ? MXATTN_OK : MXATTN_ECUDA;
}
