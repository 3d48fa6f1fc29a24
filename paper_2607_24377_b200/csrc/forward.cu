// Fused MXFP4 attention forward for sm_100a (paper Algorithm 2, lines 6-19).
//
// One CTA owns two query tiles of 128 rows of one head and walks the KV tiles (B_c = 128 keys)
// in ascending order.  Roles (576 threads):
//   warps 0-7   softmax group 0 (query tile 0): two threads per query row, 64 key columns each
//               (warps 0-3 take columns 0-63, warps 4-7 columns 64-127; warp w works on the
//               tensor-memory lanes 32*(w%4) .. +31, i.e. rows 32*(w%4) .. +31 of the tile)
//   warps 8-15  softmax group 1 (query tile 1), same split
//   warp  16    producer: bulk async copies (TMA unit) of K-hat / V-hat tile images + scale atoms, four
//               stages; the K and V images of a tile complete one mbarrier
//   warp  17    MMA issuer: block-scaled FP4 tcgen05.mma (kind::mxf4, E8M0 scales), one thread.  What this
//               thread does per tile (5 waits, 4 scale-atom copies, 8 MMAs, 5 commits and the scalar
//               instructions between them) is on the kernel's critical path, so its loop is kept as short
//               as the dependencies allow and is unrolled by the number of stages.
//
// Both GEMMs are dense FP4 contractions with fp32 accumulators in tensor memory:
//   GEMM 1  S   = Q-hat_t K-hat_j^T              (M=128, N=128, K=128 as two K=64 instructions)
//   GEMM 2  O_t += P-hat_t [V-hat_j | 1]         (M=128, N=144, K=128)
// The 16 extra B rows of GEMM 2 hold the constant 1.0, so column 128 of the accumulator is the
// row sum of the QUANTIZED exponentials, P-hat 1 -- exactly the values the tensor core consumed.
// That is the PNQ row sum (paper Eq. 22, Algorithm 2 line 14) at no ALU cost; the direct
// placement (Eq. 12) instead accumulates the unquantized exponentials in a register.
//
// Per KV tile a softmax thread (Algorithm 2 lines 10-14, for its half row):
//   reads its 64 scores from tensor memory, takes its two 32-block maxima, exchanges the half-row
//   maximum with its partner thread through shared memory (64-thread named barrier),
//   m_new = max(m, rowmax);  for each of its blocks b, with c = softmax_scale * log2 e:
//     d     = (bmax_b - m_new) * c  = log2 of the block's largest exponential (<= 0)
//     e_b   = floor(d) - 2, plus one under UOS when frac(d) > log2 1.8125      (no exponential needed:
//             floor(log2 pmax) = floor(d), and the mantissa of pmax is 2^frac(d))
//     x     = exp2(s * c - (m_new * c + e_b))   == P~ / 2^e_b   (the block scale folded into the exponent)
//     codes = RNE-to-E2M1(x), 16 bytes, written into the K-major, 64B-swizzled A-operand tile
//   and its two scale bytes into the scale-factor atom.  The difference (bmax_b - m_new) is formed
//   exactly first, so the block holding the row maximum has d = 0 and gets e = -2 under both rules,
//   the scale the paper's Appendix J derives; the elements take one fused multiply-add (issued two at a
//   time as a packed fp32x2 instruction) and one ex2.approx each.
//   If a row maximum of the warp moved, the thread rescales its 64 accumulator columns in tensor
//   memory by alpha = exp(m - m_new) (line 15); those tensor-memory round trips are interleaved with
//   the exponentials (the loop body exists in two straight-line versions).
//
// Tensor-memory map (512 columns): S [0,128) shared by both groups (each group copies its scores
// to registers at once, so the buffer is free again long before the other group needs it),
// O_0 [128,272), O_1 [272,416), scale factors from 416.
//
// Epilogue: O = O~ / l; the bf16 result is staged in shared memory (one 32-row x 128-byte box per softmax warp,
// 128-byte swizzle) and leaves as one tensor copy per warp through a tensor map of the output, so that whole
// lines are written and the stores do not queue in front of the next tile's shared-memory traffic.
//
// Two launch shapes: one CTA per work item (two query tiles of one head), or -- more items than SMs and a short
// KV sequence -- one CTA per SM that walks the items and keeps barriers, tensor memory and the K/V ring across
// them (template flag kPersist).
//
// Every mbarrier wait is bounded; on expiry the CTA records a code in `status`, drains and exits.
#include <cuda.h>              // CUtensorMap and the enumerations of its encoder (types only: nothing links libcuda)
#include <cudaTypedefs.h>

#include <string.h>

#include <type_traits>

#include "common.cuh"
#include "tc_helpers.cuh"

namespace mxattn {
namespace fwd {

constexpr int kSplit = 2;                        // threads per query row (one per row measured 25 % slower)
constexpr int kCols = kTile / kSplit;            // key columns per softmax thread
constexpr int kBlocksPerThread = 4 / kSplit;
constexpr int kSoftmaxWarps = 8 * kSplit;
constexpr int kThreads = 32 * (kSoftmaxWarps + 2);   // softmax warps + producer + MMA issuer
constexpr int kStages = 4;
constexpr int kNV = 144;                         // GEMM 2 N: 128 channels + 16 rows of ones
constexpr int kVStageBytes = kNV * 64;           // 9216
constexpr int kDumpTileBytes = kTileCodeBytes + kTileScaleBytes + kTile * 4;   // debug dump: codes, scale atom, m per row

// shared memory map (byte offsets from a 1024-aligned base)
constexpr int kOffQ = 0;                                   // 2 buffers x 2 tiles x 8192 (the second buffer: persistent variant)
constexpr int kOffK = kOffQ + 4 * kTileCodeBytes;          // 4 x 8192
constexpr int kOffV = kOffK + kStages * kTileCodeBytes;    // 4 x 9216
constexpr int kOffP = kOffV + kStages * kVStageBytes;      // 2 x 8192
constexpr int kOffSFQ = kOffP + 2 * kTileCodeBytes;        // 2 buffers x 2 x 512
constexpr int kOffSFK = kOffSFQ + 4 * kTileScaleBytes;     // 4 x 512
constexpr int kOffSFV = kOffSFK + kStages * kTileScaleBytes;   // 4 x 512
constexpr int kOffSFOnes = kOffSFV + kStages * kTileScaleBytes; // 512
constexpr int kOffSFP = kOffSFOnes + kTileScaleBytes;      // 2 x 512
constexpr int kOffBar = kOffSFP + 2 * kTileScaleBytes;     // barriers
constexpr int kNumBars = 4 + 2 * kStages + 2 + 1 + 2 + 2;  // Q full/empty[2], K/V stage full+empty, S_full[2], S_free, P_full[2], O_done[2]
constexpr int kOffMisc = kOffBar + kNumBars * 8;           // tmem slot, abort flag
constexpr int kOffMax = kOffMisc + 64;                     // half-row maxima: [parity 2][tile 2][half 2][128] floats
#ifndef MXATTN_PERSIST_MAX_T
#define MXATTN_PERSIST_MAX_T 48
#endif
constexpr int kPersistMaxTiles = MXATTN_PERSIST_MAX_T;    // longest key/value sequence (in tiles) run by the persistent variant
constexpr int kOffOut = (kOffMax + 2 * 2 * 2 * 128 * 4 + 1023) & ~1023;   // bf16 output staging: one box per softmax warp
constexpr int kOutBoxBytes = 32 * kCols * 2;               // 32 rows x 64 bf16 (128 bytes, the span of the 128-byte swizzle)
constexpr int kSmemBytes = kOffOut + kSoftmaxWarps * kOutBoxBytes + 1024;   // + slack for the 1024 alignment
static_assert(kOffOut % 1024 == 0 && kOutBoxBytes % 1024 == 0, "swizzled boxes start on the swizzle pattern's period");
static_assert(kSmemBytes <= 227 * 1024, "shared memory per CTA");

enum Bar { BAR_Q = 0, BAR_QEMPTY = 2, BAR_KFULL = 4, BAR_KEMPTY = BAR_KFULL + kStages,     // one full / empty pair per K/V stage
           BAR_SFULL = BAR_KEMPTY + kStages, BAR_SFREE = BAR_SFULL + 2,
           BAR_PFULL = BAR_SFREE + 1, BAR_ODONE = BAR_PFULL + 2 };

// tensor-memory columns
constexpr uint32_t kColS = 0, kColO0 = 128, kColO1 = 272, kColSFQ = 416, kColSFK = 424,
                   kColSFV = 432, kColSFP = 448;

struct Params {
  const uint8_t* q_codes; const uint8_t* q_scales;
  const uint8_t* k_codes; const uint8_t* k_scales;
  const uint8_t* v_codes; const uint8_t* v_scales;
  void* out;
  int* status;
  uint8_t* dump;        // per-tile P-hat images, scales, running maxima and final row sums (debug entry point only)
  int64_t Nq, Nkv;
  int q_tiles, kv_tiles, q_pairs;
  int total_items;      // B * H * q_pairs work items (one = two query tiles of one head)
  float scale_log2e;    // softmax_scale * log2(e)
  float softmax_scale;
};

// ---------------------------------------------------------------------------------------------
// kPersist: the CTA walks several work items (blockIdx.x, blockIdx.x + gridDim.x, ...) and keeps its barriers,
// tensor memory and pipelines across them: the next item's Q tiles and first K/V tiles are fetched and its first
// scores computed while the current item drains.  Used for short KV sequences, where the per-CTA set-up, the
// latency of the first loads and the launch gap between CTAs are a large share of an item's time.
// Waits of the single-thread roles.  In the item-walking variant their loops carry the item bookkeeping as well, and
// keeping the waits' slow path out of line there shortens the time per tile by 6 %; in the one-item variant the same
// change measured 3 % slower, so that one keeps the inline form.
// kProf (cycle profile, never in a timed build): every role accumulates SM cycles per phase of its loop and writes them
// to p.dump as [CTA][warp 0..17][16] int64 (softmax warps: slots 0-8 = S-full wait, score load, maxima, pair
// exchange, O-done wait, block exponents, exponentials + pack, hand-over, epilogue; slot 9 = tiles; producer and
// issuer: slots 0-7 = cycles inside the wait with code c at slot c mod 8, slot 8 = cycles of the whole loop, slot 9 = tiles).
#define MBAR_WAIT_ROLE(...) (kProf ? prof_wait(__VA_ARGS__) : (kPersist ? mbar_wait1(__VA_ARGS__) : mbar_wait(__VA_ARGS__)))
#define PROF_MARK(i) do { if (kProf) { const long long prof_now = clock64(); prof_t[i] += prof_now - prof_prev; prof_prev = prof_now; } } while (0)
constexpr int kProfSlots = 16;
template <bool kUos, bool kPnq, bool kOutF32, bool kDump, bool kPersist, bool kProf = false>
__global__ void __launch_bounds__(kThreads, 1) attention_kernel(const Params p, const __grid_constant__ CUtensorMap out_map) {
  static_assert(!(kDump && kPersist), "the tile dump is written by the one-item-per-CTA variant only");
  static_assert(!(kDump && kProf), "the dump buffer holds either the tile dump or the cycle profile");
  long long prof_t[kProfSlots];
  long long prof_prev = 0;
  if (kProf) {
#pragma unroll
    for (int i = 0; i < kProfSlots; ++i) prof_t[i] = 0;
  }
  auto prof_wait = [&](uint32_t b, uint32_t par, volatile int* af, int* st, int code) {
    const long long t0 = clock64();
    const bool r = mbar_wait(b, par, af, st, code);
    prof_t[code & 7] += clock64() - t0;
    return r;
  };
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t sbase = smem_u32(smem);
  const uint32_t bar0 = sbase + kOffBar;
  auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + kOffMisc);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + kOffMisc + 8);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (*reinterpret_cast<volatile int*>(p.status) != 0) return;   // an earlier CTA gave up: drain the grid quickly
  const int T = p.kv_tiles;
  const int bh0 = blockIdx.x / p.q_pairs, pair0 = blockIdx.x - bh0 * p.q_pairs;

  // ---- setup -------------------------------------------------------------------------------
  if (tid == 0) {
    mbar_init(bar(BAR_Q + 0), 1); mbar_init(bar(BAR_Q + 1), 1);
    mbar_init(bar(BAR_QEMPTY + 0), 1); mbar_init(bar(BAR_QEMPTY + 1), 1);
    for (int s = 0; s < kStages; ++s) {
      mbar_init(bar(BAR_KFULL + s), 1); mbar_init(bar(BAR_KEMPTY + s), 1);
    }
    mbar_init(bar(BAR_SFULL + 0), 1); mbar_init(bar(BAR_SFULL + 1), 1);
    mbar_init(bar(BAR_SFREE), 4 * kSplit);                  // one arrival per softmax warp of the draining group
    mbar_init(bar(BAR_PFULL + 0), 4 * kSplit); mbar_init(bar(BAR_PFULL + 1), 4 * kSplit);   // one arrival per softmax warp
    mbar_init(bar(BAR_ODONE + 0), 1); mbar_init(bar(BAR_ODONE + 1), 1);
    abort_flag[0] = 0;
    abort_flag[1] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // constant rows of ones appended to every V stage (E2M1 code 2 = 1.0) and their scale atom (2^0)
  for (int i = tid; i < kStages * 16 * 64 / 16; i += kThreads) {
    const int s = i / 64, c = i % 64;
    reinterpret_cast<uint4*>(smem + kOffV + s * kVStageBytes + kTileCodeBytes)[c] =
        make_uint4(0x22222222u, 0x22222222u, 0x22222222u, 0x22222222u);
  }
  for (int i = tid; i < kTileScaleBytes / 16; i += kThreads)
    reinterpret_cast<uint4*>(smem + kOffSFOnes)[i] = make_uint4(0x7F7F7F7Fu, 0x7F7F7F7Fu, 0x7F7F7F7Fu, 0x7F7F7F7Fu);
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
      int F = 0;                                   // tiles issued so far, over all items of this CTA
      int q_issued = 0;                            // items whose Q tiles were issued
      bool ok = true;
      if (kProf) prof_prev = clock64();
      for (int n = 0, item = blockIdx.x; (kPersist ? item < p.total_items : n < 1) && ok; ++n, item += gridDim.x) {
        const int bh = item / p.q_pairs, pair = item - bh * p.q_pairs;
        const int qb = kPersist ? (n & 1) : 0;     // Q buffer
        // the Q buffer of item n - 2 is free once every GEMM 1 of that item has completed
        if (kPersist && n >= 2) ok = MBAR_WAIT_ROLE(bar(BAR_QEMPTY + qb), (uint32_t)(((n - 2) >> 1) & 1), abort_flag, p.status, 13);
        if (!ok) break;
        const int64_t qt0 = (int64_t)bh * p.q_tiles + 2 * pair;
        const int64_t qt1 = (2 * pair + 1 < p.q_tiles) ? qt0 + 1 : qt0;     // odd tail: reuse tile 0 (result unused)
        const uint32_t sq = sbase + kOffQ + qb * 2 * kTileCodeBytes, ssf = sbase + kOffSFQ + qb * 2 * kTileScaleBytes;
        mbar_expect_tx(bar(BAR_Q + qb), 2 * (kTileCodeBytes + kTileScaleBytes));
        bulk_g2s(sq, p.q_codes + qt0 * kTileCodeBytes, kTileCodeBytes, bar(BAR_Q + qb));
        bulk_g2s(sq + kTileCodeBytes, p.q_codes + qt1 * kTileCodeBytes, kTileCodeBytes, bar(BAR_Q + qb));
        bulk_g2s(ssf, p.q_scales + qt0 * kTileScaleBytes, kTileScaleBytes, bar(BAR_Q + qb));
        bulk_g2s(ssf + kTileScaleBytes, p.q_scales + qt1 * kTileScaleBytes, kTileScaleBytes, bar(BAR_Q + qb));
        q_issued = n + 1;
        const int64_t kv0 = (int64_t)bh * T;
        for (int j = 0; j < T && ok; ++j, ++F) {
          const int s = F % kStages;
          const uint32_t ph = (uint32_t)((F / kStages) & 1);
          if (F >= kStages) ok = MBAR_WAIT_ROLE(bar(BAR_KEMPTY + s), ph ^ 1u, abort_flag, p.status, 11);
          if (!ok) break;
          // K-hat_j and V-hat_j travel together: one full / one empty barrier per stage (the issuer thread's time
          // per tile is what bounds the kernel, and every wait or commit it does not need shortens it)
          mbar_expect_tx(bar(BAR_KFULL + s), 2 * (kTileCodeBytes + kTileScaleBytes));
          bulk_g2s(sbase + kOffK + s * kTileCodeBytes, p.k_codes + (kv0 + j) * kTileCodeBytes, kTileCodeBytes, bar(BAR_KFULL + s));
          bulk_g2s(sbase + kOffSFK + s * kTileScaleBytes, p.k_scales + (kv0 + j) * kTileScaleBytes, kTileScaleBytes, bar(BAR_KFULL + s));
          bulk_g2s(sbase + kOffV + s * kVStageBytes, p.v_codes + (kv0 + j) * kTileCodeBytes, kTileCodeBytes, bar(BAR_KFULL + s));
          bulk_g2s(sbase + kOffSFV + s * kTileScaleBytes, p.v_scales + (kv0 + j) * kTileScaleBytes, kTileScaleBytes, bar(BAR_KFULL + s));
        }
      }
      if (kProf) { prof_t[8] = clock64() - prof_prev; prof_t[9] = F; }
      if (!ok || *abort_flag) {
        // gave up: let copies already in flight land before the CTA's shared memory is released
        const long long t0 = clock64();
        for (int f = (F > kStages ? F - kStages : 0); f < F; ++f)
          while (!mbar_try(bar(BAR_KFULL + f % kStages), (uint32_t)((f / kStages) & 1)) && clock64() - t0 < 200000000LL) {}
        for (int n = (q_issued > 2 ? q_issued - 2 : 0); n < q_issued; ++n) {
          const int qb = kPersist ? (n & 1) : 0;
          while (!mbar_try(bar(BAR_Q + qb), (uint32_t)((kPersist ? (n >> 1) : 0) & 1)) && clock64() - t0 < 200000000LL) {}
        }
      }
    }
  } else if (warp == kSoftmaxWarps + 1) {
    // =============================== MMA issuer =============================================
    if (lane == 0) {
      if (kProf) prof_prev = clock64();
      bool ok = MBAR_WAIT_ROLE(bar(BAR_Q), 0, abort_flag, p.status, 21);
      uint32_t sfree_n = 0;      // completed phases of S_FREE consumed so far
      // Descriptor words are loop invariants up to a stage offset: the low word is the shared
      // address >> 4 (all tiles sit below 256 KiB, so it fits the 14-bit field), the high word is
      // constant (stride between 8-row groups, descriptor version, swizzle mode).
      constexpr uint32_t kDescHiTile = (512u >> 4) | (1u << 14) | (4u << 29);   // 64-byte swizzle, K-major
      const uint32_t q_lo = (sbase + kOffQ) >> 4, k_lo = (sbase + kOffK) >> 4;
      const uint32_t v_lo = (sbase + kOffV) >> 4, p_lo = (sbase + kOffP) >> 4;
      auto desc = [](uint32_t lo) { return ((uint64_t)kDescHiTile << 32) | lo; };
      // A tile is named by its item n (0, 1, ... of this CTA), its index j inside the item and its index f among
      // all tiles of the CTA (f = n T + j; f = j without kPersist).  Stages, slots and barrier parities follow f.
      auto gemm1 = [&](int t, int n, int j, int f) {      // S = Q_t K_j^T
        const uint32_t a = q_lo + (uint32_t)t * (kTileCodeBytes >> 4);
        const uint32_t b = k_lo + (uint32_t)(f % kStages) * (kTileCodeBytes >> 4);
        const uint32_t sfa = tmem + kColSFQ + 4 * t, sfb = tmem + kColSFK + 4 * (f & 1);
        tc_mma(tmem + kColS, desc(a), desc(b), make_idesc(128, 0), sfa, sfb, 0u);
        tc_mma(tmem + kColS, desc(a + 2), desc(b + 2), make_idesc(128, 1), sfa, sfb, 1u);   // K 64..127: +32 bytes
        tc_commit(bar(BAR_SFULL + t));
        return true;
      };
      auto gemm2 = [&](int t, int n, int j, int f) {      // O_t += P_t [V_j | 1]
        tc_cp_sf(tmem + kColSFP + 4 * t, sbase + kOffSFP + t * kTileScaleBytes);
        const uint32_t a = p_lo + (uint32_t)t * (kTileCodeBytes >> 4);
        const uint32_t b = v_lo + (uint32_t)(f % kStages) * (kVStageBytes >> 4);
        const uint32_t d = tmem + (t ? kColO1 : kColO0);
        const uint32_t sfa = tmem + kColSFP + 4 * t, sfb = tmem + kColSFV + 8 * (f & 1);
        tc_mma(d, desc(a), desc(b), make_idesc(kNV, 0), sfa, sfb, j > 0 ? 1u : 0u);
        tc_mma(d, desc(a + 2), desc(b + 2), make_idesc(kNV, 1), sfa, sfb, 1u);
        tc_commit(bar(BAR_ODONE + t));
        return true;
      };
      // K-hat and V-hat of tile f have landed (and, unless `first`, the score buffer is free): one fence, then the
      // scale atoms of both go to tensor memory -- V's two tiles ahead of its GEMM, which keeps that copy out of the
      // path from "P is ready" to "GEMM 2 issued" (slot f & 1 was last read by the GEMMs of tile f - 2, issued before)
      auto wait_kv = [&](int f, bool first) {
        const int s = f % kStages;
        if (!MBAR_WAIT_ROLE(bar(BAR_KFULL + s), (uint32_t)((f / kStages) & 1), abort_flag, p.status, 22)) return false;
        if (!first) {
          if (!MBAR_WAIT_ROLE(bar(BAR_SFREE), sfree_n & 1u, abort_flag, p.status, 23)) return false;
          ++sfree_n;
        }
        tc_fence_after();
        tc_cp_sf(tmem + kColSFK + 4 * (f & 1), sbase + kOffSFK + s * kTileScaleBytes);
        tc_cp_sf(tmem + kColSFV + 8 * (f & 1), sbase + kOffSFV + s * kTileScaleBytes);
        return true;
      };
      auto wait_sfree = [&]() {
        const bool r = MBAR_WAIT_ROLE(bar(BAR_SFREE), sfree_n & 1u, abort_flag, p.status, 23);
        ++sfree_n;
        tc_fence_after();
        return r;
      };
      if (ok) {
        tc_fence_after();
        tc_cp_sf(tmem + kColSFQ + 0, sbase + kOffSFQ);
        tc_cp_sf(tmem + kColSFQ + 4, sbase + kOffSFQ + kTileScaleBytes);
        tc_cp_sf(tmem + kColSFV + 4, sbase + kOffSFOnes);        // scales of the ones rows, both slots
        tc_cp_sf(tmem + kColSFV + 12, sbase + kOffSFOnes);
      }
      // K-hat of tile f has landed: its scale atom goes to tensor memory (slot f & 1 was last read by the score products
      // of tile f - 2, issued before).  Kept apart from the wait for the score buffer, so that nothing but that wait
      // stands between "the other group has taken its scores" and the next score product.
      auto k_ready = [&](int f) {
        const int s = f % kStages;
        if (!MBAR_WAIT_ROLE(bar(BAR_KFULL + s), (uint32_t)((f / kStages) & 1), abort_flag, p.status, 22)) return false;
        tc_fence_after();
        tc_cp_sf(tmem + kColSFK + 4 * (f & 1), sbase + kOffSFK + s * kTileScaleBytes);
        return true;
      };
      // V-hat's scale atom of tile f (its stage has landed together with K-hat's; slot f & 1 was last read by the output
      // products of tile f - 2)
      auto v_scales = [&](int f) { tc_cp_sf(tmem + kColSFV + 8 * (f & 1), sbase + kOffSFV + (f % kStages) * kTileScaleBytes); };
      if (!kPersist) {
        // prologue: S(0,0), S(1,0), S(0,1)
        ok = ok && k_ready(0);
        if (ok) { v_scales(0); gemm1(0, 0, 0, 0); }
        ok = ok && wait_sfree();
        if (ok) gemm1(1, 0, 0, 0);
        if (T > 1) {
          ok = ok && k_ready(1);
          if (ok) v_scales(1);
          ok = ok && wait_sfree();
          if (ok) gemm1(0, 0, 1, 1);
        }
        // unrolled by the number of stages: stage indices, parities and descriptor offsets become constants, and the
        // thread's scalar instructions between its tcgen05 instructions are part of the kernel's critical path
#pragma unroll 4
        for (int j = 0; j < T && ok; ++j) {
          const int s = j % kStages;
          ok = MBAR_WAIT_ROLE(bar(BAR_PFULL + 0), (uint32_t)(j & 1), abort_flag, p.status, 24);     // V_j arrived with K_j
          if (!ok) break;
          tc_fence_after();
          gemm2(0, 0, j, j);
          if (j + 1 < T) {
            ok = wait_sfree();
            if (!ok) break;
            gemm1(1, 0, j + 1, j + 1);
          }
          if (j + 2 < T) {                           // off the critical chain: the thread would wait for P-hat here anyway
            ok = k_ready(j + 2);
            if (!ok) break;
          }
          ok = MBAR_WAIT_ROLE(bar(BAR_PFULL + 1), (uint32_t)(j & 1), abort_flag, p.status, 26);
          if (!ok) break;
          tc_fence_after();
          gemm2(1, 0, j, j);
          if (j + 2 < T) {
            ok = wait_sfree();
            if (!ok) break;
            gemm1(0, 0, j + 2, j + 2);
          }
          tc_commit(bar(BAR_KEMPTY + s));            // K_j and V_j may be overwritten once everything issued so far has completed
          if (j + 2 < T) v_scales(j + 2);
        }
      } else {
        // The same instruction stream over all tiles of all items of this CTA, f = 0 .. F_end - 1: the scores of
        // the next item's first tiles are issued while the current item's last tiles are still in the softmax warps.
        // Per tile the thread keeps one cursor (item n0, tile j0 of tile f) and derives two flags from it; what an
        // item boundary adds is then one branch per GEMM 1.  `edge` of a GEMM 1 means: for query tile 0, the first
        // tile of an item other than the CTA's first (wait for its Q tiles, copy their scales: every GEMM 1 of the
        // previous item has been issued by then); for query tile 1, the last tile of its item (release the Q buffer).
        // No barrier guards the accumulators across items: GEMM 2 of an item's first tile waits for that tile's
        // P-hat, which the group's warps publish after their epilogue has read the previous item's accumulator.
        const int n_items = (p.total_items - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;
        const int F_end = n_items * T;
        auto gemm1p = [&](int t, int n, int f, bool edge) {      // n: the item of tile f
          const int qb = n & 1;
          if (t == 0 && edge) {
            if (!MBAR_WAIT_ROLE(bar(BAR_Q + qb), (uint32_t)((n >> 1) & 1), abort_flag, p.status, 21)) return false;
            tc_fence_after();
            tc_cp_sf(tmem + kColSFQ + 0, sbase + kOffSFQ + qb * 2 * kTileScaleBytes);
            tc_cp_sf(tmem + kColSFQ + 4, sbase + kOffSFQ + (qb * 2 + 1) * kTileScaleBytes);
          }
          const uint32_t a = q_lo + (uint32_t)(qb * 2 + t) * (kTileCodeBytes >> 4);
          const uint32_t b = k_lo + (uint32_t)(f % kStages) * (kTileCodeBytes >> 4);
          const uint32_t sfa = tmem + kColSFQ + 4 * t, sfb = tmem + kColSFK + 4 * (f & 1);
          tc_mma(tmem + kColS, desc(a), desc(b), make_idesc(128, 0), sfa, sfb, 0u);
          tc_mma(tmem + kColS, desc(a + 2), desc(b + 2), make_idesc(128, 1), sfa, sfb, 1u);
          tc_commit(bar(BAR_SFULL + t));
          if (t == 1 && edge) tc_commit(bar(BAR_QEMPTY + qb));
          return true;
        };
        const bool one = (T == 1);
        int n0 = 0, j0 = 0;                          // tile f
        ok = ok && wait_kv(0, true);
        if (ok) ok = gemm1p(0, 0, 0, false);
        ok = ok && wait_sfree();
        if (ok) ok = gemm1p(1, 0, 0, one);
        if (F_end > 1) {
          ok = ok && wait_kv(1, false);
          if (ok) ok = gemm1p(0, one ? 1 : 0, 1, one);
        }
#pragma unroll 4
        for (int f = 0; f < F_end && ok; ++f) {
          const bool item_end = (j0 == T - 1);       // tile f + 1 starts an item
          const bool pre_end = one || (j0 == T - 2); // tile f + 1 ends an item, tile f + 2 starts one
          const int n1 = n0 + (item_end ? 1 : 0), n2 = n1 + (pre_end ? 1 : 0);
          ok = MBAR_WAIT_ROLE(bar(BAR_PFULL + 0), (uint32_t)(f & 1), abort_flag, p.status, 24);
          if (!ok) break;
          tc_fence_after();
          gemm2(0, 0, j0, f);
          // On the last tile of an item the score buffer is released only after the first group's epilogue, so
          // the second group's GEMM 2 (and with it that group's epilogue) goes first there.
          if (!item_end && f + 1 < F_end) {
            ok = wait_sfree();
            if (!ok) break;
            ok = gemm1p(1, n1, f + 1, pre_end);
            if (!ok) break;
          }
          ok = MBAR_WAIT_ROLE(bar(BAR_PFULL + 1), (uint32_t)(f & 1), abort_flag, p.status, 26);
          if (!ok) break;
          tc_fence_after();
          gemm2(1, 0, j0, f);
          tc_commit(bar(BAR_KEMPTY + f % kStages));
          if (item_end && f + 1 < F_end) {
            ok = wait_sfree();
            if (!ok) break;
            ok = gemm1p(1, n1, f + 1, pre_end);
            if (!ok) break;
          }
          if (f + 2 < F_end) {
            ok = wait_kv(f + 2, false);
            if (!ok) break;
            ok = gemm1p(0, n2, f + 2, pre_end);
            if (!ok) break;
          }
          if (++j0 == T) { j0 = 0; ++n0; }
        }
      }
      if (kProf) {
        prof_t[8] = clock64() - prof_prev;
        prof_t[9] = kPersist ? (long long)((p.total_items - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x) * T : T;
      }
    }
  } else if (warp < kSoftmaxWarps) {
    // =============================== softmax groups =========================================
    const int t = warp >> 3;                       // query tile of this group
    const int h = (warp >> 2) & 1;                 // which 64 key columns of the tile
    const int row = (warp & 3) * 32 + lane;        // row within the tile == TMEM lane
    const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t t_s = tmem + kColS + lane_addr + kCols * h;
    const uint32_t t_o = tmem + (t ? kColO1 : kColO0) + lane_addr;     // column 0 of this row's accumulator
    const float c = p.scale_log2e;
    float m_run, l_run;                            // l_run: direct placement only (this thread's 64 columns)
    // shared-space byte addresses of this thread's slots: its two 16-byte code chunks, its two scale
    // bytes, and the half-row maximum exchange (own slot / partner's slot; + 2048 on odd tiles)
    const uint32_t aP0 = sbase + kOffP + t * kTileCodeBytes + tile_code_offset(row, 2 * h);
    const uint32_t aP1 = sbase + kOffP + t * kTileCodeBytes + tile_code_offset(row, 2 * h + 1);
    const uint32_t aSF = sbase + kOffSFP + t * kTileScaleBytes + tile_scale_offset(row, 2 * h);
    const uint32_t aMaxOwn = sbase + kOffMax + (t * 256 + h * 128 + row) * 4;
    const uint32_t aMaxPartner = sbase + kOffMax + (t * 256 + (h ^ 1) * 128 + row) * 4;
    const int pair_bar = 1 + (warp & 3) + 4 * t;   // named barrier shared with the partner warp (w, w^4)
    // The two warps of a pair meet at a named barrier in every tile (and once more per item under direct placement).
    // A warp whose bounded wait has run out therefore does not leave: it stops computing and waiting, but keeps every
    // remaining appointment with its partner (keep_company below), for this item and all later ones, so that the
    // partner -- which may have found the same mbarrier complete a moment earlier -- is never left alone at the
    // barrier.  The hot path carries no check for this.  Their waits watch a flag that nothing sets (they give up on
    // their own cycle limit only) and raise the CTA's flag on expiry.
    volatile int* const own_limit_only = abort_flag + 1;
    bool ok = true;
    // Work items of this CTA (exactly one without kPersist).  F0 = tiles of the earlier items: the parities of the
    // barriers that complete once per tile follow F0 + j.  X0 counts the earlier exchanges through the half-row
    // slots (one per tile, plus the row-sum exchange of direct placement), which alternate between two buffers.
    int item = blockIdx.x, F0 = 0, X0 = 0;
    do {
    int bh = bh0, pair = pair0;                     // with kPersist: set in the epilogue, the only place that needs them
    m_run = -INFINITY;
    l_run = 0.0f;

    int j = 0;                                      // after the loop: the first tile whose meeting has not been kept yet
    if (kProf && F0 == 0) prof_prev = clock64();
    if (ok) for (; j < T; ++j) {
      ok = __all_sync(0xFFFFFFFFu, mbar_wait(bar(BAR_SFULL + t), (uint32_t)((F0 + j) & 1), own_limit_only, p.status, 31, kWaitLimitCycles, abort_flag));
      if (!ok) break;
      PROF_MARK(0);
      tc_fence_after();
      uint32_t sr[kCols];
      TMEM_LD64(t_s, sr);
      tmem_ld_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(BAR_SFREE));  // the score buffer may be overwritten
      PROF_MARK(1);

      if (j == T - 1) {                            // ragged last tile: keys beyond Nkv do not exist
        const int valid = (int)(p.Nkv - (int64_t)j * kTile) - kCols * h;
#pragma unroll
        for (int i = 0; i < kCols; ++i)
          if (i >= valid) sr[i] = 0xFF800000u;     // -inf
      }
      float bmax[kBlocksPerThread];
#pragma unroll
      for (int b = 0; b < kBlocksPerThread; ++b) {  // four independent chains of 8, then combine
        float q4[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const uint32_t* v = sr + 32 * b + 8 * u;
          float mx = max3(__uint_as_float(v[0]), __uint_as_float(v[1]), __uint_as_float(v[2]));
          mx = max3(mx, __uint_as_float(v[3]), __uint_as_float(v[4]));
          mx = max3(mx, __uint_as_float(v[5]), __uint_as_float(v[6]));
          q4[u] = fmaxf(mx, __uint_as_float(v[7]));
        }
        bmax[b] = fmaxf(max3(q4[0], q4[1], q4[2]), q4[3]);
      }
      float own_max = bmax[0];
#pragma unroll
      for (int b = 1; b < kBlocksPerThread; ++b) own_max = fmaxf(own_max, bmax[b]);
      // half-row maximum -> partner thread (same row, other 64 columns), double-buffered by tile parity
      const uint32_t par = (uint32_t)((X0 + j) & 1) * 2048u;
      PROF_MARK(2);
      sts32f(aMaxOwn + par, own_max);
      asm volatile("bar.sync %0, 64;" ::"r"(pair_bar) : "memory");      // only the two warps that share these rows
      const float partner_max = lds32f(aMaxPartner + par);
      PROF_MARK(3);
      // GEMM 2 of the previous tile must have read P_t and updated O_t before this tile writes P_t or rescales
      // O_t; the probe of that barrier is issued while the partner's maximum is on its way
      const bool o_ready = (j == 0) || mbar_test(bar(BAR_ODONE + t), (uint32_t)((F0 + j - 1) & 1));
      const float m_new = max3(m_run, own_max, partner_max);   // line 10
      const bool moved = (m_new != m_run) && (j > 0);
      const float m_old = m_run;
      m_run = m_new;
      const float nmc = -(m_new * c);
      if (!__all_sync(0xFFFFFFFFu, o_ready)) {
        ok = __all_sync(0xFFFFFFFFu, mbar_wait(bar(BAR_ODONE + t), (uint32_t)((F0 + j - 1) & 1), own_limit_only, p.status, 32, kWaitLimitCycles, abort_flag));
        if (!ok) { ++j; break; }                   // this tile's meeting has been kept
      }
      tc_fence_after();
      PROF_MARK(4);
      const bool rescale = __any_sync(0xFFFFFFFFu, moved);     // line 15: O~ <- Diag(alpha) O~
      // alpha = exp(m_old - m_new) (line 11) is exactly 1 for every row of a warp in which no maximum
      // moved, so it is only evaluated on the rescaling path
      float alpha = 1.0f;

      // lines 12-13: exponentials, already divided by the block scale, rounded to E2M1.  Two
      // straight-line versions: the common one, and one that also rescales this thread's 64
      // accumulator columns with the tensor-memory round trips interleaved into the exponentials.
      // Shared exponent of each block from d = log2(pmax) = (bmax_b - m_new) * c <= 0, with no
      // exponential: floor(log2 pmax) = floor(d), and the UOS rule raises the exponent iff the
      // mantissa 2^(d - floor d) exceeds 1.8125, i.e. iff frac(d) > log2(1.8125).  d = 0 (the
      // block holding the row maximum) gives e = -2 under both rules, as Appendix J derives.
      // A block whose maximum underflows fp32 (d < -126, or fully masked) is a zero block.
      float nbs[kBlocksPerThread], sigma[kBlocksPerThread];
      uint32_t sf_half = 0;
#pragma unroll
      for (int b = 0; b < kBlocksPerThread; ++b) {
        const float d = (bmax[b] - m_new) * c;
        const float rn = (d + 12582912.0f) - 12582912.0f;              // round to nearest integer
        const float fl = rn > d ? rn - 1.0f : rn;                       // floor(d)
        float ef = fl - 2.0f;
        if (kUos && (d - fl) > 0.85798097f) ef += 1.0f;
        ef = fmaxf(ef, -127.0f);
        if (d < -126.0f) ef = 0.0f;
        const int e = __float_as_int(ef + 12582912.0f) - 0x4B400000;    // exact small-integer conversion
        nbs[b] = nmc - ef;
        sigma[b] = __uint_as_float((uint32_t)(127 + e) << 23);          // 2^e (direct placement only)
        sf_half |= (uint32_t)(e + 127) << (8 * b);
      }
      // the scale bytes go out before the exponentials, so only the code stores precede the proxy fence
      sts16(aSF, sf_half);
      PROF_MARK(5);
      uint8_t* dump_tile = nullptr;
      if (kDump && 2 * pair + t < p.q_tiles) {       // image of this (query tile, KV tile): codes, scale atom, m
        dump_tile = p.dump + ((((int64_t)bh * p.q_tiles + 2 * pair + t) * T) + j) * kDumpTileBytes;
        *reinterpret_cast<uint16_t*>(dump_tile + kTileCodeBytes + tile_scale_offset(row, 2 * h)) = (uint16_t)sf_half;
        if (h == 0) reinterpret_cast<float*>(dump_tile + kTileCodeBytes + kTileScaleBytes)[row] = m_new * p.softmax_scale;   // the kernel keeps m in unscaled score units
      }
      float l_tile = 0.0f;
      const uint64_t cc2 = dup2(c);
      auto tile_body = [&](auto resc_tag) {
        constexpr bool kResc = decltype(resc_tag)::value;
        if (kResc) alpha = ex2((m_old - m_new) * c);
#pragma unroll
        for (int b = 0; b < kBlocksPerThread; ++b) {
          const uint64_t nb2 = dup2(nbs[b]);
          uint4 w;
          float sx = 0.0f;
#pragma unroll
          for (int g = 0; g < 4; ++g) {             // 8 elements per step (8 accumulator columns in flight)
            uint32_t oc[8];
            const uint32_t t_oc = t_o + kCols * h + 32 * b + 8 * g;
            if (kResc) TMEM_LD8(t_oc, oc);
            float x[8];
#pragma unroll
            for (int i = 0; i < 8; i += 2) {           // x = exp2(s * c + nb), two elements per multiply-add
              fma2(sr[32 * b + 8 * g + i], sr[32 * b + 8 * g + i + 1], cc2, nb2, x[i], x[i + 1]);
              x[i] = ex2(x[i]);
              x[i + 1] = ex2(x[i + 1]);
            }
            const uint32_t pk = pack_e2m1x8(x[0], x[1], x[2], x[3], x[4], x[5], x[6], x[7]);
            if (g == 0) w.x = pk; else if (g == 1) w.y = pk; else if (g == 2) w.z = pk; else w.w = pk;
            if (!kPnq) {                              // two packed additions and three plain ones per eight elements
              float s0, s1;
              add2x2(x[0], x[1], x[2], x[3], x[4], x[5], x[6], x[7], s0, s1);
              sx += s0 + s1;
            }
            if (kResc) {
              tmem_ld_wait();
#pragma unroll
              for (int i = 0; i < 8; ++i) oc[i] = __float_as_uint(__uint_as_float(oc[i]) * alpha);
              TMEM_ST8(t_oc, oc);
            }
          }
          sts128(b == 0 ? aP0 : aP1, w);
          if (kDump && dump_tile) *reinterpret_cast<uint4*>(dump_tile + tile_code_offset(row, kBlocksPerThread * h + b)) = w;
          if (!kPnq) l_tile = fmaf(sx, sigma[b], l_tile);   // Eq. 12
        }
        if (kResc) {
          if (kPnq && h == 0) {                     // column 128: the running row sum P-hat 1
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
      if (!kPnq) l_run = fmaf(alpha, l_run, l_tile);                         // line 14 (direct)
      PROF_MARK(6);
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(BAR_PFULL + t));
      PROF_MARK(7);
      if (kProf) prof_t[9] += 1;
    }

    if (!ok) pair_keep_company(pair_bar, T - j);    // gave up (now or in an earlier item): only the meetings are kept

    // ---- epilogue: O = O~ / l (line 18) ----
    if (kPersist && !kOutF32) {                    // the previous item's output copy has read this warp's box
      if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
      __syncwarp();
    }
    if (ok) ok = __all_sync(0xFFFFFFFFu, mbar_wait(bar(BAR_ODONE + t), (uint32_t)((F0 + T - 1) & 1), own_limit_only, p.status, 33, kWaitLimitCycles, abort_flag));
    float l = l_run;
    if (!kPnq) {                                   // add the partner's half of the row sum (a meeting that is always kept)
      const uint32_t par = (uint32_t)((X0 + T) & 1) * 2048u;
      sts32f(aMaxOwn + par, l_run);
      asm volatile("bar.sync %0, 64;" ::"r"(pair_bar) : "memory");
      l = l_run + lds32f(aMaxPartner + par);
    }
    if (ok) {
      tc_fence_after();
      if (kPersist) { bh = item / p.q_pairs; pair = item - bh * p.q_pairs; }
      const int qtile = 2 * pair + t;
      const int64_t grow = (int64_t)qtile * kTile + row;
      if (kPersist && !kOutF32) {
        // Item-walking variant: the epilogue is part of every item's critical path.  Row sum and all 64 accumulator
        // columns are loaded with one wait, then the bf16 rows go to this warp's swizzled box and out as one tensor
        // copy (see the comments of the general path).
        uint32_t lr = 0, r64[kCols];
        if (kPnq) asm volatile("tcgen05.ld.sync.aligned.32x32b.x1.b32 {%0}, [%1];" : "=r"(lr) : "r"(t_o + 128) : "memory");
        TMEM_LD64(t_o + kCols * h, r64);
        tmem_ld_wait();
        if (kPnq) l = __uint_as_float(lr);
        const float inv_l = 1.0f / l;
        const uint32_t aBox = sbase + kOffOut + (t * 8 + h * 4 + (row >> 5)) * kOutBoxBytes;
        const uint32_t aRow = aBox + (row & 31) * (kCols * 2);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          uint32_t hh[4];
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const float a = __uint_as_float(r64[8 * i + 2 * k]) * inv_l, b2 = __uint_as_float(r64[8 * i + 2 * k + 1]) * inv_l;
            asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(hh[k]) : "f"(b2), "f"(a));
          }
          sts128(aRow + ((i ^ (row & 7)) << 4), make_uint4(hh[0], hh[1], hh[2], hh[3]));
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0 && qtile < p.q_tiles && (int64_t)qtile * kTile + (row & ~31) < p.Nq) {
          asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%1, %2, %3}], [%4];"
                       ::"l"(&out_map), "r"(kCols * h), "r"(qtile * kTile + (row & ~31)), "r"(bh), "r"(aBox) : "memory");
          asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        }
      } else {
      if (kPnq) {
        uint32_t lr;
        asm volatile("tcgen05.ld.sync.aligned.32x32b.x1.b32 {%0}, [%1];" : "=r"(lr) : "r"(t_o + 128) : "memory");
        tmem_ld_wait();
        l = __uint_as_float(lr);
      }
      const bool store = (qtile < p.q_tiles) && (grow < p.Nq);
      const float inv_l = 1.0f / l;                // line 18 as one reciprocal and 64 multiplies per thread
      if (kDump && h == 0 && qtile < p.q_tiles)
        reinterpret_cast<float*>(p.dump + (int64_t)p.total_items / p.q_pairs * p.q_tiles * T * kDumpTileBytes)
            [((int64_t)bh * p.q_tiles + qtile) * kTile + row] = l;
      const int64_t obase = ((int64_t)bh * p.Nq + grow) * kHeadDim + kCols * h;
      if (kOutF32) {
#pragma unroll 1
        for (int c0 = 0; c0 < kCols; c0 += 32) {
          uint32_t r32[32];
          TMEM_LD32(t_o + kCols * h + c0, r32);
          tmem_ld_wait();
          if (store) {
            float4* dst = reinterpret_cast<float4*>(static_cast<float*>(p.out) + obase + c0);
#pragma unroll
            for (int i = 0; i < 8; ++i)
              dst[i] = make_float4(__uint_as_float(r32[4 * i]) * inv_l, __uint_as_float(r32[4 * i + 1]) * inv_l,
                                   __uint_as_float(r32[4 * i + 2]) * inv_l, __uint_as_float(r32[4 * i + 3]) * inv_l);
          }
        }
      } else {
        // bf16: the warp's 32 half rows (128 bytes each) go to shared memory and from there to global memory as one
        // tensor copy (box of 32 rows x 64 columns; rows at or beyond Nq are clipped by the copy).  Written from
        // registers, a warp's 16-byte stores land 256 bytes apart (one partly filled sector per lane and
        // instruction); and any store instruction of these warps queues 64 KiB per item in front of the next
        // tile's shared-memory traffic.  The box uses the 128-byte swizzle (16-byte chunk c of row r sits at
        // chunk c ^ (r & 7)), which also spreads a quarter warp's stores over all banks.
        const uint32_t aBox = sbase + kOffOut + (t * 8 + h * 4 + (row >> 5)) * kOutBoxBytes;    // one box per warp
        const uint32_t aRow = aBox + (row & 31) * (kCols * 2);
#pragma unroll 1
        for (int c0 = 0; c0 < kCols; c0 += 32) {
          uint32_t r32[32];
          TMEM_LD32(t_o + kCols * h + c0, r32);
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            uint32_t hh[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              const float a = __uint_as_float(r32[8 * i + 2 * k]) * inv_l, b2 = __uint_as_float(r32[8 * i + 2 * k + 1]) * inv_l;
              asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(hh[k]) : "f"(b2), "f"(a));
            }
            sts128(aRow + ((((c0 >> 3) + i) ^ (row & 7)) << 4), make_uint4(hh[0], hh[1], hh[2], hh[3]));
          }
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if ((row & 31) == 0 && qtile < p.q_tiles && (int64_t)qtile * kTile + (row & ~31) < p.Nq) {
          asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%1, %2, %3}], [%4];"
                       ::"l"(&out_map), "r"(kCols * h), "r"(qtile * kTile + (row & ~31)), "r"(bh), "r"(aBox) : "memory");
          asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        }
      }
      }
    }
    PROF_MARK(8);
    F0 += T;
    X0 += T + (kPnq ? 0 : 1);
    } while (kPersist && (item += (int)gridDim.x) < p.total_items);     // also after giving up: the meetings go on
  }

  if (kProf && lane == 0) {
    long long* dst = reinterpret_cast<long long*>(p.dump) + ((int64_t)blockIdx.x * (kThreads / 32) + warp) * kProfSlots;
#pragma unroll
    for (int i = 0; i < kProfSlots; ++i) dst[i] = prof_t[i];
  }
  // ---- teardown ------------------------------------------------------------------------------
  if (!kOutF32 && warp < kSoftmaxWarps && lane == 0)
    asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");     // the output copies have left shared memory
  tc_fence_before();
  __syncthreads();
  if (warp == kSoftmaxWarps + 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");
  }
}

// Self-test of the bounded wait: one warp waits on a barrier that nothing ever arrives on, with a
// short limit; the wait must give up, record its code in `status`, and the kernel must end normally.
__global__ void bounded_wait_selftest_kernel(int* status, long long limit_cycles) {
  __shared__ uint64_t barrier;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&barrier), 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  const bool done = mbar_wait(smem_u32(&barrier), 0u, &abort_flag, status, 77, limit_cycles);
  if (done && threadIdx.x == 0) atomicCAS(status, 0, -1);      // must not happen
}

// Self-test of the way two paired softmax warps stay in step when one of them gives up: warp 0 waits, with a short
// limit, on a barrier that nothing arrives on, gives up (code 77 in status[0]) and from then on only keeps the pair's
// `meetings` appointments (pair_keep_company, the routine the attention kernel uses); warp 1's own waits succeed, so it
// works through all its meetings, exchanging a value each time, and must come out of the last one: it then records
// the number of meetings it completed in status[1].  Nothing faults; the kernel ends normally.
__global__ void pair_abandon_selftest_kernel(int* status, long long limit_cycles, int meetings) {
  __shared__ uint64_t barriers[2];
  __shared__ int abort_flag[2];
  __shared__ float slots[2][32];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&barriers[0]), 1);           // never completes
    mbar_init(smem_u32(&barriers[1]), 1);           // completes at once
    abort_flag[0] = abort_flag[1] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    mbar_arrive(smem_u32(&barriers[1]));
  }
  __syncthreads();
  const int pair_bar = 1;
  int kept = 0;
  bool ok = true;
  for (; kept < meetings; ++kept) {
    ok = __all_sync(0xFFFFFFFFu, mbar_wait(smem_u32(&barriers[warp]), 0u, &abort_flag[1], status, 77, limit_cycles, &abort_flag[0]));
    if (!ok) break;
    sts32f(smem_u32(&slots[warp][lane]), (float)kept);
    asm volatile("bar.sync %0, 64;" ::"r"(pair_bar) : "memory");
  }
  if (!ok) pair_keep_company(pair_bar, meetings - kept);
  else if (lane == 0) atomicCAS(status + 1, 0, kept);
}

}  // namespace fwd

int launch_pair_abandon_selftest(int* status, long long limit_cycles, int meetings, cudaStream_t stream) {
  fwd::pair_abandon_selftest_kernel<<<1, 64, 0, stream>>>(status, limit_cycles, meetings);
  return cudaGetLastError() == cudaSuccess ? MXATTN_OK : MXATTN_ECUDA;
}

int launch_bounded_wait_selftest(int* status, long long limit_cycles, cudaStream_t stream) {
  fwd::bounded_wait_selftest_kernel<<<1, 32, 0, stream>>>(status, limit_cycles);
  return cudaGetLastError() == cudaSuccess ? MXATTN_OK : MXATTN_ECUDA;
}

size_t forward_profile_bytes(int B, int H, int64_t Nq, int64_t Nkv) {
  const int64_t qt = (Nq + kTile - 1) / kTile;
  return (size_t)((int64_t)B * H * ((qt + 1) / 2) * (fwd::kThreads / 32) * fwd::kProfSlots * 8);     // sized for one CTA per work item
}

size_t forward_dump_bytes(int B, int H, int64_t Nq, int64_t Nkv) {
  const int64_t qt = (Nq + kTile - 1) / kTile, kt = (Nkv + kTile - 1) / kTile;
  return (size_t)((int64_t)B * H * qt * kt * fwd::kDumpTileBytes + (int64_t)B * H * qt * kTile * 4);
}

int launch_forward(const void* q_codes, const void* q_scales, const void* k_codes, const void* k_scales,
                   const void* v_codes, const void* v_scales, void* o, int B, int H, int64_t Nq, int64_t Nkv,
                   float softmax_scale, unsigned flags, int* status, cudaStream_t stream, void* dump, bool profile) {
  using namespace fwd;
  Params p;
  p.q_codes = (const uint8_t*)q_codes; p.q_scales = (const uint8_t*)q_scales;
  p.k_codes = (const uint8_t*)k_codes; p.k_scales = (const uint8_t*)k_scales;
  p.v_codes = (const uint8_t*)v_codes; p.v_scales = (const uint8_t*)v_scales;
  p.out = o; p.status = status; p.dump = (uint8_t*)dump; p.Nq = Nq; p.Nkv = Nkv;
  const int64_t qt = (Nq + kTile - 1) / kTile, kt = (Nkv + kTile - 1) / kTile;
  const int64_t pairs = (qt + 1) / 2;
  const int64_t grid = (int64_t)B * H * pairs;
  if (qt > 0x3FFFFFFF || kt > 0x3FFFFFFF || grid > 0x7FFFFFFF) return MXATTN_EUNSUPPORTED;
  p.q_tiles = (int)qt; p.kv_tiles = (int)kt; p.q_pairs = (int)pairs; p.total_items = (int)grid;
  p.scale_log2e = softmax_scale * 1.4426950408889634f;
  p.softmax_scale = softmax_scale;

  const bool uos = flags & MXATTN_FLAG_UOS, pnq = flags & MXATTN_FLAG_PNQ, f32 = flags & MXATTN_FLAG_OUT_FP32;
  // Short key/value sequences with more work items than SMs: one CTA per SM walks the items, so that the set-up,
  // the first loads and the epilogue of one item overlap the tiles of its neighbours.  Long sequences keep one
  // item per CTA (the hardware's block scheduler then balances the tail better than a static assignment).
  static int n_sm = 0;
  if (n_sm == 0) {
    int dev = 0, v = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0)
      return MXATTN_ECUDA;
    n_sm = v;
  }
  const bool persist = (!dump || profile) && grid > n_sm && kt <= kPersistMaxTiles;
  // Descriptor of the bf16 output as a [B H][Nq][128] tensor with boxes of 32 rows x 64 columns (the epilogue's copies).
  CUtensorMap out_map;
  memset(&out_map, 0, sizeof(out_map));
  if (!f32) {
    static PFN_cuTensorMapEncodeTiled encode = nullptr;
    if (!encode) {
      void* fn = nullptr;
      cudaDriverEntryPointQueryResult qres;
      if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
          qres != cudaDriverEntryPointSuccess || !fn)
        return MXATTN_ECUDA;
      encode = reinterpret_cast<PFN_cuTensorMapEncodeTiled>(fn);
    }
    if (Nq > 0x7FFFFFFFLL || (uint64_t)Nq * kHeadDim * 2 >= (1ULL << 40)) return MXATTN_EUNSUPPORTED;
    const cuuint64_t dims[3] = {(cuuint64_t)kHeadDim, (cuuint64_t)Nq, (cuuint64_t)B * H};
    const cuuint64_t strides[2] = {(cuuint64_t)kHeadDim * 2, (cuuint64_t)Nq * kHeadDim * 2};     // bytes, dimensions 1 and 2
    const cuuint32_t box[3] = {(cuuint32_t)kCols, 32u, 1u};
    const cuuint32_t estr[3] = {1u, 1u, 1u};
    if (encode(&out_map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, o, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return MXATTN_ECUDA;
  }
  void (*kern)(const Params, const CUtensorMap) = nullptr;
#define PICK(U, P, F)                                                                     \
  if (uos == U && pnq == P && f32 == F)                                                   \
    kern = persist ? attention_kernel<U, P, F, false, true> : attention_kernel<U, P, F, false, false>;
  PICK(false, false, false) PICK(false, false, true) PICK(false, true, false) PICK(false, true, true)
  PICK(true, false, false) PICK(true, false, true) PICK(true, true, false) PICK(true, true, true)
#undef PICK
  if (profile) {                                  // cycle profile: the UOS + PNQ, bf16-output kernels with the counters compiled in
    if (!dump || !uos || !pnq || f32) return MXATTN_EINVAL;
    kern = persist ? attention_kernel<true, true, false, false, true, true> : attention_kernel<true, true, false, false, false, true>;
  } else if (dump) {                              // debug entry point: fp32 output only
    if (!f32) return MXATTN_EINVAL;
#define PICKD(U, P) if (uos == U && pnq == P) kern = attention_kernel<U, P, true, true, false>;
    PICKD(false, false) PICKD(false, true) PICKD(true, false) PICKD(true, true)
#undef PICKD
  }
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess)
    return MXATTN_ECUDA;
  kern<<<(unsigned)(persist ? n_sm : grid), kThreads, kSmemBytes, stream>>>(p, out_map);
  count_launch(1);
  return cudaGetLastError() == cudaSuccess ? MXATTN_OK : MXATTN_ECUDA;
}

}  // namespace mxattn
