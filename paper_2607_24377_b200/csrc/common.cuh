// Device helpers shared by the quantize and attention kernels (sm_100a only).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/mxattn.h"

namespace mxattn {

constexpr int kBlock = 32;       // elements per MXFP4 block (paper Section 2)
constexpr int kHeadDim = 128;    // supported head dimension
constexpr int kTile = 128;       // rows per operand tile and keys per KV tile (B_c)
constexpr int kTileCodeBytes = kTile * kHeadDim / 2;   // 8192
constexpr int kTileScaleBytes = kTile * kHeadDim / kBlock;  // 512

// Shared exponent e of a block whose maximum magnitude has fp32 bit pattern `u` (sign cleared).
// OCP: floor(log2 M) - 2 (paper Eq. 5).  UOS: ceil(log2(M / 7.25)) (paper Eq. 13, Algorithm 1).
// With M = mu * 2^E, mu in [1, 2): 7.25 = 1.8125 * 2^2, so the ceiling equals E - 2 when
// mu <= 1.8125 and E - 1 otherwise; in fp32 bits "mu > 1.8125" is "mantissa field > 0x680000".
// log2 is never evaluated.  M == 0 gives e = 0 (sigma = 1); e is clamped to [-127, 127]
// (subnormal M always clamps to -127; the upper clamp cannot be reached by a finite fp32).
__device__ __forceinline__ int shared_exponent(uint32_t u, bool uos) {
  if (u == 0u) return 0;
  const int eb = (int)(u >> 23);
  if (eb == 0) return -127;
  const int raise = (uos && (u & 0x7FFFFFu) > 0x680000u) ? 1 : 0;
  const int e = eb - 129 + raise;
  return e < -127 ? -127 : e;
}

// The ceiling family e = ceil(log2(M / q)) for an arbitrary boundary q > 0 (paper Eq. 7; TFS is q = 6,
// OAS at block 32 is q = 7, UOS is q = 7.25): with M = mu * 2^E and q = mu_q * 2^Eq,
// e = E - Eq + [mu > mu_q], decided on the bit patterns.  `q_bits` is the fp32 pattern of q.
__device__ __forceinline__ int shared_exponent_ceil(uint32_t u, uint32_t q_bits) {
  if (u == 0u) return 0;
  const int eb = (int)(u >> 23);
  if (eb == 0) return -127;
  const int e = eb - (int)(q_bits >> 23) + (((u & 0x7FFFFFu) > (q_bits & 0x7FFFFFu)) ? 1 : 0);
  return e < -127 ? -127 : (e > 127 ? 127 : e);
}

// Rule word used by the quantize kernels: 0 = OCP floor rule, otherwise the fp32 bit pattern of the
// ceiling-family boundary q (UOS: 7.25f).  For q = 7.25 this is exactly shared_exponent(u, true).
constexpr uint32_t kRuleOcp = 0u;
constexpr uint32_t kRuleUos = 0x40E80000u;   // 7.25f
__device__ __forceinline__ int shared_exponent_rule(uint32_t u, uint32_t rule) {
  return rule == kRuleOcp ? shared_exponent(u, false) : shared_exponent_ceil(u, rule);
}

// 2^-e as fp32 for e in [-127, 126] (exact, normal number).
__device__ __forceinline__ float pow2_neg(int e) {
  return __uint_as_float((uint32_t)(127 - e) << 23);
}

// Eight fp32 values -> eight E2M1 codes packed little-end first (x0 in bits 0-3).
// cvt.rn.satfinite rounds to nearest-even and saturates at +-6; its first source operand goes to
// the upper nibble.
__device__ __forceinline__ uint32_t pack_e2m1x8(float x0, float x1, float x2, float x3,
                                                float x4, float x5, float x6, float x7) {
  uint32_t out;
  asm("{\n\t"
      ".reg .b8 b0, b1, b2, b3;\n\t"
      "cvt.rn.satfinite.e2m1x2.f32 b0, %2, %1;\n\t"
      "cvt.rn.satfinite.e2m1x2.f32 b1, %4, %3;\n\t"
      "cvt.rn.satfinite.e2m1x2.f32 b2, %6, %5;\n\t"
      "cvt.rn.satfinite.e2m1x2.f32 b3, %8, %7;\n\t"
      "mov.b32 %0, {b0, b1, b2, b3};\n\t"
      "}"
      : "=r"(out)
      : "f"(x0), "f"(x1), "f"(x2), "f"(x3), "f"(x4), "f"(x5), "f"(x6), "f"(x7));
  return out;
}

__device__ __forceinline__ float bf16lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

// Byte offset of the 16-byte code chunk of block c (0..3) of row r (0..127) inside an 8 KiB
// operand tile: rows of 64 bytes, 16-byte chunks XOR-swizzled with bits 1-2 of the row
// (the tensor core's 64-byte swizzle mode for a K-major operand).
__device__ __host__ __forceinline__ int tile_code_offset(int r, int c) {
  return r * 64 + ((c ^ ((r >> 1) & 3)) << 4);
}
// Byte offset of the scale of (row r, block c) inside a 512-byte scale-factor atom.
__device__ __host__ __forceinline__ int tile_scale_offset(int r, int c) {
  return (r & 31) * 16 + (r >> 5) * 4 + c;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Internal launchers (defined in quantize.cu / forward.cu); all return an mxattn_status.
int launch_quantize(const void* in, void* codes, void* scales, int64_t batch, int64_t rows,
                    int64_t cols, int block_axis, int mode, int layout, cudaStream_t stream,
                    uint32_t rule_override = 0xFFFFFFFFu);
int launch_tensor_amax(const void* in, float* amax, int64_t batch, int64_t rows, int64_t cols, cudaStream_t stream);
int launch_quantize_nvfp4(const void* in, void* codes, void* scales, const float* amax, float* tensor_scale, int64_t batch,
                          int64_t rows, int64_t cols, int block_axis, int layout, cudaStream_t stream);
int launch_forward(const void* q_codes, const void* q_scales, const void* k_codes,
                   const void* k_scales, const void* v_codes, const void* v_scales, void* o,
                   int B, int H, int64_t Nq, int64_t Nkv, float softmax_scale, unsigned flags,
                   int* status, cudaStream_t stream, void* dump = nullptr, bool profile = false);
size_t forward_dump_bytes(int B, int H, int64_t Nq, int64_t Nkv);
size_t forward_profile_bytes(int B, int H, int64_t Nq, int64_t Nkv);
size_t bf16_workspace_bytes(int B, int H, int64_t Nq, int64_t Nkv);
int launch_forward_bf16(const void* q, const void* k, const void* v, void* o, int B, int H, int64_t Nq, int64_t Nkv,
                        float softmax_scale, unsigned flags, void* workspace, size_t workspace_bytes, cudaStream_t stream);
size_t nvfp4_workspace_bytes(int B, int H, int64_t Nq, int64_t Nkv);
int launch_forward_nvfp4(const void* q, const void* k, const void* v, void* o, int B, int H, int64_t Nq, int64_t Nkv,
                         float softmax_scale, unsigned flags, void* workspace, size_t workspace_bytes, cudaStream_t stream);
int launch_rowsum_diag(const void* q_codes, const void* q_scales, const void* k_codes, const void* k_scales,
                       void* out, int B, int H, int64_t Nq, int64_t Nkv, float softmax_scale, uint32_t rule,
                       int* status, cudaStream_t stream);
int launch_bounded_wait_selftest(int* status, long long limit_cycles, cudaStream_t stream);
int launch_pair_abandon_selftest(int* status, long long limit_cycles, int meetings, cudaStream_t stream);
void count_launch(int n);

}  // namespace mxattn
