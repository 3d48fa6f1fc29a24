/*
 * mxattn — MXFP4 attention forward with Universal Optimal Scaling (UOS) and Pre-Normalization
 * Quantization (PNQ) for NVIDIA B200 (sm_100a).  C ABI.
 *
 * Conventions for every entry point
 *   - Pointers are DEVICE pointers owned by the caller unless a parameter says "host".
 *     The library allocates no memory, never frees, and (except where stated) never
 *     synchronizes: work is enqueued on `stream` (a cudaStream_t passed as void*; NULL = the
 *     legacy default stream).
 *   - Every device pointer must be 16-byte aligned.
 *   - Return value: MXATTN_OK (0) or a negative mxattn_status.  On an argument error nothing
 *     is launched.  Inputs must be finite; NaN/Inf give unspecified values but never a hang.
 *   - bf16 tensors are contiguous, row-major, innermost dimension last.
 *
 * Number formats (paper, Section 2 "MXFP4 Block Quantization")
 *   - A block is 32 consecutive elements along the block axis that share one scale
 *     sigma = 2^e, stored as an E8M0 byte e + 127 (0xFF is never produced).
 *   - Elements are E2M1 codes: bit 3 = sign, bits 0-2 = index into {0, .5, 1, 1.5, 2, 3, 4, 6};
 *     round-to-nearest (ties to the even code), saturating at 6.  The sign of the input is kept
 *     even when the magnitude rounds to zero.
 *   - Codes are packed two per byte along the block axis: element 2k in bits 0-3 of byte k,
 *     element 2k+1 in bits 4-7.
 */
#ifndef MXATTN_H
#define MXATTN_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Shared-scale rule.
 * OCP: e = floor(log2 M) - 2 (paper Eq. 5, the floor rule; normalized block maximum in [4, 8)).
 * UOS: e = ceil(log2(M / 7.25)) (paper Eq. 13 with q* = 29/4, Theorem 1, Algorithm 1;
 *      normalized block maximum in (3.625, 7.25]).
 * M is the largest magnitude in the block; an all-zero block gets sigma = 1 (byte 127) and
 * all-zero codes; e is clamped to [-127, 127]. */
typedef enum { MXATTN_MODE_OCP = 0, MXATTN_MODE_UOS = 1 } mxattn_mode;
/* OR-able into `mode` of the quantizer: first apply the fixed orthogonal Hadamard rotation
 * y = x H_128 / sqrt(128) to every row (paper Algorithm 2, lines 1-2; Section 4.3), then quantize y.
 * H_128 is the Sylvester matrix, H[i][j] = (-1)^popcount(i & j).  There is no rounding to bf16 between the rotation
 * and the quantizer.  How this library evaluates it (not part of the paper's definition): x H_128 as a bf16 matrix
 * product on the tensor core -- the entries of H are +-1, so every product is exact and the sums are accumulated in
 * fp32 -- followed by one fp32 multiply by fl32(1/sqrt(128)).  Against the exact product rounded once to fp32 this
 * carries about 1e-7 of relative rounding noise, which can move a code or a scale byte only where a rotated value
 * sits that close to a rounding boundary (none in 1.6e7 values of the test recipes; the tests bound the rate by 1e-5).
 * Only block_axis 1 with cols == 128. */
enum { MXATTN_MODE_HADAMARD = 0x100 };

/* Flags of the forward pass.
 * UOS      : use the UOS rule for Q, K, V and the softmax tiles (else the OCP rule for all four).
 * PNQ      : the row sum l is accumulated from the QUANTIZED exponentials (paper Eq. 22,
 *            Algorithm 2 line 14); without it l is accumulated from the unquantized ones
 *            (the "direct" placement, paper Eq. 12).
 * OUT_FP32 : `o` is fp32 instead of bf16.
 * HADAMARD : see below. */
enum { MXATTN_FLAG_UOS = 1, MXATTN_FLAG_PNQ = 2, MXATTN_FLAG_OUT_FP32 = 4,
       /* rotate Q and K with the fixed Hadamard matrix before quantizing them (Algorithm 2 lines 1-2);
        * Q K^T is unchanged by the rotation in exact arithmetic, the quantization error is not */
       MXATTN_FLAG_HADAMARD = 8 };

typedef enum {
  MXATTN_OK = 0,
  MXATTN_EINVAL = -1,       /* null pointer, non-positive size, unknown mode / flag / layout */
  MXATTN_EUNSUPPORTED = -2, /* d != 128; cols % 32 != 0 on block_axis 1; tile layout with cols != 128 */
  MXATTN_EALIGN = -3,       /* a pointer is not 16-byte aligned */
  MXATTN_EWORKSPACE = -4,   /* workspace missing or too small */
  MXATTN_ECUDA = -5,        /* a CUDA runtime call or the launch failed (see cudaGetLastError) */
  MXATTN_ETIMEOUT = -6,     /* a bounded device-side wait expired (reported by mxattn_device_status) */
  MXATTN_ESCRATCH_TOO_SMALL = -7 /* mxattn_forward_static: the problem does not fit the built-in scratch array */
} mxattn_status;

/* Layout of the quantizer's outputs. */
enum {
  /* Canonical (for inspection / parity):
   *   block_axis 1: codes [rows, cols/2] bytes, scales [rows, cols/32] bytes.
   *   block_axis 0: outputs are TRANSPOSED so that they are contiguous along the block axis, and
   *                 the block axis is zero-extended to rows_pad = 128*ceil(rows/128):
   *                 codes [cols, rows_pad/2], scales [cols, rows_pad/32]; a block that is all
   *                 padding has zero codes and scale byte 127. */
  MXATTN_LAYOUT_CANONICAL = 0,
  /* Tile images consumed by the forward kernel (cols must be 128).  Rows are cut into tiles of
   * 128 (zero-extended); per matrix the outputs are
   *   codes  [ceil(rows/128)][8192]  and  scales [ceil(rows/128)][512].
   * Within a tile let (r, c) be (row in tile, block 0..3 along cols) for block_axis 1, and
   * (column, block of 32 rows 0..3) for block_axis 0; the 16 code bytes of that block sit at
   *   r*64 + ((c ^ ((r >> 1) & 3)) * 16)        (a 64-byte-swizzled, K-major operand tile)
   * and its scale byte at  (r % 32)*16 + (r / 32)*4 + c  (the tensor core's scale-factor atom). */
  MXATTN_LAYOUT_TILE = 1
};

/* Quantize one bf16 matrix in[rows, cols] to MXFP4 (paper Algorithm 1 for mode UOS; Eq. 5 for
 * mode OCP; element rounding Eq. 4), canonical layout.
 *   block_axis 1: blocks run along cols (Q and K: along the head dimension). cols % 32 == 0.
 *   block_axis 0: blocks run along rows (V: along the token axis), outputs transposed (see above).
 * codes / e8m0_scales: caller-allocated, sizes as given under MXATTN_LAYOUT_CANONICAL. */
int mxattn_quantize_mxfp4(const void* in, void* codes, void* e8m0_scales,
                          int64_t rows, int64_t cols, int block_axis, int mode, void* stream);

/* `batch` independent matrices in[batch][rows, cols] (one per attention head: blocks along the
 * token axis must not straddle heads), output layout selectable.  Output b starts at
 * b * (bytes of one matrix's output) in `codes` and `e8m0_scales`. */
int mxattn_quantize_mxfp4_batched(const void* in, void* codes, void* e8m0_scales, int64_t batch,
                                  int64_t rows, int64_t cols, int block_axis, int mode, int layout,
                                  void* stream);

/* The ceiling family with an arbitrary boundary: e = ceil(log2(M / qmax)) (paper Eq. 7), for the
 * scale-rule comparisons of the paper: qmax = 6 is Truncation-Free Scaling (Eq. 8), 7 is the OAS rule at
 * block size 32 (Appendix G), 7.25 is UOS, and a sweep over [6, 8] reproduces the setting of the
 * paper's Q_max study (Section 5.4.1).  4 <= qmax < 16.  Other arguments as
 * mxattn_quantize_mxfp4_batched. */
int mxattn_quantize_mxfp4_qmax(const void* in, void* codes, void* e8m0_scales, int64_t batch,
                               int64_t rows, int64_t cols, int block_axis, float qmax, int layout,
                               void* stream);

/* ---- NVFP4, the comparison format of the paper (named in its Introduction next to MXFP4; Section 5.2, baseline
 * "NVFP4": Q, K, V and the softmax tile in that format, nothing else changed) -----------------------------------
 * Elements are E2M1 codes as above; a block is 16 consecutive elements along the block axis with an E4M3 scale
 * (OCP 8-bit float, 4 exponent bits with bias 7, 3 mantissa bits, subnormals, no infinities, largest value 448 =
 * code 0x7E; never negative); each matrix of the batch has one fp32 tensor-level scale.  The paper only names the
 * format; the arithmetic is the usual two-level recipe, every step in IEEE fp32 in this order:
 *     g   = fl32(2688 / A)      A = tensor_amax[b], the largest magnitude of matrix b (A = 0: g = 1)
 *     s_T = fl32(1 / g)         -> tensor_scale[b]
 *     d   = E4M3( fl32(fl32(M * g) * fl32(1/6)) )   M = block maximum; round-to-nearest-even, saturating at 448
 *     code = sign | E2M1( fl32(|x| * fl32(g / d)) ) (all codes of the block zero when d = 0)
 * so that x is approximated by value(code) * d * s_T. */

/* Largest magnitude of each of `batch` bf16 matrices in[batch][rows, cols] -> amax[batch] (device fp32).
 * rows * cols must be a multiple of 8.  One read pass over the input. */
int mxattn_tensor_amax(const void* in, void* amax, int64_t batch, int64_t rows, int64_t cols, void* stream);

/* NVFP4 quantization of `batch` bf16 matrices with the tensor maxima `tensor_amax` (device fp32 [batch], e.g. from
 * mxattn_tensor_amax; a caller that wants one scale for the whole batch passes the same value in every entry).
 * tensor_scale: device fp32 [batch] that receives s_T, or NULL.
 * Layouts as for mxattn_quantize_mxfp4_batched with twice the scales:
 *   canonical  block_axis 1: codes [rows, cols/2], scales [rows, cols/16]          (cols % 16 == 0)
 *              block_axis 0: codes [cols, rows_pad/2], scales [cols, rows_pad/16]  (transposed; rows_pad = 128*ceil(rows/128);
 *                            padding blocks have code 0 and scale code 0)
 *   tile       (cols == 128) codes [ceil(rows/128)][8192] exactly as for MXFP4; scales [ceil(rows/128)][1024]: two
 *              scale-factor atoms of 512 bytes, atom a = blocks 4a..4a+3 (64 elements); inside an atom the byte of
 *              (row r, block c mod 4) sits at (r % 32)*16 + (r / 32)*4 + (c mod 4). */
int mxattn_quantize_nvfp4(const void* in, void* codes, void* e4m3_scales, const void* tensor_amax,
                          void* tensor_scale, int64_t batch, int64_t rows, int64_t cols, int block_axis,
                          int layout, void* stream);

/* Bytes of device scratch the forward pass needs for the quantized Q, K, V tile images, their
 * scales and a status word.  0 if the shape is unsupported. */
size_t mxattn_forward_workspace_bytes(int B, int H, int64_t Nq, int64_t Nkv, int d);

/* Register the scratch used by mxattn_forward.  Caller-owned device memory that must stay valid
 * until all enqueued forwards have finished.  Process-global: not thread-safe. */
int mxattn_set_workspace(void* dev_ptr, size_t bytes);

/* MXAttention forward (paper Algorithm 2: lines 3-19, preceded by the Hadamard rotation of Q and K of lines 1-2
 * when MXATTN_FLAG_HADAMARD is set).  q [B,H,Nq,d], k, v [B,H,Nkv,d] bf16; o [B,H,Nq,d] bf16 (fp32 with
 * MXATTN_FLAG_OUT_FP32).  d must be 128.  Non-causal, no mask.  softmax_scale > 0 multiplies the
 * quantized product Q-hat K-hat^T (line 9).  KV tiles are 128 keys, visited in ascending order.
 * Enqueues three quantize launches (Q, K along d; V along tokens) and one fused attention
 * launch.  Uses the workspace registered with mxattn_set_workspace. */
int mxattn_forward(const void* q, const void* k, const void* v, void* o,
                   int B, int H, int64_t Nq, int64_t Nkv, int d,
                   float softmax_scale, unsigned flags, void* stream);

/* Re-entrant form of mxattn_forward with an explicit workspace. */
int mxattn_forward_ws(const void* q, const void* k, const void* v, void* o,
                      int B, int H, int64_t Nq, int64_t Nkv, int d,
                      float softmax_scale, unsigned flags,
                      void* workspace, size_t workspace_bytes, void* stream);

/* The fused attention launch alone (Algorithm 2 lines 6-19) on operands already quantized in
 * MXATTN_LAYOUT_TILE by mxattn_quantize_mxfp4_batched with batch = B*H:
 * q_* from q (block_axis 1), k_* from k (block_axis 1), v_* from v (block_axis 0).
 * `status` points to 4 device ints (zeroed by the caller) that receive a non-zero code if a
 * bounded device-side wait expires. */
int mxattn_forward_prequantized(const void* q_codes, const void* q_scales,
                                const void* k_codes, const void* k_scales,
                                const void* v_codes, const void* v_scales, void* o,
                                int B, int H, int64_t Nq, int64_t Nkv, int d,
                                float softmax_scale, unsigned flags, void* status, void* stream);

/* Debugging aid for small problems: mxattn_forward_ws that also writes out what the softmax loop
 * produced, so that Algorithm 2 lines 10-14 can be checked tile by tile (the quantized probabilities
 * P-hat code for code, the running maxima and the final row sums) instead of only through O.
 * flags must contain MXATTN_FLAG_OUT_FP32.  `dump` is caller-owned device memory of at least
 * mxattn_forward_debug_dump_bytes() bytes (MXATTN_EWORKSPACE if smaller, MXATTN_EUNSUPPORTED above
 * 1 GiB), 16-byte aligned, laid out as
 *   [B*H][query tiles][KV tiles] records of 9216 bytes:
 *        8192 bytes  P-hat codes of the 128 x 128 tile, MXATTN_LAYOUT_TILE image (rows = queries,
 *                    blocks of 32 along the keys)
 *         512 bytes  its E8M0 scales, MXATTN_LAYOUT_TILE scale atom
 *         512 bytes  128 fp32: the running maximum m after this KV tile, per query row of the tile
 *   then [B*H][query tiles][128] fp32: the final row sum l (Algorithm 2 line 14) per query row.
 * Rows beyond Nq and columns beyond Nkv hold the values of the zero padding (code 0). */
size_t mxattn_forward_debug_dump_bytes(int B, int H, int64_t Nq, int64_t Nkv, int d);
int mxattn_forward_debug_dump(const void* q, const void* k, const void* v, void* o,
                              int B, int H, int64_t Nq, int64_t Nkv, int d,
                              float softmax_scale, unsigned flags,
                              void* workspace, size_t workspace_bytes,
                              void* dump, size_t dump_bytes, void* stream);

/* Performance-analysis aid: mxattn_forward_ws (flags exactly MXATTN_FLAG_UOS | MXATTN_FLAG_PNQ, bf16 output) through
 * an instantiation of the attention kernel that counts, per role, the SM cycles spent in each phase of the key-tile
 * loop of Algorithm 2 (the timed kernels are compiled without the counters; reading the cycle counter perturbs the
 * loop by a few percent).  `profile`: caller-owned device memory of mxattn_forward_cycle_profile_bytes() bytes,
 * zeroed by the caller, that receives [CTA][warp 0..17][16] int64.  One CTA per work item (two query tiles of one
 * head), or, for short key/value sequences with more work items than SMs, one CTA per SM (then only the first
 * #SMs records are written).
 *   warps 0-15 (softmax): [0] wait for the scores, [1] score load, [2] block and row maxima, [3] exchange with the
 *     partner warp, [4] wait for the previous output product, [5] block exponents, [6] exponentials + packing
 *     (+ rescaling), [7] hand-over of P-hat, [8] epilogue, [9] tiles processed;
 *   warp 16 (copy producer): [3] wait for a free K/V stage, [5] wait for a free Q buffer, [8] whole loop, [9] tiles;
 *   warp 17 (MMA issuer): [0] / [2] wait for P-hat of query tile 0 / 1, [5] wait for Q, [6] wait for K/V, [7] wait
 *     for the score buffer, [8] whole loop, [9] tiles. */
size_t mxattn_forward_cycle_profile_bytes(int B, int H, int64_t Nq, int64_t Nkv, int d);
int mxattn_forward_cycle_profile(const void* q, const void* k, const void* v, void* o,
                                 int B, int H, int64_t Nq, int64_t Nkv, int d,
                                 float softmax_scale, unsigned flags,
                                 void* workspace, size_t workspace_bytes,
                                 void* profile, size_t profile_bytes, void* stream);

/* Row-sum diagnostic of MXFP4 probability quantization (paper Section 5.3, figure "Row-sum
 * diagnostics", panels A, B, D).  Per query row: P = softmax(Q-hat K-hat^T * softmax_scale) as if
 * materialized (Q, K quantized as in mxattn_forward, same rule), rounded to fp32 and quantized in
 * 32-blocks along the keys; out receives six fp32 per row:
 *   [0] the row sum of the quantized probabilities (1 would be exact normalization),
 *   [1] the part of (row sum - 1) due to non-zero probabilities that quantize to zero,
 *   [2] ... due to saturation (scaled value above the largest E2M1 value 6),
 *   [3] ... due to downward rounding of the remaining elements,  [4] ... due to upward rounding,
 *   [5] the row's entropy -sum p ln p.
 * q: [B,H,Nq,d], k: [B,H,Nkv,d] bf16 device pointers; out: [B,H,Nq,6] fp32 device pointer; d = 128.
 * flags: MXATTN_FLAG_UOS (rule for Q, K and P; otherwise the OCP rule), MXATTN_FLAG_HADAMARD.
 * workspace: at least mxattn_forward_workspace_bytes(B,H,Nq,Nkv,d) bytes (holds Q-hat, K-hat and the
 * status word read by mxattn_device_status).  The scores are computed twice by the FP4 tensor-core
 * GEMM of the attention kernel; nothing of size Nq x Nkv is stored.  Same error codes as mxattn_forward_ws. */
int mxattn_rowsum_diagnostic(const void* q, const void* k, void* out,
                             int B, int H, int64_t Nq, int64_t Nkv, int d,
                             float softmax_scale, unsigned flags,
                             void* workspace, size_t workspace_bytes, void* stream);

/* bf16 variant of the same fused kernel, with no quantization anywhere: the FlashAttention-2
 * recurrence the paper starts from (Section 2, Eq. 2-3) with bf16 operands on the tensor cores, the
 * exponentials rounded to bf16 for the second GEMM and the row sum taken from the fp32 exponentials.
 * It is the high-precision reference point for the MXFP4 variants (the paper's "FP16" baseline,
 * Section 5.2).  Same tensor layouts as mxattn_forward; flags: only MXATTN_FLAG_OUT_FP32.
 * The workspace holds re-tiled copies of Q, K and V^T (mxattn_forward_bf16_workspace_bytes, about the
 * size of the inputs) and the status word at its start. */
size_t mxattn_forward_bf16_workspace_bytes(int B, int H, int64_t Nq, int64_t Nkv, int d);
int mxattn_forward_bf16(const void* q, const void* k, const void* v, void* o,
                        int B, int H, int64_t Nq, int64_t Nkv, int d,
                        float softmax_scale, unsigned flags,
                        void* workspace, size_t workspace_bytes, void* stream);

/* The paper's comparison baseline "NVFP4" (Section 5.2): the same fused forward pass with Q, K, V and the softmax tile
 * quantized to NVFP4 (see mxattn_quantize_nvfp4) instead of MXFP4, nothing else changed -- same tiling (KV tiles of
 * 128 keys in ascending order), same recurrence.  Tensor-level scales: one per head for each of Q, K and V (the
 * largest magnitude of that head's matrix); for the softmax tile the constant 1/2688, because its largest value is
 * known to be 1 (readings: the paper does not say how the baseline chooses them).
 * flags: MXATTN_FLAG_PNQ (row sum from the quantized probabilities, as in MXAttention; without it the direct
 * placement, which is what the paper's baseline uses) and MXATTN_FLAG_OUT_FP32.  Same tensor layouts as
 * mxattn_forward.  Enqueues three tensor-maximum launches, three quantize launches and the attention launch.
 * The workspace (mxattn_forward_nvfp4_workspace_bytes) holds the quantized operands and, at its start, the status word. */
size_t mxattn_forward_nvfp4_workspace_bytes(int B, int H, int64_t Nq, int64_t Nkv, int d);
int mxattn_forward_nvfp4(const void* q, const void* k, const void* v, void* o,
                         int B, int H, int64_t Nq, int64_t Nkv, int d,
                         float softmax_scale, unsigned flags,
                         void* workspace, size_t workspace_bytes, void* stream);

/* Bytes of device memory mxattn_forward_host needs (inputs, output and workspace). */
size_t mxattn_forward_host_arena_bytes(int B, int H, int64_t Nq, int64_t Nkv, int d, unsigned flags);

/* End-to-end form for callers whose tensors live in HOST memory (pinned memory, so that the copies
 * are asynchronous): runs mxattn_forward_ws in stages of one or more heads (one head first, then as many
 * per stage as it takes to fill the GPU's SMs) out of `device_arena` and writes o into o_host.  The stages
 * are pipelined over the caller's `stream` and four helper streams that the library creates once per
 * device: host->device copies of the next stages, their quantization, and the device->host copy of the
 * previous stage overlap the attention kernels, whose launches alternate between `stream` and a helper
 * stream so that one stage's CTAs start as the previous stage's finish.  Work already queued on `stream`
 * is waited for first;
 * the call returns after everything has finished (it SYNCHRONIZES).  `device_arena` is caller-owned
 * device memory of at least mxattn_forward_host_arena_bytes(); no device memory is allocated.
 * Returns MXATTN_ETIMEOUT if a bounded device-side wait expired in any head. */
int mxattn_forward_host(const void* q_host, const void* k_host, const void* v_host, void* o_host,
                        int B, int H, int64_t Nq, int64_t Nkv, int d,
                        float softmax_scale, unsigned flags,
                        void* device_arena, size_t arena_bytes, void* stream);

/* Size of the scratch array built into the library for mxattn_forward_static (32 MiB). */
#define MXATTN_STATIC_SCRATCH_BYTES (32u << 20)

/* mxattn_forward for callers that cannot allocate device memory.  (The paper has no counterpart
 * to this entry point; it exists for deployment reasons only.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside a host framework whose
 * device memory is fully pre-planned, in a plugin that must not allocate after start-up, or in a
 * latency-critical loop that cannot afford an allocator call.  Such a caller can hand over q, k, v
 * and o (it owns those anyway) but has nowhere to get the forward pass's scratch from, and cannot
 * call mxattn_set_workspace / mxattn_forward_ws without memory of its own.
 *
 * Same arguments, layouts and result as mxattn_forward.  The scratch (the quantized tile images
 * of Q, K and V, their scales and the status word) is a fixed array of MXATTN_STATIC_SCRATCH_BYTES
 * in device global memory that is part of the library image: every GPU that loads the library
 * holds it until the process exits.  The call makes no cudaMalloc / cudaFree and uses no
 * allocating library routine.
 *
 * Limits and rules:
 *   - mxattn_forward_workspace_bytes(B, H, Nq, Nkv, d) must not exceed
 *     MXATTN_STATIC_SCRATCH_BYTES, otherwise MXATTN_ESCRATCH_TOO_SMALL is returned and nothing is
 *     launched (for example B*H = 8 heads of Nq = Nkv = 8192 fit; the Wan2.2-sized problem does not).
 *   - The first call on each device looks up the array's device address (with that device
 *     current) and caches it; make that first call outside any stream capture.
 *   - All calls on a device share the one array, and it keeps what the previous call left there.
 *     Everything the pass relies on being zero (the status word; padding inside the tile images)
 *     is rewritten by each call.  Two calls whose work overlaps on the GPU (different streams, or
 *     different host threads) race on the array: serialize them.
 *   - The status word is the first int of the array; a bounded device-side wait that expires is
 *     not reported by this entry point itself -- results are then unspecified, as for
 *     mxattn_forward. */
int mxattn_forward_static(const void* q, const void* k, const void* v, void* o,
                          int B, int H, int64_t Nq, int64_t Nkv, int d,
                          float softmax_scale, unsigned flags, void* stream);

/* Dense block-scaled FP4 GEMM, the measuring stick for the attention kernel's two GEMMs (paper Section 1 names the two
 * matrix products as the dominant operations of the forward pass; Algorithm 2, the score and the output products):
 *     C[M, N] = A[M, K] B[N, K]^T      MXFP4 operands, fp32 accumulation, C row-major fp32 (out_fp32 != 0) or bf16.
 * Operands are MXATTN_LAYOUT_TILE images ordered [K/128][rows/128]: tile (kb, t) holds rows 128 t .. 128 t + 127 and
 * the K elements 128 kb .. 128 kb + 127 -- what mxattn_quantize_mxfp4_batched(batch = K/128, rows, cols = 128,
 * block_axis 1, MXATTN_LAYOUT_TILE) writes for an input arranged as [K/128][rows][128].
 * tile_n: columns of C per CTA, 256 or 128 (the N of the multiply instruction; a CTA always takes 128 rows).
 * M % 128 == 0, N % tile_n == 0, K % 128 == 0, each at most 16384.
 * resident == 0: k_steps must equal K/128; an ordinary GEMM whose operand tiles stream through shared memory.
 * resident != 0: the first min(k_steps, 6) K blocks are loaded once and the k_steps (up to 2^20; beyond 6 a multiple of
 *   6, with K >= 768) multiply steps cycle over them, so C = sum over steps i of A_(i mod 6) B_(i mod 6)^T: after the
 *   first round the issuing thread executes multiply instructions only -- no global-memory traffic, no scale copies,
 *   no barriers --, which measures the rate of the FP4 tensor pipe itself.
 * flops = 2 M N 128 k_steps.  `status`: 4 device ints, zeroed by the caller, non-zero if a bounded wait expired. */
int mxattn_probe_fp4_gemm(const void* a_codes, const void* a_scales, const void* b_codes, const void* b_scales,
                          void* c, int64_t M, int64_t N, int64_t K, int64_t k_steps, int resident, int out_fp32,
                          int tile_n, void* status, void* stream);

/* Synchronizes `stream`, then copies to *host_out (host pointer) the status word of the rotating quantizer, the one
 * quantize kernel with a device-side wait (for its tensor-core product): 0 = no bounded wait of it ever expired in
 * this process on the current device. */
int mxattn_quantizer_status(int* host_out, void* stream);

/* Synchronizes `stream`, then copies the workspace's status word to *host_out (host pointer):
 * 0 = no bounded wait expired since the workspace was last used by a forward. */
int mxattn_device_status(const void* workspace, int* host_out, void* stream);

/* Exercises the failure path of the device-side waits without disturbing the GPU: a one-warp kernel
 * waits on a barrier that nothing arrives on, gives up after `limit_cycles` SM cycles (at most 2e9) and
 * writes the code 77 into status[0] (4 device ints, zeroed by the caller).  The kernel ends normally
 * and the context stays usable.  Every wait inside the attention kernels uses the same routine with a
 * limit of about two seconds. */
int mxattn_selftest_bounded_wait(void* status, int64_t limit_cycles, void* stream);

/* Exercises, again without disturbing the GPU, the way the attention kernel's paired softmax warps stay in step when
 * one of them gives up: two warps meet at a named barrier in every key tile (each holds half of a query row's scores;
 * the row maximum of Algorithm 2 needs both halves).  Here warp 0's wait runs out after `limit_cycles` (code 77 in
 * status[0]); from then on it only keeps the pair's remaining appointments, as the attention kernel's warps do.
 * Warp 1, whose waits all succeed, works through `meetings` (1 .. 100000) of them and records how many it completed
 * in status[1] -- `meetings` if no warp was left stranded.  `status`: 4 device ints, zeroed by the caller. */
int mxattn_selftest_pair_abandon(void* status, int64_t limit_cycles, int meetings, void* stream);

/* Number of kernel launches the last forward call of this process enqueued (for accounting). */
int mxattn_last_launch_count(void);

const char* mxattn_strerror(int status);

#ifdef __cplusplus
}
#endif
#endif /* MXATTN_H */
