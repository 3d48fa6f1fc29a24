// C-ABI entry points that orchestrate the kernels: workspace carving, the three quantize
// launches plus the fused attention launch (paper Algorithm 2, lines 3-19), and the host-buffer
// end-to-end form.
#include <vector>

#include "common.cuh"
#include <nvtx3/nvToolsExt.h>      // header-only: the ranges cost nothing unless a profiling tool is attached

namespace mxattn {

// NVTX range for the lifetime of the object: the host-side enqueue of a launch or of a pipeline stage, so that a
// timeline shows which call and which stage queued which kernels.
struct TraceRange {
  explicit TraceRange(const char* name) { nvtxRangePushA(name); }
  ~TraceRange() { nvtxRangePop(); }
  TraceRange(const TraceRange&) = delete;
  TraceRange& operator=(const TraceRange&) = delete;
};

static int g_launches = 0;
static void* g_workspace = nullptr;
static size_t g_workspace_bytes = 0;

void count_launch(int n) { g_launches += n; }

struct WorkspaceLayout {
  size_t q_codes, q_scales, k_codes, k_scales, v_codes, v_scales, status, total;
};

static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

static bool carve(int B, int H, int64_t Nq, int64_t Nkv, int d, WorkspaceLayout* w) {
  if (B <= 0 || H <= 0 || Nq <= 0 || Nkv <= 0 || d != kHeadDim) return false;
  const size_t bh = (size_t)B * H;
  const size_t qt = (size_t)((Nq + kTile - 1) / kTile), kt = (size_t)((Nkv + kTile - 1) / kTile);
  size_t off = 0;
  w->status = off;   off += 256;
  w->q_codes = off;  off += align_up(bh * qt * kTileCodeBytes, 256);
  w->q_scales = off; off += align_up(bh * qt * kTileScaleBytes, 256);
  w->k_codes = off;  off += align_up(bh * kt * kTileCodeBytes, 256);
  w->k_scales = off; off += align_up(bh * kt * kTileScaleBytes, 256);
  w->v_codes = off;  off += align_up(bh * kt * kTileCodeBytes, 256);
  w->v_scales = off; off += align_up(bh * kt * kTileScaleBytes, 256);
  w->total = off;
  return true;
}

// `qstream` / `qdone`: if given, the three quantize launches go to `qstream`, `qdone` is recorded behind them and
// the attention launch on `stream` waits for it (the host pipeline uses this to quantize the next stage's
// operands while the current stage's attention kernel drains).
static int forward_ws(const void* q, const void* k, const void* v, void* o, int B, int H, int64_t Nq,
                      int64_t Nkv, int d, float softmax_scale, unsigned flags, void* workspace,
                      size_t workspace_bytes, cudaStream_t stream, void* dump = nullptr,
                      cudaStream_t qstream = nullptr, cudaEvent_t qdone = nullptr, bool profile = false) {
  if (!q || !k || !v || !o) return MXATTN_EINVAL;
  if (B <= 0 || H <= 0 || Nq <= 0 || Nkv <= 0) return MXATTN_EINVAL;
  if (flags & ~(unsigned)(MXATTN_FLAG_UOS | MXATTN_FLAG_PNQ | MXATTN_FLAG_OUT_FP32 | MXATTN_FLAG_HADAMARD)) return MXATTN_EINVAL;
  if (!(softmax_scale > 0.0f) || !(softmax_scale < 3.0e38f)) return MXATTN_EINVAL;
  if (d != kHeadDim) return MXATTN_EUNSUPPORTED;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o)) return MXATTN_EALIGN;
  WorkspaceLayout w;
  if (!carve(B, H, Nq, Nkv, d, &w)) return MXATTN_EUNSUPPORTED;
  if (!workspace || workspace_bytes < w.total) return MXATTN_EWORKSPACE;
  if (!aligned16(workspace)) return MXATTN_EALIGN;
  g_launches = 0;
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  const int mode = (flags & MXATTN_FLAG_UOS) ? MXATTN_MODE_UOS : MXATTN_MODE_OCP;
  const int qk_mode = mode | ((flags & MXATTN_FLAG_HADAMARD) ? MXATTN_MODE_HADAMARD : 0);   // Algorithm 2 lines 1-2
  const int64_t bh = (int64_t)B * H;
  cudaStream_t qs = qstream ? qstream : stream;
  if (cudaMemsetAsync(ws + w.status, 0, 16, qs) != cudaSuccess) return MXATTN_ECUDA;
  int rc;
  // Algorithm 2 lines 3-5: Q-hat, K-hat (blocks along d), V-hat (blocks along tokens)
  {
    TraceRange tr("mxattn quantize Q K V");
    if ((rc = launch_quantize(q, ws + w.q_codes, ws + w.q_scales, bh, Nq, d, 1, qk_mode, MXATTN_LAYOUT_TILE, qs))) return rc;
    if ((rc = launch_quantize(k, ws + w.k_codes, ws + w.k_scales, bh, Nkv, d, 1, qk_mode, MXATTN_LAYOUT_TILE, qs))) return rc;
    if ((rc = launch_quantize(v, ws + w.v_codes, ws + w.v_scales, bh, Nkv, d, 0, mode, MXATTN_LAYOUT_TILE, qs))) return rc;
  }
  if (qstream) {
    if (cudaEventRecord(qdone, qstream) != cudaSuccess || cudaStreamWaitEvent(stream, qdone, 0) != cudaSuccess) return MXATTN_ECUDA;
  }
  // lines 6-19
  TraceRange tr("mxattn attention");
  return launch_forward(ws + w.q_codes, ws + w.q_scales, ws + w.k_codes, ws + w.k_scales, ws + w.v_codes,
                        ws + w.v_scales, o, B, H, Nq, Nkv, softmax_scale, flags,
                        reinterpret_cast<int*>(ws + w.status), stream, dump, profile);
}

}  // namespace mxattn

using namespace mxattn;

extern "C" size_t mxattn_forward_workspace_bytes(int B, int H, int64_t Nq, int64_t Nkv, int d) {
  WorkspaceLayout w;
  return carve(B, H, Nq, Nkv, d, &w) ? w.total : 0;
}

extern "C" int mxattn_set_workspace(void* dev_ptr, size_t bytes) {
  if (dev_ptr && !aligned16(dev_ptr)) return MXATTN_EALIGN;
  g_workspace = dev_ptr;
  g_workspace_bytes = dev_ptr ? bytes : 0;
  return MXATTN_OK;
}

extern "C" int mxattn_forward(const void* q, const void* k, const void* v, void* o, int B, int H,
                              int64_t Nq, int64_t Nkv, int d, float softmax_scale, unsigned flags,
                              void* stream) {
  return forward_ws(q, k, v, o, B, H, Nq, Nkv, d, softmax_scale, flags, g_workspace, g_workspace_bytes,
                    (cudaStream_t)stream);
}

extern "C" int mxattn_forward_ws(const void* q, const void* k, const void* v, void* o, int B, int H,
                                 int64_t Nq, int64_t Nkv, int d, float softmax_scale, unsigned flags,
                                 void* workspace, size_t workspace_bytes, void* stream) {
  return forward_ws(q, k, v, o, B, H, Nq, Nkv, d, softmax_scale, flags, workspace, workspace_bytes,
                    (cudaStream_t)stream);
}

extern "C" int mxattn_rowsum_diagnostic(const void* q, const void* k, void* out, int B, int H, int64_t Nq,
                                        int64_t Nkv, int d, float softmax_scale, unsigned flags,
                                        void* workspace, size_t workspace_bytes, void* stream_) {
  cudaStream_t stream = (cudaStream_t)stream_;
  if (!q || !k || !out) return MXATTN_EINVAL;
  if (B <= 0 || H <= 0 || Nq <= 0 || Nkv <= 0) return MXATTN_EINVAL;
  if (flags & ~(unsigned)(MXATTN_FLAG_UOS | MXATTN_FLAG_HADAMARD)) return MXATTN_EINVAL;
  if (!(softmax_scale > 0.0f) || !(softmax_scale < 3.0e38f)) return MXATTN_EINVAL;
  if (d != kHeadDim) return MXATTN_EUNSUPPORTED;
  if (!aligned16(q) || !aligned16(k) || !aligned16(out)) return MXATTN_EALIGN;
  WorkspaceLayout w;
  if (!carve(B, H, Nq, Nkv, d, &w)) return MXATTN_EUNSUPPORTED;
  if (!workspace || workspace_bytes < w.total) return MXATTN_EWORKSPACE;
  if (!aligned16(workspace)) return MXATTN_EALIGN;
  g_launches = 0;
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  const int mode = (flags & MXATTN_FLAG_UOS) ? MXATTN_MODE_UOS : MXATTN_MODE_OCP;
  const int qk_mode = mode | ((flags & MXATTN_FLAG_HADAMARD) ? MXATTN_MODE_HADAMARD : 0);
  const int64_t bh = (int64_t)B * H;
  if (cudaMemsetAsync(ws + w.status, 0, 16, stream) != cudaSuccess) return MXATTN_ECUDA;
  int rc;
  if ((rc = launch_quantize(q, ws + w.q_codes, ws + w.q_scales, bh, Nq, d, 1, qk_mode, MXATTN_LAYOUT_TILE, stream))) return rc;
  if ((rc = launch_quantize(k, ws + w.k_codes, ws + w.k_scales, bh, Nkv, d, 1, qk_mode, MXATTN_LAYOUT_TILE, stream))) return rc;
  return launch_rowsum_diag(ws + w.q_codes, ws + w.q_scales, ws + w.k_codes, ws + w.k_scales, out, B, H, Nq, Nkv,
                            softmax_scale, (flags & MXATTN_FLAG_UOS) ? kRuleUos : kRuleOcp,
                            reinterpret_cast<int*>(ws + w.status), stream);
}

extern "C" size_t mxattn_forward_debug_dump_bytes(int B, int H, int64_t Nq, int64_t Nkv, int d) {
  if (B <= 0 || H <= 0 || Nq <= 0 || Nkv <= 0 || d != kHeadDim) return 0;
  return forward_dump_bytes(B, H, Nq, Nkv);
}

extern "C" int mxattn_forward_debug_dump(const void* q, const void* k, const void* v, void* o, int B, int H,
                                         int64_t Nq, int64_t Nkv, int d, float softmax_scale, unsigned flags,
                                         void* workspace, size_t workspace_bytes, void* dump,
                                         size_t dump_bytes, void* stream) {
  if (!dump) return MXATTN_EINVAL;
  if (!(flags & MXATTN_FLAG_OUT_FP32)) return MXATTN_EINVAL;
  if (B <= 0 || H <= 0 || Nq <= 0 || Nkv <= 0) return MXATTN_EINVAL;
  if (d != kHeadDim) return MXATTN_EUNSUPPORTED;
  const size_t need = forward_dump_bytes(B, H, Nq, Nkv);
  if (need > ((size_t)1 << 30)) return MXATTN_EUNSUPPORTED;      // a debugging aid for small problems
  if (dump_bytes < need) return MXATTN_EWORKSPACE;
  if (!aligned16(dump)) return MXATTN_EALIGN;
  return forward_ws(q, k, v, o, B, H, Nq, Nkv, d, softmax_scale, flags, workspace, workspace_bytes,
                    (cudaStream_t)stream, dump);
}

extern "C" size_t mxattn_forward_cycle_profile_bytes(int B, int H, int64_t Nq, int64_t Nkv, int d) {
  if (B <= 0 || H <= 0 || Nq <= 0 || Nkv <= 0 || d != kHeadDim) return 0;
  return forward_profile_bytes(B, H, Nq, Nkv);
}

extern "C" int mxattn_forward_cycle_profile(const void* q, const void* k, const void* v, void* o, int B, int H,
                                            int64_t Nq, int64_t Nkv, int d, float softmax_scale, unsigned flags,
                                            void* workspace, size_t workspace_bytes, void* profile,
                                            size_t profile_bytes, void* stream) {
  if (!profile) return MXATTN_EINVAL;
  if (flags != (unsigned)(MXATTN_FLAG_UOS | MXATTN_FLAG_PNQ)) return MXATTN_EINVAL;
  if (B <= 0 || H <= 0 || Nq <= 0 || Nkv <= 0) return MXATTN_EINVAL;
  if (d != kHeadDim) return MXATTN_EUNSUPPORTED;
  if (profile_bytes < forward_profile_bytes(B, H, Nq, Nkv)) return MXATTN_EWORKSPACE;
  if (!aligned16(profile)) return MXATTN_EALIGN;
  return forward_ws(q, k, v, o, B, H, Nq, Nkv, d, softmax_scale, flags, workspace, workspace_bytes,
                    (cudaStream_t)stream, profile, nullptr, nullptr, true);
}

extern "C" int mxattn_forward_prequantized(const void* q_codes, const void* q_scales, const void* k_codes,
                                           const void* k_scales, const void* v_codes, const void* v_scales,
                                           void* o, int B, int H, int64_t Nq, int64_t Nkv, int d,
                                           float softmax_scale, unsigned flags, void* status, void* stream) {
  if (!q_codes || !q_scales || !k_codes || !k_scales || !v_codes || !v_scales || !o || !status) return MXATTN_EINVAL;
  if (B <= 0 || H <= 0 || Nq <= 0 || Nkv <= 0) return MXATTN_EINVAL;
  if (flags & ~(unsigned)(MXATTN_FLAG_UOS | MXATTN_FLAG_PNQ | MXATTN_FLAG_OUT_FP32 | MXATTN_FLAG_HADAMARD)) return MXATTN_EINVAL;
  if (!(softmax_scale > 0.0f) || !(softmax_scale < 3.0e38f)) return MXATTN_EINVAL;
  if (d != kHeadDim) return MXATTN_EUNSUPPORTED;
  if (!aligned16(q_codes) || !aligned16(q_scales) || !aligned16(k_codes) || !aligned16(k_scales) ||
      !aligned16(v_codes) || !aligned16(v_scales) || !aligned16(o) || !aligned16(status))
    return MXATTN_EALIGN;
  g_launches = 0;
  return launch_forward(q_codes, q_scales, k_codes, k_scales, v_codes, v_scales, o, B, H, Nq, Nkv,
                        softmax_scale, flags, static_cast<int*>(status), (cudaStream_t)stream);
}

// ---------------------------------------------------------------------------------------------
// Host-buffer form.  Heads are independent, so the call is pipelined in stages of one or more heads over five
// streams -- the caller's and four helper streams (copies in, quantization, a second attention stream, copies out):
// host->device copies of the next stage and the device->host copy of the previous one overlap the kernels of the
// current stage (PCIe is full duplex).  The helper streams and the events are created on first use, once per
// device, and kept for the life of the process; no device memory is allocated.
struct HostPipe {
  cudaStream_t in = nullptr, quant = nullptr, out = nullptr, attn = nullptr;
  std::vector<cudaEvent_t> ev;
};
static HostPipe g_pipe[64];

static HostPipe* host_pipe(size_t n_events) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  HostPipe& hp = g_pipe[dev];
  if (!hp.in && cudaStreamCreateWithFlags(&hp.in, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
  if (!hp.out && cudaStreamCreateWithFlags(&hp.out, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
  if (!hp.quant) {
    // the quantize launches are short and feed the next attention launch: they go first when SMs free up
    int lo = 0, hi = 0;
    if (cudaDeviceGetStreamPriorityRange(&lo, &hi) != cudaSuccess) return nullptr;
    if (cudaStreamCreateWithPriority(&hp.quant, cudaStreamNonBlocking, hi) != cudaSuccess) return nullptr;
  }
  if (!hp.attn && cudaStreamCreateWithFlags(&hp.attn, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
  while (hp.ev.size() < n_events) {
    cudaEvent_t e;
    if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) return nullptr;
    hp.ev.push_back(e);
  }
  return &hp;
}

// How many heads a pipeline stage of mxattn_forward_host takes (after the first stage, which takes one).  A stage
// is one attention launch of g * ceil(ceil(Nq/128)/2) CTAs.  Consecutive stages' launches go to two streams, so
// the CTAs of the next stage start on the SMs the current one leaves and a partly filled last wave costs
// nothing; what is left to weigh is a launch that cannot fill the device at all (small heads: take several),
// the fixed cost per stage, and the last stage's copy out, which nothing hides.  The estimate (attention at
// ~1.8 PFLOP/s, copies at ~50 GB/s, 20 us of launches and events per stage) only has to rank the candidates.
static int heads_per_stage(size_t bh, int64_t Nq, int64_t Nkv, size_t out_bytes_per_head) {
  int dev = 0, n_sm = 148;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
  if (n_sm <= 0) n_sm = 148;
  const double ctas = (double)(((Nq + kTile - 1) / kTile + 1) / 2);
  const double t_head = 4.0 * (double)Nq * (double)Nkv * kHeadDim / 1.8e15;
  const double t_out = (double)out_bytes_per_head / 50e9;
  int best = 1;
  double best_t = 1e300;
  for (int g = 1; g <= 8 && (size_t)g <= bh; ++g) {
    if (g > 1 && bh / g < 3) break;                 // keep at least three stages to overlap
    const double fill = g * ctas / n_sm;
    const double eff = fill < 1.0 ? fill : 1.0;
    const double t = (double)bh * t_head / eff + g * t_out + 20e-6 * (double)((bh + g - 1) / g);
    if (t < best_t * 0.995) { best_t = t; best = g; }
  }
  return best;
}

extern "C" size_t mxattn_forward_host_arena_bytes(int B, int H, int64_t Nq, int64_t Nkv, int d, unsigned flags) {
  WorkspaceLayout w;
  if (!carve(1, 1, Nq, Nkv, d, &w) || B <= 0 || H <= 0) return 0;     // one workspace slice per head
  const size_t bh = (size_t)B * H;
  const size_t qb = align_up(bh * (size_t)Nq * d * 2, 256), kb = align_up(bh * (size_t)Nkv * d * 2, 256);
  const size_t ob = align_up(bh * (size_t)Nq * d * ((flags & MXATTN_FLAG_OUT_FP32) ? 4 : 2), 256);
  return qb + 2 * kb + ob + bh * w.total;
}

extern "C" int mxattn_forward_host(const void* q_host, const void* k_host, const void* v_host, void* o_host,
                                   int B, int H, int64_t Nq, int64_t Nkv, int d, float softmax_scale,
                                   unsigned flags, void* device_arena, size_t arena_bytes, void* stream_) {
  if (!q_host || !k_host || !v_host || !o_host) return MXATTN_EINVAL;
  const size_t need = mxattn_forward_host_arena_bytes(B, H, Nq, Nkv, d, flags);
  if (need == 0) return (d != kHeadDim) ? MXATTN_EUNSUPPORTED : MXATTN_EINVAL;
  if (!device_arena || arena_bytes < need) return MXATTN_EWORKSPACE;
  if (!aligned16(device_arena)) return MXATTN_EALIGN;
  cudaStream_t stream = (cudaStream_t)stream_;
  const size_t bh = (size_t)B * H;
  const size_t osz = (flags & MXATTN_FLAG_OUT_FP32) ? 4 : 2;
  const size_t qh = (size_t)Nq * d * 2, kh = (size_t)Nkv * d * 2, oh = (size_t)Nq * d * osz;   // bytes per head
  WorkspaceLayout w;
  carve(1, 1, Nq, Nkv, d, &w);
  uint8_t* a = static_cast<uint8_t*>(device_arena);
  uint8_t* dq = a;
  uint8_t* dk = dq + align_up(bh * qh, 256);
  uint8_t* dv = dk + align_up(bh * kh, 256);
  uint8_t* dout = dv + align_up(bh * kh, 256);
  uint8_t* ws = dout + align_up(bh * oh, 256);
  // The first stage takes one head (nothing hides its copy in), the others g heads each.
  const int g = heads_per_stage(bh, Nq, Nkv, oh);
  const size_t stages = (g == 1) ? bh : 1 + (bh - 1 + g - 1) / g;
  auto first_head = [&](size_t st) {
    if (g == 1 || st == 0) return st;
    const size_t h = 1 + (st - 1) * (size_t)g;
    return h < bh ? h : bh;
  };
  HostPipe* hp = host_pipe(3 * stages + 2);
  if (!hp) return MXATTN_ECUDA;
  cudaEvent_t* ev = hp->ev.data();
  bool fail = false;
  auto ck = [&](cudaError_t e) { if (e != cudaSuccess) fail = true; };
  ck(cudaEventRecord(ev[3 * stages], stream));                   // work already queued on the caller's stream comes first
  ck(cudaStreamWaitEvent(hp->in, ev[3 * stages], 0));
  ck(cudaStreamWaitEvent(hp->attn, ev[3 * stages], 0));
  int rc = MXATTN_OK;
  for (size_t st = 0; st < stages && !fail && rc == MXATTN_OK; ++st) {
    TraceRange tr("mxattn host stage");
    const size_t i = first_head(st), n = first_head(st + 1) - i;  // heads of the stage; heads are contiguous in memory
    // attention launches alternate between the caller's stream and one of the pipeline's, so that the CTAs of a
    // stage start on the SMs the previous stage's last CTAs leave (no tail, no launch gap between stages)
    cudaStream_t as = (st & 1) ? hp->attn : stream;
    ck(cudaMemcpyAsync(dq + i * qh, static_cast<const char*>(q_host) + i * qh, n * qh, cudaMemcpyHostToDevice, hp->in));
    ck(cudaMemcpyAsync(dk + i * kh, static_cast<const char*>(k_host) + i * kh, n * kh, cudaMemcpyHostToDevice, hp->in));
    ck(cudaMemcpyAsync(dv + i * kh, static_cast<const char*>(v_host) + i * kh, n * kh, cudaMemcpyHostToDevice, hp->in));
    ck(cudaEventRecord(ev[3 * st], hp->in));
    ck(cudaStreamWaitEvent(hp->quant, ev[3 * st], 0));
    // the stage's workspace starts at its first head's slice (n slices are at least as large as one workspace for
    // n heads); its operands are quantized on a stream of their own, behind the copies and ahead of the attention
    // launch, so that they fill the SMs the previous stage's attention kernel frees as it drains
    rc = forward_ws(dq + i * qh, dk + i * kh, dv + i * kh, dout + i * oh, 1, (int)n, Nq, Nkv, d, softmax_scale, flags,
                    ws + i * w.total, n * w.total, as, nullptr, hp->quant, ev[3 * st + 1]);
    ck(cudaEventRecord(ev[3 * st + 2], as));
    ck(cudaStreamWaitEvent(hp->out, ev[3 * st + 2], 0));
    ck(cudaMemcpyAsync(static_cast<char*>(o_host) + i * oh, dout + i * oh, n * oh, cudaMemcpyDeviceToHost, hp->out));
  }
  ck(cudaEventRecord(ev[3 * stages + 1], hp->out));
  ck(cudaStreamWaitEvent(stream, ev[3 * stages + 1], 0));
  // everything enqueued so far must drain before returning, also on an error path
  ck(cudaStreamSynchronize(hp->in));
  ck(cudaStreamSynchronize(hp->quant));
  ck(cudaStreamSynchronize(stream));
  ck(cudaStreamSynchronize(hp->attn));
  ck(cudaStreamSynchronize(hp->out));
  g_launches = 4 * (int)stages;
  if (rc != MXATTN_OK) return rc;
  if (fail) return MXATTN_ECUDA;
  // one status word per stage, at the start of its workspace slice
  std::vector<int> stw(stages, 0);
  if (cudaMemcpy(stw.data(), ws, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return MXATTN_ECUDA;
  if (stages > 1 && cudaMemcpy2D(stw.data() + 1, sizeof(int), ws + first_head(1) * w.total, (size_t)g * w.total, sizeof(int),
                                 stages - 1, cudaMemcpyDeviceToHost) != cudaSuccess) return MXATTN_ECUDA;
  for (size_t i = 0; i < stages; ++i)
    if (stw[i]) return MXATTN_ETIMEOUT;
  return MXATTN_OK;
}

// ---------------------------------------------------------------------------------------------
// Forward pass for callers that cannot allocate device memory.
//
// Some hosts of this library may not call cudaMalloc at all: code running inside another
// framework's memory plan where every byte is pre-assigned, plugins loaded into a process that
// forbids allocation after start-up, or latency-critical loops where an allocator call (and the
// implicit synchronization it can bring) is not acceptable.  For them the scratch that
// mxattn_forward needs lives in the library image itself: a fixed array in device global memory,
// present on every GPU that loads the library for as long as the process lives.
static __device__ __align__(256) unsigned char g_static_scratch[MXATTN_STATIC_SCRATCH_BYTES];

// In host code `g_static_scratch` is only a handle for the runtime, not a device address, so the
// address is looked up once per device (with that device current) and cached.
constexpr int kMaxDevices = 64;
static void* g_static_scratch_ptr[kMaxDevices] = {nullptr};

extern "C" int mxattn_forward_static(const void* q, const void* k, const void* v, void* o, int B, int H,
                                     int64_t Nq, int64_t Nkv, int d, float softmax_scale, unsigned flags,
                                     void* stream) {
  const size_t need = mxattn_forward_workspace_bytes(B, H, Nq, Nkv, d);
  if (need == 0) return (d != kHeadDim) ? MXATTN_EUNSUPPORTED : MXATTN_EINVAL;
  if (need > (size_t)MXATTN_STATIC_SCRATCH_BYTES) return MXATTN_ESCRATCH_TOO_SMALL;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return MXATTN_ECUDA;
  if (!g_static_scratch_ptr[dev]) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) return MXATTN_ECUDA;
    g_static_scratch_ptr[dev] = ptr;
  }
  return forward_ws(q, k, v, o, B, H, Nq, Nkv, d, softmax_scale, flags, g_static_scratch_ptr[dev],
                    (size_t)MXATTN_STATIC_SCRATCH_BYTES, (cudaStream_t)stream);
}

extern "C" size_t mxattn_forward_bf16_workspace_bytes(int B, int H, int64_t Nq, int64_t Nkv, int d) {
  if (B <= 0 || H <= 0 || Nq <= 0 || Nkv <= 0 || d != kHeadDim) return 0;
  return bf16_workspace_bytes(B, H, Nq, Nkv);
}

extern "C" int mxattn_forward_bf16(const void* q, const void* k, const void* v, void* o, int B, int H, int64_t Nq,
                                   int64_t Nkv, int d, float softmax_scale, unsigned flags, void* workspace,
                                   size_t workspace_bytes, void* stream) {
  if (!q || !k || !v || !o) return MXATTN_EINVAL;
  if (B <= 0 || H <= 0 || Nq <= 0 || Nkv <= 0) return MXATTN_EINVAL;
  if (flags & ~(unsigned)MXATTN_FLAG_OUT_FP32) return MXATTN_EINVAL;
  if (!(softmax_scale > 0.0f) || !(softmax_scale < 3.0e38f)) return MXATTN_EINVAL;
  if (d != kHeadDim) return MXATTN_EUNSUPPORTED;
  if (!workspace) return MXATTN_EWORKSPACE;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o) || !aligned16(workspace)) return MXATTN_EALIGN;
  g_launches = 0;
  return launch_forward_bf16(q, k, v, o, B, H, Nq, Nkv, softmax_scale, flags, workspace, workspace_bytes,
                             (cudaStream_t)stream);
}

extern "C" size_t mxattn_forward_nvfp4_workspace_bytes(int B, int H, int64_t Nq, int64_t Nkv, int d) {
  if (B <= 0 || H <= 0 || Nq <= 0 || Nkv <= 0 || d != kHeadDim) return 0;
  return nvfp4_workspace_bytes(B, H, Nq, Nkv);
}

extern "C" int mxattn_forward_nvfp4(const void* q, const void* k, const void* v, void* o, int B, int H, int64_t Nq,
                                    int64_t Nkv, int d, float softmax_scale, unsigned flags, void* workspace,
                                    size_t workspace_bytes, void* stream) {
  if (!q || !k || !v || !o) return MXATTN_EINVAL;
  if (B <= 0 || H <= 0 || Nq <= 0 || Nkv <= 0) return MXATTN_EINVAL;
  if (flags & ~(unsigned)(MXATTN_FLAG_PNQ | MXATTN_FLAG_OUT_FP32)) return MXATTN_EINVAL;
  if (!(softmax_scale > 0.0f) || !(softmax_scale < 3.0e38f)) return MXATTN_EINVAL;
  if (d != kHeadDim) return MXATTN_EUNSUPPORTED;
  if (!workspace) return MXATTN_EWORKSPACE;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o) || !aligned16(workspace)) return MXATTN_EALIGN;
  g_launches = 0;
  return launch_forward_nvfp4(q, k, v, o, B, H, Nq, Nkv, softmax_scale, flags, workspace, workspace_bytes,
                              (cudaStream_t)stream);
}

extern "C" int mxattn_device_status(const void* workspace, int* host_out, void* stream) {
  if (!workspace || !host_out) return MXATTN_EINVAL;
  if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return MXATTN_ECUDA;
  if (cudaMemcpy(host_out, workspace, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return MXATTN_ECUDA;
  return MXATTN_OK;
}

extern "C" int mxattn_selftest_bounded_wait(void* status, int64_t limit_cycles, void* stream) {
  if (!status || limit_cycles <= 0 || limit_cycles > 2000000000LL) return MXATTN_EINVAL;
  if (!aligned16(status)) return MXATTN_EALIGN;
  return launch_bounded_wait_selftest(static_cast<int*>(status), (long long)limit_cycles, (cudaStream_t)stream);
}

extern "C" int mxattn_selftest_pair_abandon(void* status, int64_t limit_cycles, int meetings, void* stream) {
  if (!status || limit_cycles <= 0 || limit_cycles > 2000000000LL || meetings <= 0 || meetings > 100000) return MXATTN_EINVAL;
  if (!aligned16(status)) return MXATTN_EALIGN;
  return launch_pair_abandon_selftest(static_cast<int*>(status), (long long)limit_cycles, meetings, (cudaStream_t)stream);
}

extern "C" int mxattn_last_launch_count(void) { return g_launches; }

extern "C" const char* mxattn_strerror(int status) {
  switch (status) {
    case MXATTN_OK: return "ok";
    case MXATTN_EINVAL: return "invalid argument";
    case MXATTN_EUNSUPPORTED: return "unsupported shape";
    case MXATTN_EALIGN: return "pointer not 16-byte aligned";
    case MXATTN_EWORKSPACE: return "workspace missing or too small";
    case MXATTN_ECUDA: return "CUDA runtime error";
    case MXATTN_ETIMEOUT: return "device-side bounded wait expired";
    case MXATTN_ESCRATCH_TOO_SMALL:
      return "problem needs more scratch than the built-in static array holds (MXATTN_STATIC_SCRATCH_BYTES); "
             "use mxattn_forward_ws with caller-provided memory";
    default: return "unknown status";
  }
}
