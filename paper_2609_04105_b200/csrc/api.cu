// C-ABI glue that is not tied to one kernel: status strings, device check, host-buffer path.
#include "common.cuh"

namespace fp4attn {

int check_device_sm100() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return FP4ATTN_ERR_CUDA;
  static std::atomic<int> cached[kMaxDevices];                 // 0 unknown, else status + 1
  const int c = cached[dev].load(std::memory_order_acquire);
  if (c) return c - 1;
  int major = 0, minor = 0;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&minor, cudaDevAttrComputeCapabilityMinor, dev) != cudaSuccess)
    return FP4ATTN_ERR_CUDA;
  const int rc = (major == 10 && minor == 0) ? FP4ATTN_OK : FP4ATTN_ERR_UNSUPPORTED_ARCH;
  cached[dev].store(rc + 1, std::memory_order_release);
  return rc;
}

}  // namespace fp4attn

extern "C" const char* fp4attn_status_string(int status) {
  switch (status) {
    case FP4ATTN_OK: return "ok";
    case FP4ATTN_ERR_INVALID_ARG: return "invalid argument";
    case FP4ATTN_ERR_UNSUPPORTED_SHAPE: return "unsupported shape (d in {64,128}, N a multiple of 128)";
    case FP4ATTN_ERR_UNSUPPORTED_ARCH: return "device is not compute capability 10.0";
    case FP4ATTN_ERR_ALIGNMENT: return "pointer alignment";
    case FP4ATTN_ERR_WORKSPACE: return "workspace missing or too small";
    case FP4ATTN_ERR_CUDA: return "CUDA call failed";
    case FP4ATTN_ERR_TIMEOUT: return "bounded in-kernel wait ran out";
    case FP4ATTN_ERR_RANGE: return "logits outside the range of the fixed row reference";
    default: return "unknown status";
  }
}

extern "C" int fp4attn_version(void) { return 300; }

static size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

namespace {
struct HostPlan {
  size_t x[3], packed[3], sf[3], G, qws, O, LSE, total;
};
bool plan(int fmt, int B, int H, int N, int d, HostPlan* p) {
  const size_t elems = (size_t)B * H * N * d;
  const size_t pk = fp4attn_packed_bytes(B, H, N, d);
  const size_t sq = fp4attn_scale_bytes(fmt, FP4ATTN_ROLE_Q, B, H, N, d);
  const size_t sv = fp4attn_scale_bytes(FP4ATTN_FMT_MXFP4, FP4ATTN_ROLE_V, B, H, N, d);
  if (!pk || !sq || !sv) return false;
  size_t off = 0;
  for (int i = 0; i < 3; ++i) { p->x[i] = off; off += align256(elems * 2); }
  for (int i = 0; i < 3; ++i) { p->packed[i] = off; off += align256(pk); }
  p->sf[0] = off; off += align256(sq);
  p->sf[1] = off; off += align256(sq);
  p->sf[2] = off; off += align256(sv);
  p->G = off; off += 256;
  p->qws = off; off += align256(fp4attn_quantize_workspace_bytes(fmt, 0, B, H, N, d) + 256);
  p->O = off; off += align256(elems * 2);
  p->LSE = off; off += align256((size_t)B * H * N * 4);
  p->total = off;
  return true;
}

// ---- MXFP4 host path, pipelined over groups of (batch, head) units.
// (batch, head) units are independent and MXFP4 needs no tensor-wide pass, so the copy in of group c + 1, the
// kernels of group c and the copy out of group c - 1 overlap: the path then costs about as much as its
// largest leg (the host-to-device copy) instead of the sum of the three.  The copies run on two internal
// streams (created on first use per device, kept until the process exits) that fork from and join back into
// the caller's stream through events, so the caller still synchronises only its own stream.
constexpr int kNoPipeline = -1;
constexpr int kMaxGroups = 16;
struct HostPipe {
  cudaStream_t h2d = nullptr, d2h = nullptr;
  cudaEvent_t start = nullptr, end = nullptr, in[kMaxGroups] = {}, done[kMaxGroups] = {};
  bool ready = false;
};
void destroy(HostPipe& hp) {
  if (hp.h2d) cudaStreamDestroy(hp.h2d);
  if (hp.d2h) cudaStreamDestroy(hp.d2h);
  if (hp.start) cudaEventDestroy(hp.start);
  if (hp.end) cudaEventDestroy(hp.end);
  for (int c = 0; c < kMaxGroups; ++c) {
    if (hp.in[c]) cudaEventDestroy(hp.in[c]);
    if (hp.done[c]) cudaEventDestroy(hp.done[c]);
  }
  hp = HostPipe();
}
std::mutex g_pipe_mutex;                                        // one pipelined enqueue at a time: the events are shared
HostPipe g_pipes[fp4attn::kMaxDevices];                         // guarded by g_pipe_mutex
// caller holds g_pipe_mutex
HostPipe* host_pipe() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= fp4attn::kMaxDevices) return nullptr;
  HostPipe& hp = g_pipes[dev];
  if (!hp.ready) {
    bool ok = cudaStreamCreateWithFlags(&hp.h2d, cudaStreamNonBlocking) == cudaSuccess &&
              cudaStreamCreateWithFlags(&hp.d2h, cudaStreamNonBlocking) == cudaSuccess &&
              cudaEventCreateWithFlags(&hp.start, cudaEventDisableTiming) == cudaSuccess &&
              cudaEventCreateWithFlags(&hp.end, cudaEventDisableTiming) == cudaSuccess;
    for (int c = 0; ok && c < kMaxGroups; ++c)
      ok = cudaEventCreateWithFlags(&hp.in[c], cudaEventDisableTiming) == cudaSuccess &&
           cudaEventCreateWithFlags(&hp.done[c], cudaEventDisableTiming) == cudaSuccess;
    if (!ok) { destroy(hp); return nullptr; }                   // nothing half-made is kept
    hp.ready = true;
  }
  return &hp;
}
// First unit of group c when BH units are cut into `groups` groups whose sizes differ by at most one: the larger groups
// come first, so that what runs after the last copy in (the last group's kernels and copy out) is as short as possible.
inline int group_begin(int BH, int groups, int c) { return BH - (int)((long long)BH * (groups - c) / groups); }
int enqueue_groups(HostPipe* hp, int groups, const void* q_host, const void* k_host, const void* v_host, float softmax_scale,
                   int BH, int N, int d, void* O_host, float* LSE_host, char* ws, const HostPlan& p, size_t workspace_bytes,
                   int* dev_status, cudaStream_t st) {
  const size_t head_elems = (size_t)N * d;
  const size_t sfq_head = fp4attn_scale_bytes(FP4ATTN_FMT_MXFP4, FP4ATTN_ROLE_Q, 1, 1, N, d);
  const size_t sfv_head = fp4attn_scale_bytes(FP4ATTN_FMT_MXFP4, FP4ATTN_ROLE_V, 1, 1, N, d);
  const char* src[3] = {(const char*)q_host, (const char*)k_host, (const char*)v_host};
#define FP4ATTN_CUDA_OK(call) do { if ((call) != cudaSuccess) return FP4ATTN_ERR_CUDA; } while (0)
  for (int c = 0; c < groups; ++c) {
    const int h0 = group_begin(BH, groups, c), nh = group_begin(BH, groups, c + 1) - h0;
    for (int i = 0; i < 3; ++i)
      FP4ATTN_CUDA_OK(cudaMemcpyAsync(ws + p.x[i] + h0 * head_elems * 2, src[i] + h0 * head_elems * 2, nh * head_elems * 2,
                                      cudaMemcpyHostToDevice, hp->h2d));
    FP4ATTN_CUDA_OK(cudaEventRecord(hp->in[c], hp->h2d));
  }
  for (int c = 0; c < groups; ++c) {
    const int h0 = group_begin(BH, groups, c), nh = group_begin(BH, groups, c + 1) - h0;
    FP4ATTN_CUDA_OK(cudaStreamWaitEvent(st, hp->in[c], 0));
    const size_t sf_head[3] = {sfq_head, sfq_head, sfv_head};
    for (int i = 0; i < 3; ++i) {
      const int rc = fp4attn_quantize(ws + p.x[i] + h0 * head_elems * 2, FP4ATTN_FMT_MXFP4, i, 1, nh, N, d,
                                      ws + p.packed[i] + h0 * head_elems / 2, ws + p.sf[i] + h0 * sf_head[i], nullptr,
                                      ws + p.qws, workspace_bytes - p.qws, (fp4attn_stream_t)st);
      if (rc != FP4ATTN_OK) return rc;
    }
    fp4attn_operands ops = {};
    ops.q = ws + p.packed[0] + h0 * head_elems / 2; ops.k = ws + p.packed[1] + h0 * head_elems / 2;
    ops.v = ws + p.packed[2] + h0 * head_elems / 2;
    ops.q_sf = ws + p.sf[0] + h0 * sfq_head; ops.k_sf = ws + p.sf[1] + h0 * sfq_head; ops.v_sf = ws + p.sf[2] + h0 * sfv_head;
    ops.qk_fmt = FP4ATTN_FMT_MXFP4;
    ops.softmax_scale = softmax_scale;
    const int rc = fp4attn_fwd(&ops, 1, nh, N, d, ws + p.O + h0 * head_elems * 2, (float*)(ws + p.LSE) + (size_t)h0 * N, dev_status,
                               (fp4attn_stream_t)st);
    if (rc != FP4ATTN_OK) return rc;
    FP4ATTN_CUDA_OK(cudaEventRecord(hp->done[c], st));
    FP4ATTN_CUDA_OK(cudaStreamWaitEvent(hp->d2h, hp->done[c], 0));
    FP4ATTN_CUDA_OK(cudaMemcpyAsync((char*)O_host + h0 * head_elems * 2, ws + p.O + h0 * head_elems * 2, nh * head_elems * 2,
                                    cudaMemcpyDeviceToHost, hp->d2h));
    if (LSE_host)
      FP4ATTN_CUDA_OK(cudaMemcpyAsync(LSE_host + (size_t)h0 * N, (float*)(ws + p.LSE) + (size_t)h0 * N, (size_t)nh * N * 4,
                                      cudaMemcpyDeviceToHost, hp->d2h));
  }
#undef FP4ATTN_CUDA_OK
  return FP4ATTN_OK;
}
int attention_host_pipelined(const void* q_host, const void* k_host, const void* v_host, float softmax_scale, int B, int H,
                             int N, int d, void* O_host, float* LSE_host, char* ws, const HostPlan& p,
                             size_t workspace_bytes, int* dev_status, cudaStream_t st) {
  const int BH = B * H;
  // Groups of heads: at least 4 (8 from 32 heads on), and about one per 32 MB of input, so that the first copy in and
  // the last kernels and copy out - the parts nothing overlaps - stay small against the whole (measured at
  // B=1, H=16, N=32768: 4 / 8 / 12 / 16 groups 9.31 / 8.74 / 8.28 / 8.62 ms, the copies alone 7.56 ms; at B=4, H=16,
  // N=4096: 4.34 / 4.39 / 4.64 ms for 4 / 8 / 16)
  int groups = BH < 8 ? 1 : (BH < 2 * kMaxGroups ? 4 : 8);
  if (groups > 1) {
    const long long by_bytes = (long long)(3ull * BH * N * d * 2 / (32ull << 20));
    if (by_bytes > groups) groups = (int)(by_bytes < kMaxGroups ? by_bytes : kMaxGroups);
    if (groups > BH) groups = BH;
  }
  if (groups == 1) return kNoPipeline;
  std::lock_guard<std::mutex> lock(g_pipe_mutex);
  HostPipe* hp = host_pipe();
  if (!hp) return kNoPipeline;
  if (cudaEventRecord(hp->start, st) != cudaSuccess ||         // fork: the copies start after the stream's earlier work
      cudaStreamWaitEvent(hp->h2d, hp->start, 0) != cudaSuccess || cudaStreamWaitEvent(hp->d2h, hp->start, 0) != cudaSuccess)
    return FP4ATTN_ERR_CUDA;
  const int rc = enqueue_groups(hp, groups, q_host, k_host, v_host, softmax_scale, BH, N, d, O_host, LSE_host, ws, p,
                                workspace_bytes, dev_status, st);
  // join on every exit, also a failed one: whatever reached the internal streams stays ordered before the
  // caller's later work on its stream (which may reuse the workspace and the host buffers)
  bool joined = cudaEventRecord(hp->end, hp->h2d) == cudaSuccess && cudaStreamWaitEvent(st, hp->end, 0) == cudaSuccess;
  joined = joined && cudaEventRecord(hp->end, hp->d2h) == cudaSuccess && cudaStreamWaitEvent(st, hp->end, 0) == cudaSuccess;
  return rc != FP4ATTN_OK ? rc : (joined ? FP4ATTN_OK : FP4ATTN_ERR_CUDA);
}
}  // namespace

extern "C" size_t fp4attn_attention_host_workspace_bytes(int qk_fmt, int B, int H, int N, int d) {
  HostPlan p;
  return plan(qk_fmt, B, H, N, d, &p) ? p.total : 0;
}

// The status word of the host path lives in the 256-byte slot of the workspace that also holds the two
// NVFP4 encode factors (floats 0 and 1); it is cleared on the caller's stream before the first kernel of the
// call and handed to every attention launch of the call.
static int* host_status_word(char* ws, const HostPlan& p) { return reinterpret_cast<int*>(ws + p.G + 64); }

static int finish_host_call(int rc, int* dev_status, int* status_host, cudaStream_t st) {
  if (rc == FP4ATTN_OK && status_host &&
      cudaMemcpyAsync(status_host, dev_status, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess)
    return FP4ATTN_ERR_CUDA;
  return rc;
}

extern "C" int fp4attn_attention_host(const void* q_host, const void* k_host, const void* v_host, int qk_fmt,
                                      float softmax_scale, int B, int H, int N, int d, void* O_host,
                                      float* LSE_host, int* status_host, void* workspace, size_t workspace_bytes,
                                      fp4attn_stream_t stream) {
  if (!q_host || !k_host || !v_host || !O_host) return FP4ATTN_ERR_INVALID_ARG;
  if (qk_fmt != FP4ATTN_FMT_MXFP4 && qk_fmt != FP4ATTN_FMT_NVFP4) return FP4ATTN_ERR_INVALID_ARG;
  if (B <= 0 || H <= 0 || N <= 0 || d <= 0) return FP4ATTN_ERR_INVALID_ARG;
  HostPlan p;
  if (!plan(qk_fmt, B, H, N, d, &p)) return FP4ATTN_ERR_UNSUPPORTED_SHAPE;
  if (!workspace || workspace_bytes < p.total) return FP4ATTN_ERR_WORKSPACE;
  if ((uintptr_t)workspace & 255) return FP4ATTN_ERR_ALIGNMENT;
  char* ws = (char*)workspace;
  cudaStream_t st = (cudaStream_t)stream;
  const size_t elems = (size_t)B * H * N * d;
  int* dev_status = host_status_word(ws, p);
  if (cudaMemsetAsync(dev_status, 0, sizeof(int), st) != cudaSuccess) return FP4ATTN_ERR_CUDA;
  if (qk_fmt == FP4ATTN_FMT_MXFP4) {
    const int rc = attention_host_pipelined(q_host, k_host, v_host, softmax_scale, B, H, N, d, O_host, LSE_host, ws, p,
                                            workspace_bytes, dev_status, st);
    if (rc != kNoPipeline) return finish_host_call(rc, dev_status, status_host, st);
  }
  const void* src[3] = {q_host, k_host, v_host};
  for (int i = 0; i < 3; ++i)
    if (cudaMemcpyAsync(ws + p.x[i], src[i], elems * 2, cudaMemcpyHostToDevice, st) != cudaSuccess)
      return FP4ATTN_ERR_CUDA;
  float* G = (float*)(ws + p.G);
  const int fmts[3] = {qk_fmt, qk_fmt, FP4ATTN_FMT_MXFP4};
  for (int i = 0; i < 3; ++i) {
    int rc = fp4attn_quantize(ws + p.x[i], fmts[i], i, B, H, N, d, ws + p.packed[i], ws + p.sf[i],
                              i < 2 ? G + i : nullptr, ws + p.qws, workspace_bytes - p.qws, stream);
    if (rc != FP4ATTN_OK) return rc;
  }
  fp4attn_operands ops = {};
  ops.q = ws + p.packed[0]; ops.k = ws + p.packed[1]; ops.v = ws + p.packed[2];
  ops.q_sf = ws + p.sf[0]; ops.k_sf = ws + p.sf[1]; ops.v_sf = ws + p.sf[2];
  ops.q_G = qk_fmt == FP4ATTN_FMT_NVFP4 ? G : nullptr;
  ops.k_G = qk_fmt == FP4ATTN_FMT_NVFP4 ? G + 1 : nullptr;
  ops.qk_fmt = qk_fmt;
  ops.softmax_scale = softmax_scale;
  int rc = fp4attn_fwd(&ops, B, H, N, d, ws + p.O, (float*)(ws + p.LSE), dev_status, stream);
  if (rc != FP4ATTN_OK) return rc;
  if (cudaMemcpyAsync(O_host, ws + p.O, elems * 2, cudaMemcpyDeviceToHost, st) != cudaSuccess) return FP4ATTN_ERR_CUDA;
  if (LSE_host &&
      cudaMemcpyAsync(LSE_host, ws + p.LSE, (size_t)B * H * N * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess)
    return FP4ATTN_ERR_CUDA;
  return finish_host_call(FP4ATTN_OK, dev_status, status_host, st);
}

namespace fp4attn { void drop_tensor_map_cache(); }

extern "C" int fp4attn_release(void) {
  std::lock_guard<std::mutex> lock(g_pipe_mutex);
  int prev = 0;
  const bool have_dev = cudaGetDevice(&prev) == cudaSuccess;
  bool ok = true;
  for (int dev = 0; dev < fp4attn::kMaxDevices; ++dev) {
    if (!g_pipes[dev].ready) continue;
    ok = cudaSetDevice(dev) == cudaSuccess && ok;
    destroy(g_pipes[dev]);
  }
  if (have_dev) cudaSetDevice(prev);
  fp4attn::drop_tensor_map_cache();
  return ok ? FP4ATTN_OK : FP4ATTN_ERR_CUDA;
}
