// C-ABI glue that is not tied to one kernel: status strings, device check, host-buffer path.
#include "common.cuh"

namespace fp4attn {

int check_device_sm100() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return FP4ATTN_ERR_CUDA;
  static int cached_dev = -1, cached_rc = FP4ATTN_OK;
  if (dev == cached_dev) return cached_rc;
  int major = 0, minor = 0;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&minor, cudaDevAttrComputeCapabilityMinor, dev) != cudaSuccess)
    return FP4ATTN_ERR_CUDA;
  cached_rc = (major == 10 && minor == 0) ? FP4ATTN_OK : FP4ATTN_ERR_UNSUPPORTED_ARCH;
  cached_dev = dev;
  return cached_rc;
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
    default: return "unknown status";
  }
}

extern "C" int fp4attn_version(void) { return 100; }

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
}  // namespace

extern "C" size_t fp4attn_attention_host_workspace_bytes(int qk_fmt, int B, int H, int N, int d) {
  HostPlan p;
  return plan(qk_fmt, B, H, N, d, &p) ? p.total : 0;
}

extern "C" int fp4attn_attention_host(const void* q_host, const void* k_host, const void* v_host, int qk_fmt,
                                      float softmax_scale, int B, int H, int N, int d, void* O_host,
                                      float* LSE_host, void* workspace, size_t workspace_bytes,
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
  int rc = fp4attn_fwd(&ops, B, H, N, d, ws + p.O, (float*)(ws + p.LSE), nullptr, stream);
  if (rc != FP4ATTN_OK) return rc;
  if (cudaMemcpyAsync(O_host, ws + p.O, elems * 2, cudaMemcpyDeviceToHost, st) != cudaSuccess) return FP4ATTN_ERR_CUDA;
  if (LSE_host &&
      cudaMemcpyAsync(LSE_host, ws + p.LSE, (size_t)B * H * N * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess)
    return FP4ATTN_ERR_CUDA;
  return FP4ATTN_OK;
}
