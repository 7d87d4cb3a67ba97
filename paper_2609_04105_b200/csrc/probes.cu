// Arithmetic ceiling of the softmax warps: the score -> code arithmetic of Algorithm "direct-p-pack"
// (block maximum, block exponent, 2^x or the affine map, E2M1 conversion and packing) run by itself - no tensor
// products, no tensor-memory traffic, no hand-offs - by as many warps per scheduler as the attention kernel gives it.
// The benchmark divides the attention kernel's rate by the rate this bound allows.
#include "attn_common.cuh"

namespace fp4attn {

constexpr int kProbeWarps = 4 * kTeams;      // the attention kernel's softmax warps: four per scheduler

__device__ __forceinline__ void probe_lds4(uint32_t addr, uint32_t* r) {
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void probe_sts4(uint32_t addr, const uint32_t* r) {
  asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" :: "r"(addr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]));
}

// Every warp converts `iters` blocks of 32 rows x 32 scores.  The scores of a block come from shared memory through
// eight loads that all lanes address alike (one wavefront each, so the loads cost issue slots like the kernel's
// tensor-memory load but no shared-memory bandwidth); the four code words go back to shared memory.
template <int PMAP>
__global__ void __launch_bounds__(32 * kProbeWarps, 1) softmax_arith_probe_kernel(int iters, float c32, float A, float B,
                                                                                 unsigned long long* cycles_out) {
  extern __shared__ __align__(16) uint8_t probe_smem[];
  const int tid = threadIdx.x, warp = tid >> 5;
  float* f = reinterpret_cast<float*>(probe_smem);
  if ((tid & 31) == 0) {
    for (int j = 0; j < 32; ++j) {                              // scores of a standard normal's range, fixed pattern
      const unsigned h = (unsigned)(warp * 32 + j + 977) * 2654435761u;
      f[warp * 32 + j] = (float)((h >> 8) & 0xffffu) * (1.0f / 8192.0f) - 4.0f;
    }
  }
  __syncthreads();
  const uint32_t in = smem_u32(probe_smem) + warp * 128;
  const uint32_t out = smem_u32(probe_smem) + kProbeWarps * 128 + tid * 16;
  int acc = 0;
  const long long t0 = clock64();
  for (int it = 0; it < iters; ++it) {
    uint32_t sraw[32], w[4];
    int E;
#pragma unroll
    for (int j = 0; j < 8; ++j) probe_lds4(in + 16 * j, &sraw[4 * j]);
    direct_p_block<PMAP, false, 0>(sraw, c32, A, B, 32, E, w);
    probe_sts4(out, w);
    acc += E;
  }
  const long long t1 = clock64();
  if (acc == 0x7fffffff) cycles_out[1] = 0;                     // keeps the exponent live; never true
  if ((tid & 31) == 0) atomicMax(cycles_out, (unsigned long long)(t1 - t0));
}

}  // namespace fp4attn

using namespace fp4attn;

extern "C" int fp4attn_softmax_arith_probe(int p_map, int exact_pairs, int iters, unsigned long long* cycles_out,
                                           fp4attn_stream_t stream) {
  if (iters <= 0 || iters > (1 << 20) || !cycles_out) return FP4ATTN_ERR_INVALID_ARG;   // 2^20 blocks per warp: about half a second
  int variant;                                                  // the kernels' template argument, as in fp4attn_fwd
  if (p_map == FP4ATTN_PMAP_IDEAL) variant = 0;
  else if (p_map == FP4ATTN_PMAP_AFFINE) variant = 1;
  else if (p_map == FP4ATTN_PMAP_HYBRID && exact_pairs == 0x1111) variant = 2;
  else if (p_map == FP4ATTN_PMAP_HYBRID && exact_pairs == 0x5555) variant = 3;
  else if (p_map == FP4ATTN_PMAP_HYBRID && exact_pairs == 0x7777) variant = 4;
  else return FP4ATTN_ERR_INVALID_ARG;
  int rc = check_device_sm100();
  if (rc != FP4ATTN_OK) return rc;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return FP4ATTN_ERR_CUDA;
  const int smem = 120 * 1024;                                  // more than half an SM's shared memory: one CTA per SM
  cudaStream_t st = (cudaStream_t)stream;
  if (cudaMemsetAsync(cycles_out, 0, 2 * sizeof(unsigned long long), st) != cudaSuccess) return FP4ATTN_ERR_CUDA;
  // the affine map's coefficients: any finite pair costs the same
  const float c32 = 0.18f, A = 1.3f, B = 0.4f;
#define FP4ATTN_PROBE(PM)                                                                                              \
  case PM:                                                                                                             \
    if (cudaFuncSetAttribute(softmax_arith_probe_kernel<PM>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) !=     \
        cudaSuccess) return FP4ATTN_ERR_CUDA;                                                                          \
    softmax_arith_probe_kernel<PM><<<sms, 32 * kProbeWarps, smem, st>>>(iters, c32, A, B, cycles_out);                 \
    break;
  switch (variant) {
    FP4ATTN_PROBE(0)
    FP4ATTN_PROBE(1)
    FP4ATTN_PROBE(2)
    FP4ATTN_PROBE(3)
    FP4ATTN_PROBE(4)
  }
#undef FP4ATTN_PROBE
  return cudaGetLastError() == cudaSuccess ? FP4ATTN_OK : FP4ATTN_ERR_CUDA;
}
