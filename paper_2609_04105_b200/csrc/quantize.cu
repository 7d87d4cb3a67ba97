// Operand quantizers: bf16 -> packed E2M1 + scale bytes in the 128x4 atom order.
// HBM-bound: 128-bit loads, block amax by lane shuffles, 32-bit / 128-bit stores.
#include "common.cuh"

namespace fp4attn {

constexpr int kThreads = 256;
constexpr int kGroupsPerThread = 4;          // 16-byte loads in flight per thread
constexpr int kGroupsPerCta = kThreads * kGroupsPerThread;
constexpr int kMaxPartials = 1024;           // NVFP4 amax pass: one partial maximum per block
constexpr int kPartialsPerHead = 32;         // the same, per (batch, head) unit, for per-head factors

// ---------------------------------------------------------------- MXFP4, blocks along d (Q, K)
// |bf16| bit patterns order like the magnitudes, so the block maximum is taken on packed 16-bit
// integers; 6 v / alpha = v * (1.5 * 2^(129-u)) is one exact fp32 multiply.
__device__ __forceinline__ uint32_t absmax_bf16x8(const uint4& r) {
  const uint32_t m = __vmaxu2(__vmaxu2(r.x & 0x7FFF7FFFu, r.y & 0x7FFF7FFFu), __vmaxu2(r.z & 0x7FFF7FFFu, r.w & 0x7FFF7FFFu));
  return max(m & 0xFFFFu, m >> 16);
}
// E8M0 byte from the bf16 bit pattern of the block maximum a = (1 + m/128) 2^(e-127): the biased exponent
// e, plus one where the rule rounds the amplitude up (Eq. "mx-scale" allows either neighbouring power of
// two): ceiling - whenever a is not a power of two; threshold - alpha = 2^floor(log2(1.6 a)), i.e. when
// 1 + m/128 >= 1.25; floor - never.  Values above the amplitude saturate at code 6 in the conversion.
template <int RULE>
__device__ __forceinline__ uint32_t mx_scale_byte_bf16(uint32_t a16) {
  if (a16 == 0) return 0;
  const uint32_t m = a16 & 0x7Fu;
  const uint32_t up = RULE == FP4ATTN_QSCALE_CEIL ? (m != 0) : RULE == FP4ATTN_QSCALE_THR16 ? (m >= 32u) : 0u;
  return min(max((a16 >> 7) + up, 1u), 254u);
}
// v[i] <- 6 v[i] / alpha for the amplitude of byte u: exact in fp32 (one multiply by 1.5 * 2^k)
template <int N_>
__device__ __forceinline__ void mx_scale_values(float* v, uint32_t u) {
  if (u >= 2u) {
    const float s6 = __uint_as_float(((256u - u) << 23) | 0x400000u);   // 1.5 * 2^(129-u) = 6 / alpha
#pragma unroll
    for (int i = 0; i < N_; i += 2)                                       // two exact products per instruction
      asm("{\n\t.reg .b64 a, b, c;\n\tmov.b64 a, {%2, %3};\n\tmov.b64 b, {%4, %4};\n\tmul.rn.f32x2 c, a, b;\n\tmov.b64 {%0, %1}, c;\n\t}"
          : "=f"(v[i]), "=f"(v[i + 1]) : "f"(v[i]), "f"(v[i + 1]), "f"(s6));
  } else {                                                              // alpha = 2^-126: 6/alpha overflows fp32
    const float inv = mx_inv_amplitude(u);
#pragma unroll
    for (int i = 0; i < N_; ++i) v[i] = (v[i] * inv) * 6.0f;
  }
}
__device__ __forceinline__ uint32_t mx_codes_x8(const uint4& raw, uint32_t u) {
  float v[8];
  bf16x8_to_f32(raw, v);
  mx_scale_values<8>(v, u);
  return cvt_e2m1x8(v);
}
// MSE rule, blocks along d: the four eight-element groups of a block sit in four adjacent lanes, so the
// group sums meet as (g0 + g1) + (g2 + g3) in every lane.  The floor's error is in units four times
// smaller than the ceiling's, hence the factor; the floor wins only if strictly better.  Returns the
// chosen byte, `word` gets this lane's codes under it.
__device__ __forceinline__ uint32_t mx_choose_mse_rows(const uint4& raw, uint32_t a16, uint32_t& word) {
  const uint32_t uf = mx_scale_byte_bf16<FP4ATTN_QSCALE_FLOOR>(a16), uc = mx_scale_byte_bf16<FP4ATTN_QSCALE_CEIL>(a16);
  float tf[8], tc[8];
  bf16x8_to_f32(raw, tf);
#pragma unroll
  for (int i = 0; i < 8; ++i) tc[i] = tf[i];
  mx_scale_values<8>(tf, uf);
  mx_scale_values<8>(tc, uc);
  const uint32_t wf = cvt_e2m1x8(tf), wc = cvt_e2m1x8(tc);
  float ef = mx_error_x8(tf, wf), ec = mx_error_x8(tc, wc);
  ef = __fadd_rn(ef, __shfl_xor_sync(0xffffffffu, ef, 1));
  ec = __fadd_rn(ec, __shfl_xor_sync(0xffffffffu, ec, 1));
  ef = __fadd_rn(ef, __shfl_xor_sync(0xffffffffu, ef, 2));
  ec = __fadd_rn(ec, __shfl_xor_sync(0xffffffffu, ec, 2));
  const bool take_f = (uf != uc) && (ef < __fmul_rn(4.0f, ec));
  word = take_f ? wf : wc;
  return take_f ? uf : uc;
}

// grid (N * D/8 / kGroupsPerCta, B*H)
template <int D, int RULE>
__global__ void __launch_bounds__(kThreads)
quant_mx_rows_kernel(const uint4* __restrict__ x, uint32_t* __restrict__ packed,
                     uint8_t* __restrict__ sf, int N) {
  constexpr int GPR = D / 8;                       // 8-element groups per row
  const uint32_t bh = blockIdx.y;
  const uint32_t gl = blockIdx.x * kGroupsPerCta + threadIdx.x;
  const size_t gbase = (size_t)bh * N * GPR;
  uint8_t* sfb = sf + (size_t)bh * (N / 128) * 512;
  uint4 raw[kGroupsPerThread];
#pragma unroll
  for (int k = 0; k < kGroupsPerThread; ++k) raw[k] = __ldg(x + gbase + gl + k * kThreads);
#pragma unroll
  for (int k = 0; k < kGroupsPerThread; ++k) {
    const uint32_t g = gl + k * kThreads;
    uint32_t a = absmax_bf16x8(raw[k]);
    a = max(a, __shfl_xor_sync(0xffffffffu, a, 1));
    a = max(a, __shfl_xor_sync(0xffffffffu, a, 2));
    uint32_t u, word;
    if (RULE == FP4ATTN_QSCALE_MSE) {
      u = mx_choose_mse_rows(raw[k], a, word);
    } else {
      u = mx_scale_byte_bf16<RULE>(a);
      word = mx_codes_x8(raw[k], u);
    }
    packed[gbase + g] = word;
    const uint32_t row = g / GPR, seg = g % GPR;
    uint8_t* p = sfb + (row >> 7) * 512 + (row & 31) * 16 + ((row & 127) >> 5) * 4;
    if ((seg & 3) == 0) p[seg >> 2] = (uint8_t)u;                    // one lane per 32-block
    if (D == 64 && (seg & 3) == 1) p[2 + (seg >> 2)] = 0;            // padding columns
  }
}

// ---------------------------------------------------------------- MXFP4, blocks along keys (V), transposed out
// A [128 keys x D] tile (contiguous in memory) goes through shared memory; a thread owns two adjacent head-dim
// columns and one 32-key block, reads them as bf16x2 words (conflict-free) and writes two 16-byte code groups.
// Persistent CTAs walk the tiles with two tile buffers: the asynchronous copies (cp.async, 16 bytes per thread
// and copy, no registers in between) of the next tile are in flight while the current one is converted, so the
// memory system always has work although each tile passes through a load -> barrier -> convert sequence.
// grid min(tiles, CTAs that fit) , 2*D threads, dynamic shared memory kVSmem<D>
template <int D> constexpr int kVTileBytes = 128 * D * 2;
template <int D> constexpr int kVSmem = 2 * kVTileBytes<D> + 512;
__device__ __forceinline__ void cp_async_16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int PENDING>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(PENDING) : "memory"); }

template <int D, int RULE>
__global__ void __launch_bounds__(2 * D, RULE == FP4ATTN_QSCALE_MSE ? 1 : (D == 128 ? 3 : 6))
quant_mx_v_kernel(const uint4* __restrict__ x, uint4* __restrict__ packed, uint8_t* __restrict__ sf, int N, int n_tiles) {
  constexpr int T = 2 * D;                         // threads: D/2 column pairs x 4 key blocks
  constexpr int LOADS = 128 * D / 8 / T;           // 16-byte copies per thread and tile: 8
  extern __shared__ __align__(16) uint8_t vsm[];
  uint8_t* sfb = vsm + 2 * kVTileBytes<D>;
  const uint32_t sbase = (uint32_t)__cvta_generic_to_shared(vsm);
  const int tiles_per_head = N / 128;
  const int cp = threadIdx.x % (D / 2);            // column pair: columns 2cp, 2cp+1
  const int kb = threadIdx.x / (D / 2);            // key block 0..3
  auto issue = [&](int t, int buf) {               // tile t is contiguous: 128 keys x D bf16 starting at key 128 t of the flat [B*H*N] key space
    const uint4* src = x + (size_t)t * (128 * D / 8);
#pragma unroll
    for (int k = 0; k < LOADS; ++k)
      cp_async_16(sbase + buf * kVTileBytes<D> + (threadIdx.x + k * T) * 16, src + threadIdx.x + k * T);
    cp_async_commit();
  };
  int t = blockIdx.x, i = 0;
  if (t < n_tiles) issue(t, 0);
  for (; t < n_tiles; t += gridDim.x, ++i) {
    const int tn = t + gridDim.x;
    if (tn < n_tiles) { issue(tn, (i + 1) & 1); cp_async_wait<1>(); } else { cp_async_wait<0>(); }
    if (threadIdx.x < 128) reinterpret_cast<uint32_t*>(sfb)[threadIdx.x] = 0;
    __syncthreads();
    const uint32_t* tile = reinterpret_cast<const uint32_t*>(vsm + (i & 1) * kVTileBytes<D>);
    const size_t bh = t / tiles_per_head;
    const int kt = t - (int)bh * tiles_per_head;     // 128-key tile within the head
    uint32_t w[32];
    uint32_t m = 0;
#pragma unroll
    for (int r = 0; r < 32; ++r) {
      w[r] = tile[(kb * 32 + r) * (D / 2) + cp];
      m = __vmaxu2(m, w[r] & 0x7FFF7FFFu);
    }
#pragma unroll
    for (int c = 0; c < 2; ++c) {                    // low half = column 2cp, high half = column 2cp+1
      const uint32_t a16 = c ? (m >> 16) : (m & 0xFFFFu);
      uint32_t u = mx_scale_byte_bf16<RULE == FP4ATTN_QSCALE_MSE ? FP4ATTN_QSCALE_CEIL : RULE>(a16);
      float v[32];
#pragma unroll
      for (int r = 0; r < 32; ++r) v[r] = __uint_as_float(c ? (w[r] & 0xFFFF0000u) : (w[r] << 16));
      uint4 out;
      if (RULE == FP4ATTN_QSCALE_MSE) {
        // both amplitudes; group sums of eight consecutive keys combined as (g0 + g1) + (g2 + g3)
        const uint32_t uf = mx_scale_byte_bf16<FP4ATTN_QSCALE_FLOOR>(a16);
        float tf[32];
#pragma unroll
        for (int r = 0; r < 32; ++r) tf[r] = v[r];
        mx_scale_values<32>(tf, uf);
        mx_scale_values<32>(v, u);
        uint32_t wf[4], wc[4];
        float gf[4], gc[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          wf[j] = cvt_e2m1x8(tf + 8 * j);
          wc[j] = cvt_e2m1x8(v + 8 * j);
          gf[j] = mx_error_x8(tf + 8 * j, wf[j]);
          gc[j] = mx_error_x8(v + 8 * j, wc[j]);
        }
        const float ef = __fadd_rn(__fadd_rn(gf[0], gf[1]), __fadd_rn(gf[2], gf[3]));
        const float ec = __fadd_rn(__fadd_rn(gc[0], gc[1]), __fadd_rn(gc[2], gc[3]));
        const bool take_f = (uf != u) && (ef < __fmul_rn(4.0f, ec));
        out = take_f ? make_uint4(wf[0], wf[1], wf[2], wf[3]) : make_uint4(wc[0], wc[1], wc[2], wc[3]);
        u = take_f ? uf : u;
      } else {
        mx_scale_values<32>(v, u);
        out.x = cvt_e2m1x8(v);
        out.y = cvt_e2m1x8(v + 8);
        out.z = cvt_e2m1x8(v + 16);
        out.w = cvt_e2m1x8(v + 24);
      }
      const int col = 2 * cp + c;
      packed[((bh * D + col) * (size_t)(N / 2) + (size_t)kt * 64 + kb * 16) / 16] = out;
      sfb[col * 4 + kb] = (uint8_t)u;
    }
    __syncthreads();
    if (threadIdx.x < 128) {
      const int r = threadIdx.x;                     // head-dim row; rows >= D are zero padding
      uint8_t* p = sf + (bh * (size_t)tiles_per_head + kt) * 512 + (r & 31) * 16 + (r >> 5) * 4;
      *reinterpret_cast<uint32_t*>(p) = reinterpret_cast<const uint32_t*>(sfb)[r];
    }
    __syncthreads();                                 // the tile buffer and the scale staging are free again
  }
}

// ---------------------------------------------------------------- E4M3 V (FP8 P/V route), transposed out
// Same tile pipeline as the MXFP4 V kernel; a thread owns two adjacent head-dim columns and one 32-key block and
// writes 32 bytes per column: byte = Q_E4M3(fl32(v * G)), G the unit's encode factor (one per (batch, head)).
__device__ __forceinline__ uint32_t cvt_e4m3x4(float a, float b, float c, float d) {   // a in bits 0-7 ... d in bits 24-31
  uint32_t w;
  asm("{\n\t.reg .b16 lo, hi;\n\t"
      "cvt.rn.satfinite.e4m3x2.f32 lo, %2, %1;\n\t"
      "cvt.rn.satfinite.e4m3x2.f32 hi, %4, %3;\n\t"
      "mov.b32 %0, {lo, hi};\n\t}"
      : "=r"(w) : "f"(a), "f"(b), "f"(c), "f"(d));
  return w;
}
template <int D>
__global__ void __launch_bounds__(2 * D, D == 128 ? 3 : 6)
quant_e4m3_v_kernel(const uint4* __restrict__ x, uint4* __restrict__ bytes_out, const float* __restrict__ G_in, int N, int n_tiles) {
  constexpr int T = 2 * D;
  constexpr int LOADS = 128 * D / 8 / T;
  extern __shared__ __align__(16) uint8_t vsm[];
  const uint32_t sbase = (uint32_t)__cvta_generic_to_shared(vsm);
  const int tiles_per_head = N / 128;
  const int cp = threadIdx.x % (D / 2);
  const int kb = threadIdx.x / (D / 2);
  auto issue = [&](int t, int buf) {
    const uint4* src = x + (size_t)t * (128 * D / 8);
#pragma unroll
    for (int k = 0; k < LOADS; ++k)
      cp_async_16(sbase + buf * kVTileBytes<D> + (threadIdx.x + k * T) * 16, src + threadIdx.x + k * T);
    cp_async_commit();
  };
  int t = blockIdx.x, i = 0;
  if (t < n_tiles) issue(t, 0);
  for (; t < n_tiles; t += gridDim.x, ++i) {
    const int tn = t + gridDim.x;
    if (tn < n_tiles) { issue(tn, (i + 1) & 1); cp_async_wait<1>(); } else { cp_async_wait<0>(); }
    __syncthreads();
    const uint32_t* tile = reinterpret_cast<const uint32_t*>(vsm + (i & 1) * kVTileBytes<D>);
    const size_t bh = t / tiles_per_head;
    const int kt = t - (int)bh * tiles_per_head;
    const float G = __ldg(G_in + bh);
    uint32_t w[32];
#pragma unroll
    for (int r = 0; r < 32; ++r) w[r] = tile[(kb * 32 + r) * (D / 2) + cp];
#pragma unroll
    for (int c = 0; c < 2; ++c) {
      uint32_t o[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        float v[4];
#pragma unroll
        for (int e = 0; e < 4; ++e)
          v[e] = __fmul_rn(__uint_as_float(c ? (w[4 * j + e] & 0xFFFF0000u) : (w[4 * j + e] << 16)), G);
        o[j] = cvt_e4m3x4(v[0], v[1], v[2], v[3]);
      }
      const int col = 2 * cp + c;
      uint4* dst = bytes_out + ((bh * D + col) * (size_t)N + (size_t)kt * 128 + kb * 32) / 16;
      dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
      dst[1] = make_uint4(o[4], o[5], o[6], o[7]);
    }
    __syncthreads();
  }
}

// One block per unit: G = fl32(448 / max of the unit's partial maxima) (1 for an all-zero unit)
__global__ void __launch_bounds__(kThreads)
e4m3_encode_factor_kernel(const float* __restrict__ partials, int n_partials, float* __restrict__ G_out) {
  partials += (size_t)blockIdx.x * n_partials;
  float a = 0.f;
  for (int i = threadIdx.x; i < n_partials; i += kThreads) a = fmaxf(a, partials[i]);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, o));
  __shared__ float wmax[kThreads / 32];
  if ((threadIdx.x & 31) == 0) wmax[threadIdx.x >> 5] = a;
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int i = 1; i < kThreads / 32; ++i) a = fmaxf(a, wmax[i]);
    G_out[blockIdx.x] = (a == 0.f) ? 1.0f : __fdiv_rn(448.0f, a);
  }
}

// ---------------------------------------------------------------- NVFP4 pass 1: amax partials
// grid (P, U): U = 1 for the tensor-wide maximum, U = B*H for one maximum per (batch, head) unit; row y of
// the grid covers groups [y * n_groups, (y + 1) * n_groups) and writes partials[y * P .. y * P + P)
__global__ void __launch_bounds__(kThreads)
amax_partials_kernel(const uint4* __restrict__ x, size_t n_groups, float* __restrict__ partials) {
  x += (size_t)blockIdx.y * n_groups;
  partials += (size_t)blockIdx.y * gridDim.x;
  // |bf16| bit patterns order like the magnitudes: packed 16-bit maxima, four independent loads per trip
  uint32_t m = 0;
  const size_t stride = (size_t)gridDim.x * kThreads;
  size_t g = (size_t)blockIdx.x * kThreads + threadIdx.x;
  for (; g + 3 * stride < n_groups; g += 4 * stride) {
    const uint4 r0 = __ldg(x + g), r1 = __ldg(x + g + stride), r2 = __ldg(x + g + 2 * stride), r3 = __ldg(x + g + 3 * stride);
    m = max(max(m, absmax_bf16x8(r0)), max(absmax_bf16x8(r1), max(absmax_bf16x8(r2), absmax_bf16x8(r3))));
  }
  for (; g < n_groups; g += stride) m = max(m, absmax_bf16x8(__ldg(x + g)));
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xffffffffu, m, o));
  __shared__ uint32_t wmax[kThreads / 32];
  if ((threadIdx.x & 31) == 0) wmax[threadIdx.x >> 5] = m;
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int i = 1; i < kThreads / 32; ++i) m = max(m, wmax[i]);
    partials[blockIdx.x] = __uint_as_float(m << 16);
  }
}

// One block per encode factor: G = fl32(2688 / max of its partial maxima) (1 for an all-zero tensor or unit).
// grid (U): block y reads partials[y * n_partials ..) and writes G_out[y]
__global__ void __launch_bounds__(kThreads)
nv_encode_factor_kernel(const float* __restrict__ partials, int n_partials, float* __restrict__ G_out) {
  partials += (size_t)blockIdx.x * n_partials;
  float a = 0.f;
  for (int i = threadIdx.x; i < n_partials; i += kThreads) a = fmaxf(a, partials[i]);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, o));
  __shared__ float wmax[kThreads / 32];
  if ((threadIdx.x & 31) == 0) wmax[threadIdx.x >> 5] = a;
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int i = 1; i < kThreads / 32; ++i) a = fmaxf(a, wmax[i]);
    G_out[blockIdx.x] = (a == 0.f) ? 1.0f : __fdiv_rn(2688.0f, a);
  }
}

__device__ __forceinline__ uint32_t cvt_e4m3_byte(float t) {     // RNE, saturating at 448
  uint16_t r;
  asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(0.f), "f"(t));
  return r & 0xFFu;
}
__device__ __forceinline__ float e4m3_byte_to_f32(uint32_t b) {
  uint32_t h2;
  asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"((uint16_t)b));
  return __half2float(__ushort_as_half((unsigned short)(h2 & 0xFFFFu)));
}

// ---------------------------------------------------------------- NVFP4 pass 3, blocks of 16 along d (Q, K)
// grid (N * D/8 / kGroupsPerCta, B*H)
template <int D>
__global__ void __launch_bounds__(kThreads)
quant_nv_rows_kernel(const uint4* __restrict__ x, uint32_t* __restrict__ packed, uint8_t* __restrict__ sf,
                     const float* __restrict__ G_in, int N, int per_head) {
  constexpr int GPR = D / 8;
  constexpr int CT = (D / 16 + 3) / 4;
  const float G = __ldg(G_in + (per_head ? blockIdx.y : 0));    // this block's (batch, head) unit, or the tensor's
  const uint32_t bh = blockIdx.y;
  const uint32_t gl = blockIdx.x * kGroupsPerCta + threadIdx.x;
  const size_t gbase = (size_t)bh * N * GPR;
  uint8_t* sfb = sf + (size_t)bh * (N / 128) * CT * 512;
  uint4 raw[kGroupsPerThread];
#pragma unroll
  for (int k = 0; k < kGroupsPerThread; ++k) raw[k] = __ldg(x + gbase + gl + k * kThreads);
#pragma unroll
  for (int k = 0; k < kGroupsPerThread; ++k) {
    const uint32_t g = gl + k * kThreads;
    uint32_t a16 = absmax_bf16x8(raw[k]);
    a16 = max(a16, __shfl_xor_sync(0xffffffffu, a16, 1));
    const float a = __uint_as_float(a16 << 16);
    const float t = __fdiv_rn(__fmul_rn(a, G), 6.0f);
    const uint32_t sb = cvt_e4m3_byte(t);
    const float S = e4m3_byte_to_f32(sb);
    const float r = (S > 0.f) ? __fdiv_rn(G, S) : 0.f;
    float v[8];
    bf16x8_to_f32(raw[k], v);
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = __fmul_rn(v[i], r);       // sign rides along; 0*r = 0 for zero blocks
    packed[gbase + g] = cvt_e2m1x8(v);
    const uint32_t row = g / GPR, seg = g % GPR;
    if ((seg & 1) == 0) {                                        // one lane per 16-block
      const uint32_t c = seg >> 1;                               // scale column
      sfb[((row >> 7) * CT + (c >> 2)) * 512 + (row & 31) * 16 + ((row & 127) >> 5) * 4 + (c & 3)] = (uint8_t)sb;
    }
  }
}

}  // namespace fp4attn

using namespace fp4attn;

extern "C" size_t fp4attn_packed_bytes(int B, int H, int N, int d) {
  if (B <= 0 || H <= 0 || N <= 0 || d <= 0) return 0;
  return (size_t)B * H * N * d / 2;
}

static bool shape_ok(int B, int H, int N, int d) {
  return B > 0 && H > 0 && (d == 64 || d == 128) && N >= 128 && N % 128 == 0;
}

extern "C" size_t fp4attn_scale_bytes(int fmt, int role, int B, int H, int N, int d) {
  if (!shape_ok(B, H, N, d)) return 0;
  if (role == FP4ATTN_ROLE_V) {
    if (fmt != FP4ATTN_FMT_MXFP4) return 0;
    return (size_t)B * H * ((d + 127) / 128) * (N / 128) * 512;          // rows d, columns N/32
  }
  if (role != FP4ATTN_ROLE_Q && role != FP4ATTN_ROLE_K) return 0;
  if (fmt != FP4ATTN_FMT_MXFP4 && fmt != FP4ATTN_FMT_NVFP4) return 0;
  const int C = d / (fmt == FP4ATTN_FMT_MXFP4 ? 32 : 16);
  return (size_t)B * H * (N / 128) * ((C + 3) / 4) * 512;
}

extern "C" size_t fp4attn_quantize_workspace_bytes(int fmt, int role, int B, int H, int N, int d) {
  (void)role; (void)B; (void)H; (void)N; (void)d;
  return fmt == FP4ATTN_FMT_NVFP4 ? (size_t)kMaxPartials * sizeof(float) : 0;
}

namespace fp4attn {
// V kernel: persistent CTAs, as many as fit per SM with two tile buffers each (the opt-in to more than 48 KB of
// dynamic shared memory is set once per device and instance)
template <int D, int RULE>
static void launch_mx_v(const uint4* xs, int n_tiles, int N, void* packed, void* scales, cudaStream_t st) {
  static std::atomic<int> ctas[kMaxDevices];        // 0 unknown, else CTAs of the persistent grid
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return;   // the launch check below reports it
  int grid = ctas[dev].load(std::memory_order_acquire);
  if (!grid) {
    int sms = 0, per_sm = 0;
    if (cudaFuncSetAttribute(quant_mx_v_kernel<D, RULE>, cudaFuncAttributeMaxDynamicSharedMemorySize, kVSmem<D>) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, quant_mx_v_kernel<D, RULE>, 2 * D, kVSmem<D>) != cudaSuccess || per_sm < 1)
      return;
    grid = sms * per_sm;
    ctas[dev].store(grid, std::memory_order_release);
  }
  quant_mx_v_kernel<D, RULE><<<n_tiles < grid ? n_tiles : grid, 2 * D, kVSmem<D>, st>>>(xs, (uint4*)packed, (uint8_t*)scales, N, n_tiles);
}

// Shared by fp4attn_quantize and the variants that bring their own scratch.
template <int RULE>
static void launch_mx(const uint4* xs, int role, int B, int H, int N, int d, void* packed, void* scales, cudaStream_t st) {
  if (role != FP4ATTN_ROLE_V) {
    const dim3 grid2((unsigned)((size_t)N * d / 8 / kGroupsPerCta), (unsigned)(B * H));   // N % 128 == 0 makes this exact
    if (d == 128) quant_mx_rows_kernel<128, RULE><<<grid2, kThreads, 0, st>>>(xs, (uint32_t*)packed, (uint8_t*)scales, N);
    else          quant_mx_rows_kernel<64, RULE><<<grid2, kThreads, 0, st>>>(xs, (uint32_t*)packed, (uint8_t*)scales, N);
  } else if (d == 128) {
    launch_mx_v<128, RULE>(xs, B * H * (N / 128), N, packed, scales, st);
  } else {
    launch_mx_v<64, RULE>(xs, B * H * (N / 128), N, packed, scales, st);
  }
}

int launch_quantize(const void* x, int fmt, int role, int B, int H, int N, int d, void* packed, void* scales,
                    float* G_out, float* partials, cudaStream_t st, int mx_rule, bool per_head = false) {
  const size_t n_groups = (size_t)B * H * N * d / 8;
  const unsigned grid = (unsigned)(n_groups / kGroupsPerCta);
  const dim3 grid2((unsigned)((size_t)N * d / 8 / kGroupsPerCta), (unsigned)(B * H));   // N % 128 == 0 makes this exact
  const uint4* xs = reinterpret_cast<const uint4*>(x);
  if (fmt == FP4ATTN_FMT_MXFP4) {
    if (mx_rule == FP4ATTN_QSCALE_THR16)      launch_mx<FP4ATTN_QSCALE_THR16>(xs, role, B, H, N, d, packed, scales, st);
    else if (mx_rule == FP4ATTN_QSCALE_FLOOR) launch_mx<FP4ATTN_QSCALE_FLOOR>(xs, role, B, H, N, d, packed, scales, st);
    else if (mx_rule == FP4ATTN_QSCALE_MSE)   launch_mx<FP4ATTN_QSCALE_MSE>(xs, role, B, H, N, d, packed, scales, st);
    else                                      launch_mx<FP4ATTN_QSCALE_CEIL>(xs, role, B, H, N, d, packed, scales, st);
  } else {
    int n_partials;
    if (per_head) {
      n_partials = (int)(grid2.x < (unsigned)kPartialsPerHead ? grid2.x : kPartialsPerHead);
      amax_partials_kernel<<<dim3(n_partials, B * H), kThreads, 0, st>>>(xs, n_groups / ((size_t)B * H), partials);
    } else {
      n_partials = (int)(grid < (unsigned)kMaxPartials ? grid : kMaxPartials);
      amax_partials_kernel<<<n_partials, kThreads, 0, st>>>(xs, n_groups, partials);
    }
    nv_encode_factor_kernel<<<per_head ? B * H : 1, kThreads, 0, st>>>(partials, n_partials, G_out);
    if (d == 128) quant_nv_rows_kernel<128><<<grid2, kThreads, 0, st>>>(xs, (uint32_t*)packed, (uint8_t*)scales, G_out, N, per_head);
    else          quant_nv_rows_kernel<64><<<grid2, kThreads, 0, st>>>(xs, (uint32_t*)packed, (uint8_t*)scales, G_out, N, per_head);
  }
  return cudaGetLastError() == cudaSuccess ? FP4ATTN_OK : FP4ATTN_ERR_CUDA;
}

int validate_quantize(const void* x, int fmt, int role, int B, int H, int N, int d, const void* packed,
                      const void* scales, const float* G_out) {
  if (!x || !packed || !scales) return FP4ATTN_ERR_INVALID_ARG;
  if (fmt != FP4ATTN_FMT_MXFP4 && fmt != FP4ATTN_FMT_NVFP4) return FP4ATTN_ERR_INVALID_ARG;
  if (role != FP4ATTN_ROLE_Q && role != FP4ATTN_ROLE_K && role != FP4ATTN_ROLE_V) return FP4ATTN_ERR_INVALID_ARG;
  if (B <= 0 || H <= 0 || N <= 0 || d <= 0) return FP4ATTN_ERR_INVALID_ARG;
  if (!shape_ok(B, H, N, d)) return FP4ATTN_ERR_UNSUPPORTED_SHAPE;
  if (fmt == FP4ATTN_FMT_NVFP4 && role == FP4ATTN_ROLE_V) return FP4ATTN_ERR_INVALID_ARG;   // V is always MXFP4
  if (fmt == FP4ATTN_FMT_NVFP4 && !G_out) return FP4ATTN_ERR_INVALID_ARG;
  if (((uintptr_t)x | (uintptr_t)packed | (uintptr_t)scales) & 15) return FP4ATTN_ERR_ALIGNMENT;
  return FP4ATTN_OK;
}
}  // namespace fp4attn

extern "C" int fp4attn_quantize(const void* x, int fmt, int role, int B, int H, int N, int d, void* packed,
                                void* scales, float* G_out, void* workspace, size_t workspace_bytes,
                                fp4attn_stream_t stream) {
  int rc = validate_quantize(x, fmt, role, B, H, N, d, packed, scales, G_out);
  if (rc != FP4ATTN_OK) return rc;
  const size_t need = fp4attn_quantize_workspace_bytes(fmt, role, B, H, N, d);
  if (need && (!workspace || workspace_bytes < need)) return FP4ATTN_ERR_WORKSPACE;
  if (need && ((uintptr_t)workspace & 15)) return FP4ATTN_ERR_ALIGNMENT;
  rc = check_device_sm100();
  if (rc != FP4ATTN_OK) return rc;
  return launch_quantize(x, fmt, role, B, H, N, d, packed, scales, G_out, (float*)workspace, (cudaStream_t)stream,
                         FP4ATTN_QSCALE_CEIL);
}

extern "C" int fp4attn_quantize_mxfp4_rule(const void* x, int role, int scale_rule, int B, int H, int N, int d,
                                           void* packed, void* scales, fp4attn_stream_t stream) {
  if (scale_rule != FP4ATTN_QSCALE_CEIL && scale_rule != FP4ATTN_QSCALE_THR16 && scale_rule != FP4ATTN_QSCALE_FLOOR &&
      scale_rule != FP4ATTN_QSCALE_MSE)
    return FP4ATTN_ERR_INVALID_ARG;
  int rc = validate_quantize(x, FP4ATTN_FMT_MXFP4, role, B, H, N, d, packed, scales, nullptr);
  if (rc != FP4ATTN_OK) return rc;
  rc = check_device_sm100();
  if (rc != FP4ATTN_OK) return rc;
  return launch_quantize(x, FP4ATTN_FMT_MXFP4, role, B, H, N, d, packed, scales, nullptr, nullptr, (cudaStream_t)stream,
                         scale_rule);
}

extern "C" size_t fp4attn_quantize_nvfp4_per_head_workspace_bytes(int B, int H, int N, int d) {
  if (!shape_ok(B, H, N, d)) return 0;
  return (size_t)B * H * kPartialsPerHead * sizeof(float);
}

extern "C" int fp4attn_quantize_nvfp4_per_head(const void* x, int role, int B, int H, int N, int d, void* packed,
                                               void* scales, float* G_out, void* workspace, size_t workspace_bytes,
                                               fp4attn_stream_t stream) {
  int rc = validate_quantize(x, FP4ATTN_FMT_NVFP4, role, B, H, N, d, packed, scales, G_out);
  if (rc != FP4ATTN_OK) return rc;
  const size_t need = fp4attn_quantize_nvfp4_per_head_workspace_bytes(B, H, N, d);
  if (!workspace || workspace_bytes < need) return FP4ATTN_ERR_WORKSPACE;
  if ((uintptr_t)workspace & 15) return FP4ATTN_ERR_ALIGNMENT;
  rc = check_device_sm100();
  if (rc != FP4ATTN_OK) return rc;
  return launch_quantize(x, FP4ATTN_FMT_NVFP4, role, B, H, N, d, packed, scales, G_out, (float*)workspace,
                         (cudaStream_t)stream, FP4ATTN_QSCALE_CEIL, true);
}

// ---------------------------------------------------------------- allocation-free NVFP4 variant
// Scratch for the amax pass lives in the library image.  In host code the symbol below is only a
// handle; the device address is fetched once per device with cudaGetSymbolAddress.
static __device__ __align__(256) float g_noalloc_partials[kMaxPartials];

extern "C" int fp4attn_quantize_nvfp4_noalloc(const void* x, int role, int B, int H, int N, int d, void* packed,
                                              void* scales, float* G_out, fp4attn_stream_t stream) {
  int rc = validate_quantize(x, FP4ATTN_FMT_NVFP4, role, B, H, N, d, packed, scales, G_out);
  if (rc != FP4ATTN_OK) return rc;
  if ((unsigned long long)B * H * N * d > FP4ATTN_NOALLOC_MAX_ELEMENTS) return FP4ATTN_ERR_WORKSPACE;
  rc = check_device_sm100();
  if (rc != FP4ATTN_OK) return rc;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return FP4ATTN_ERR_CUDA;
  // per-device address of g_noalloc_partials; several host threads may make the first call on a device at
  // once (they all store the same address)
  static std::atomic<float*> scratch_addr[kMaxDevices];
  if (dev < 0 || dev >= kMaxDevices) return FP4ATTN_ERR_INVALID_ARG;
  float* scratch = scratch_addr[dev].load(std::memory_order_acquire);
  if (!scratch) {
    if (cudaGetSymbolAddress((void**)&scratch, g_noalloc_partials) != cudaSuccess || !scratch) return FP4ATTN_ERR_CUDA;
    scratch_addr[dev].store(scratch, std::memory_order_release);
  }
  return launch_quantize(x, FP4ATTN_FMT_NVFP4, role, B, H, N, d, packed, scales, G_out, scratch,
                         (cudaStream_t)stream, FP4ATTN_QSCALE_CEIL);
}

// ---------------------------------------------------------------- E4M3 V of the FP8 P/V route
extern "C" size_t fp4attn_quantize_v_e4m3_workspace_bytes(int B, int H, int N, int d) {
  if (!shape_ok(B, H, N, d)) return 0;
  return (size_t)B * H * kPartialsPerHead * sizeof(float);
}

template <int D>
static int launch_e4m3_v(const uint4* xs, int BH, int N, void* bytes_out, const float* G, cudaStream_t st) {
  static std::atomic<int> ctas[kMaxDevices];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return FP4ATTN_ERR_CUDA;
  int grid = ctas[dev].load(std::memory_order_acquire);
  if (!grid) {
    int sms = 0, per_sm = 0;
    if (cudaFuncSetAttribute(quant_e4m3_v_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, 2 * kVTileBytes<D>) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, quant_e4m3_v_kernel<D>, 2 * D, 2 * kVTileBytes<D>) != cudaSuccess || per_sm < 1)
      return FP4ATTN_ERR_CUDA;
    grid = sms * per_sm;
    ctas[dev].store(grid, std::memory_order_release);
  }
  const int n_tiles = BH * (N / 128);
  quant_e4m3_v_kernel<D><<<n_tiles < grid ? n_tiles : grid, 2 * D, 2 * kVTileBytes<D>, st>>>(xs, (uint4*)bytes_out, G, N, n_tiles);
  return FP4ATTN_OK;
}

extern "C" int fp4attn_quantize_v_e4m3(const void* x, int B, int H, int N, int d, void* bytes_out, float* G_out,
                                       void* workspace, size_t workspace_bytes, fp4attn_stream_t stream) {
  if (!x || !bytes_out || !G_out) return FP4ATTN_ERR_INVALID_ARG;
  if (B <= 0 || H <= 0 || N <= 0 || d <= 0) return FP4ATTN_ERR_INVALID_ARG;
  if (!shape_ok(B, H, N, d)) return FP4ATTN_ERR_UNSUPPORTED_SHAPE;
  if (((uintptr_t)x | (uintptr_t)bytes_out) & 15) return FP4ATTN_ERR_ALIGNMENT;
  const size_t need = fp4attn_quantize_v_e4m3_workspace_bytes(B, H, N, d);
  if (!workspace || workspace_bytes < need) return FP4ATTN_ERR_WORKSPACE;
  if ((uintptr_t)workspace & 15) return FP4ATTN_ERR_ALIGNMENT;
  int rc = check_device_sm100();
  if (rc != FP4ATTN_OK) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  const uint4* xs = reinterpret_cast<const uint4*>(x);
  const size_t groups_per_unit = (size_t)N * d / 8;
  const unsigned gx = (unsigned)(groups_per_unit / kGroupsPerCta);
  const int n_partials = (int)(gx < (unsigned)kPartialsPerHead ? gx : kPartialsPerHead);
  amax_partials_kernel<<<dim3(n_partials, B * H), kThreads, 0, st>>>(xs, groups_per_unit, (float*)workspace);
  e4m3_encode_factor_kernel<<<B * H, kThreads, 0, st>>>((const float*)workspace, n_partials, G_out);
  rc = d == 128 ? launch_e4m3_v<128>(xs, B * H, N, bytes_out, G_out, st) : launch_e4m3_v<64>(xs, B * H, N, bytes_out, G_out, st);
  if (rc != FP4ATTN_OK) return rc;
  return cudaGetLastError() == cudaSuccess ? FP4ATTN_OK : FP4ATTN_ERR_CUDA;
}
