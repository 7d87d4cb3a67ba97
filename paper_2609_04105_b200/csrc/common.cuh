// Shared device helpers for the fp4attn kernels (sm_100a only).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <stdint.h>

#include <atomic>
#include <mutex>

#include "../../include/fp4attn.h"

namespace fp4attn {

// Eight floats -> one 32-bit word of eight E2M1 codes (element k in nibble k).
__device__ __forceinline__ uint32_t cvt_e2m1x8(const float* v) {
  uint32_t w;
  asm("{\n\t.reg .b8 t0, t1, t2, t3;\n\t"
      "cvt.rn.satfinite.e2m1x2.f32 t0, %2, %1;\n\t"
      "cvt.rn.satfinite.e2m1x2.f32 t1, %4, %3;\n\t"
      "cvt.rn.satfinite.e2m1x2.f32 t2, %6, %5;\n\t"
      "cvt.rn.satfinite.e2m1x2.f32 t3, %8, %7;\n\t"
      "mov.b32 %0, {t0, t1, t2, t3};\n\t}"
      : "=r"(w)
      : "f"(v[0]), "f"(v[1]), "f"(v[2]), "f"(v[3]), "f"(v[4]), "f"(v[5]), "f"(v[6]), "f"(v[7]));
  return w;
}

// same, with negative inputs clamped to +0 by the conversion itself
__device__ __forceinline__ uint32_t cvt_e2m1x8_relu(const float* v) {
  uint32_t w;
  asm("{\n\t.reg .b8 t0, t1, t2, t3;\n\t"
      "cvt.rn.satfinite.relu.e2m1x2.f32 t0, %2, %1;\n\t"
      "cvt.rn.satfinite.relu.e2m1x2.f32 t1, %4, %3;\n\t"
      "cvt.rn.satfinite.relu.e2m1x2.f32 t2, %6, %5;\n\t"
      "cvt.rn.satfinite.relu.e2m1x2.f32 t3, %8, %7;\n\t"
      "mov.b32 %0, {t0, t1, t2, t3};\n\t}"
      : "=r"(w)
      : "f"(v[0]), "f"(v[1]), "f"(v[2]), "f"(v[3]), "f"(v[4]), "f"(v[5]), "f"(v[6]), "f"(v[7]));
  return w;
}

// Squared error of eight scaled values t against their codes (one word), in code units: d = t - q exact,
// fl32(d * d) added left to right in fp32 - the order the MSE amplitude rule is defined with.
__device__ __forceinline__ float mx_error_x8(const float* t, uint32_t codes) {
  float acc = 0.f;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    uint32_t h2;
    asm("{\n\t.reg .b8 b;\n\t.reg .b32 s;\n\tshr.b32 s, %1, %2;\n\tcvt.u8.u32 b, s;\n\tcvt.rn.f16x2.e2m1x2 %0, b;\n\t}"
        : "=r"(h2) : "r"(codes), "r"(8 * i));
    const float2 q = __half22float2(*reinterpret_cast<const __half2*>(&h2));
    const float d0 = __fsub_rn(t[2 * i], q.x), d1 = __fsub_rn(t[2 * i + 1], q.y);
    const float s0 = __fmul_rn(d0, d0), s1 = __fmul_rn(d1, d1);
    acc = (i == 0) ? s0 : __fadd_rn(acc, s0);
    acc = __fadd_rn(acc, s1);
  }
  return acc;
}
__device__ __forceinline__ void bf16x8_to_f32(const uint4& raw, float* v) {
  const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    v[2 * i] = __uint_as_float(w[i] << 16);
    v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
  }
}

// 2^(127-u) for u in [0, 254] (u = 254 needs the subnormal 2^-127).
__device__ __forceinline__ float mx_inv_amplitude(uint32_t u) {
  return __uint_as_float(u == 254u ? 0x00400000u : ((254u - u) << 23));
}

constexpr int kMaxDevices = 64;      // per-device host-side caches are arrays of this length

int check_device_sm100();            // FP4ATTN_OK or FP4ATTN_ERR_UNSUPPORTED_ARCH / _CUDA

}  // namespace fp4attn
