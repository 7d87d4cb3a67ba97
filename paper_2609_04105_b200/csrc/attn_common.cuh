// Pieces shared by the attention kernels (one query tile per CTA, and two query tiles per CTA): tile sizes, the
// tensor-memory and shared-memory maps, work-item decoding, and the per-block score -> code arithmetic of
// Algorithm "direct-p-pack".
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "ptx.cuh"

namespace fp4attn {
using namespace ptx;

constexpr int BM = 128;          // query rows per work item
constexpr int BN = 64;           // keys per score tile (two N32 probability blocks)
constexpr int BS = 128;          // keys per stage
constexpr int kTeams = 4;        // score slots / softmax teams
constexpr int kFirstSoftmaxWarp = 7;     // warps 3..6 are the correction warps
constexpr int kAttnThreads = 32 * (kFirstSoftmaxWarp + 4 * kTeams);
constexpr int kLazyShift = 64;   // the row reference is raised only when a block exponent exceeds it by more
                                 // than this many octaves (rescales are exact powers of 2) ...
constexpr int kRefHeadroom = 60; // ... and is then set this far ABOVE that exponent, so that a later raise
                                 // needs a jump of 124 octaves: E8M0 bytes stay within 1..191, blocks weaker
                                 // than 2^-66 of the row maximum become zero blocks
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kColS = 0, kColO = 256, kColSFQ = 400, kColSFK = 416, kColSFV = 432, kColSFP = 448,
                   kColP = 456;      // P codes: [stage parity][tile] x 8 columns (64 keys x 4 bits per row)
constexpr int kOnesRows = 16;    // rows of ones appended to V^T (the MMA's N must be a multiple of 16)

template <int D, bool NV>
struct Cfg {
  static constexpr int ROW_BYTES = D / 2;                       // packed bytes of one Q/K row
  static constexpr int KBLK = D / 64;                           // K64 instructions per QK stage
  static constexpr int CTQ = NV ? (D / 16 + 3) / 4 : 1;         // scale atoms per 128 rows of Q or K
  static constexpr int Q_BYTES = BM * ROW_BYTES;
  static constexpr int QSF_BYTES = CTQ * 512;
  static constexpr int K_BYTES = BS * ROW_BYTES;                // 128 keys
  static constexpr int V_BYTES = D * (BS / 2);                  // V^T: d rows x 64 bytes
  static constexpr int ONES_BYTES = kOnesRows * (BS / 2);       // constant rows of E2M1 1.0, written once
  static constexpr int DN = D + kOnesRows;                      // N of the PV instruction
  static constexpr int KSF_BYTES = CTQ * 512;
  static constexpr int VSF_BYTES = 512;
  static constexpr int OFF_KSF = K_BYTES + V_BYTES + ONES_BYTES;   // within a stage
  static constexpr int OFF_VSF = OFF_KSF + KSF_BYTES;
  static constexpr int STAGE_BYTES = OFF_VSF + VSF_BYTES;
  static constexpr int NST = (D == 128) ? 7 : 8;                // ring depth (stages of 128 keys)
  static constexpr int PSF_BYTES = 512;                         // one atom per stage: bytes {0,1} tile 0, {2,3} tile 1
  static constexpr int META_BYTES = BM * 16;                    // per stage parity and row: {E_0, E_1} of tile 0, of tile 1
  // shared-memory map (offsets from a 1024-byte aligned base)
  static constexpr int OFF_Q = 0;                               // two buffers
  static constexpr int OFF_QSF = OFF_Q + 2 * Q_BYTES;           // two buffers of 1 KB
  static constexpr int OFF_PSF = OFF_QSF + 2048;
  static constexpr int OFF_ONESF = OFF_PSF + 2 * PSF_BYTES;     // scale atom of 1.0 for the rows of ones
  static constexpr int OFF_META = OFF_ONESF + 512;
  static constexpr int OFF_STAGE = (OFF_META + 2 * META_BYTES + 1023) / 1024 * 1024;
  static constexpr int OFF_OUT = (OFF_STAGE + NST * STAGE_BYTES + 1023) / 1024 * 1024; // bf16 O tile staged for TMA stores: D/64 halves of [128 rows][128 B]
  static constexpr int OUT_BYTES = (D / 64) * BM * 128;
  static constexpr int OFF_BAR = OFF_OUT + OUT_BYTES;
  static constexpr int SMEM_BYTES = OFF_BAR + 1024 + 1024;      // barriers + alignment slack
  static constexpr uint64_t SWZ_QK = (ROW_BYTES == 64) ? kSwz64 : kSwz32;
  static_assert(STAGE_BYTES % 512 == 0 && OFF_STAGE % 1024 == 0 && OFF_OUT % 1024 == 0, "stage alignment");
  static_assert(SMEM_BYTES <= 227 * 1024, "shared memory");
};

struct AttnParams {
  const uint8_t *q_sf, *k_sf, *v_sf;
  const float *q_G, *k_G;
  __nv_bfloat16* O;
  float* LSE;
  int* status;
  int N, stages;           // keys, N / 128
  int n_items;             // B * H * N / 128
  float c_base;            // fl32(log2(e) * softmax_scale)
  float aff_a, aff_b;      // affine classifier u = max(0, A x + B) (only read by the affine variant)
  int thr16;               // block exponent rule: 0 = ceil(max y), 1 = floor(max y + log2 1.6)
  int causal;              // 1: query row i sees keys 0..i
  int H, Hkv;              // query heads, K/V heads (H % Hkv == 0: grouped-query attention)
  int BH;                  // B * H
  unsigned long long recip_qtiles, recip_bh;   // ceil(2^64 / (N / 128)), ceil(2^64 / BH); 0 for a divisor of 1
  int ref_fixed;           // the constant row reference of the FIXREF instances (octaves)
  const int* seq_len;      // NULL, or B token counts: batch entry b is seq_len[b] tokens padded to N (masked kernels only)
  unsigned long long recip_h;                  // ceil(2^64 / H); 0 for H = 1
};

// One work item = one 128-row query tile of one (batch, query head).
struct WorkItem {
  int qt;                  // query tile within the head
  int qrow0;               // first row of the tile in the [B*H*N] row space of Q, O, LSE
  int qtile_lin;           // (b*H + h) * qtiles + qt: index of the tile's Q scale atom(s)
  int kvh;                 // b*Hkv + h / (H/Hkv): the K/V head this query head reads
  int bh;                  // b*H + h
  int T2;                  // 128-key stages to walk (causal: up to and including the diagonal; padded: those with a key)
  int len;                 // keys that exist for this unit (N unless the batch entry is a padded sequence)
};
// floor(n / d) for n < 2^31 through the precomputed reciprocal ceil(2^64 / d) (0 stands for d = 1): the
// roles decode a work item on their critical path, and a 32-bit division costs some fifty instructions
__device__ __forceinline__ int fast_div(int n, unsigned long long recip) {
  return recip ? (int)__umul64hi((unsigned long long)n, recip) : n;
}
// MASKED: the kernels that mask the last stage of an item - the causal mask (p.causal), padded sequences
// (p.seq_len), or both.  The unmasked kernels ignore both fields.
template <bool MASKED>
__device__ __forceinline__ WorkItem decode_item(int item, const AttnParams& p, int qtiles) {
  constexpr bool CAUSAL = MASKED;
  WorkItem w;
  int bh;
  if (CAUSAL) {             // longest items first, so the persistent CTAs finish together
    const int r = fast_div(item, p.recip_bh);
    w.qt = qtiles - 1 - r;
    bh = item - r * p.BH;
  } else {                  // consecutive items share K/V in L2
    bh = fast_div(item, p.recip_qtiles);
    w.qt = item - bh * qtiles;
  }
  w.qrow0 = bh * p.N + w.qt * BM;
  w.qtile_lin = bh * qtiles + w.qt;
  w.kvh = bh;
  w.bh = bh;
  if (p.H != p.Hkv) {       // grouped-query attention
    const int b = bh / p.H, h = bh - b * p.H;
    w.kvh = b * p.Hkv + h / (p.H / p.Hkv);
  }
  w.len = p.N;
  w.T2 = p.stages;
  if (MASKED) {
    if (p.seq_len) {
      const int len = __ldg(p.seq_len + fast_div(bh, p.recip_h));
      w.len = len < 1 ? 1 : (len > p.N ? p.N : len);
      w.T2 = w.qt * BM < w.len ? (w.len + BS - 1) / BS : 1;   // a query tile beyond the length: one stage, results unused
    }
    if (p.causal && w.qt + 1 < w.T2) w.T2 = w.qt + 1;
  }
  return w;
}

// barrier slots (8 bytes each)
enum { BAR_QFULL0 = 0, BAR_QFREE0 = 2, BAR_OFULL = 4, BAR_OFREE = 5, BAR_SFULL0 = 6, BAR_SEMPTY0 = 8,
       BAR_PFULL0 = 10, BAR_PFREE0 = 12, BAR_SMDONE0 = 14, BAR_DRAIN0 = 16, BAR_RING = 18 };

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
// maximum of 32 floats held as raw bits, as a depth-4 tree of 3-input maxima
__device__ __forceinline__ float max32(const uint32_t* r) {
  float t[12];
#pragma unroll
  for (int k = 0; k < 10; ++k)
    t[k] = max3(__uint_as_float(r[3 * k]), __uint_as_float(r[3 * k + 1]), __uint_as_float(r[3 * k + 2]));
  t[10] = __uint_as_float(r[30]);
  t[11] = __uint_as_float(r[31]);
  const float a = max3(t[0], t[1], t[2]), b = max3(t[3], t[4], t[5]), c = max3(t[6], t[7], t[8]), d = max3(t[9], t[10], t[11]);
  return fmaxf(max3(a, b, c), d);
}
// two fused multiply-adds in one instruction: {x0, x1} = {s0, s1} * {c, c} + {b, b}
__device__ __forceinline__ void fma2(float s0, float s1, float c, float b, float& x0, float& x1) {
  asm("{\n\t.reg .b64 s, cc, bb, d;\n\t"
      "mov.b64 s, {%2, %3};\n\tmov.b64 cc, {%4, %4};\n\tmov.b64 bb, {%5, %5};\n\t"
      "fma.rn.f32x2 d, s, cc, bb;\n\t"
      "mov.b64 {%0, %1}, d;\n\t}"
      : "=f"(x0), "=f"(x1) : "f"(s0), "f"(s1), "f"(c), "f"(b));
}
// ---- 2^x on the FMA pipe for a share of the elements (the SFU's 16 ex2/clk/SM is the tightest unit).
// Only the E2M1 code of 2^x matters, and it changes only where 2^x crosses 0.25, 0.75, 1.25, 1.75, 2.5,
// 3.5 or 5.  2^x is therefore replaced by the degree-6 polynomial through the seven points (log2 b, b):
// equal to 2^x at every point where a code can change and monotone on [-2.75, 3.3], so the codes are
// those of the exact exponential (a 4-million-point sweep plus dense sweeps around the seven boundaries
// differ only within three fp32 ulps of x at a boundary - the same class as ex2.approx).  No range
// reduction: x is at most log2(9.6) by construction of the block exponent, and below -2.75 it is clamped
// (there the polynomial stays inside (0.18, 0.25), i.e. code 0 like 2^x).
#ifndef FP4ATTN_POLY_MASK
#define FP4ATTN_POLY_MASK 0x8421u      // which of a block's 16 element pairs take the polynomial path
#endif
// The header states which pairs take which evaluation (fp4attn.h, FP4ATTN_PMAP_IDEAL); a build with another
// pattern would change codes within rounding distance of a boundary, so it has to change that text as well.
static_assert(FP4ATTN_POLY_MASK == 0x8421u, "the pattern of polynomial pairs is part of the documented behaviour");
__device__ __forceinline__ uint64_t pack2(float a, float b) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
  return r;
}
__device__ __forceinline__ void exp2_poly6(float x0, float x1, float& p0, float& p1) {
  const uint64_t x = pack2(fmaxf(x0, -2.75f), fmaxf(x1, -2.75f));
  uint64_t q;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(q) : "l"(pack2(0.0002452842309139669f, 0.0002452842309139669f)), "l"(x),
      "l"(pack2(0.0012840019771829247f, 0.0012840019771829247f)));
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(q) : "l"(q), "l"(x), "l"(pack2(0.009303540922701359f, 0.009303540922701359f)));
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(q) : "l"(q), "l"(x), "l"(pack2(0.05597471818327904f, 0.05597471818327904f)));
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(q) : "l"(q), "l"(x), "l"(pack2(0.2401072233915329f, 0.2401072233915329f)));
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(q) : "l"(q), "l"(x), "l"(pack2(0.6930626630783081f, 0.6930626630783081f)));
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(q) : "l"(q), "l"(x), "l"(pack2(1.0000272989273071f, 1.0000272989273071f)));
  asm("mov.b64 {%0, %1}, %2;" : "=f"(p0), "=f"(p1) : "l"(q));
}

// One N32 score fragment of one row: E_B = ceil(max y) and the codes.  Nothing here depends on the
// row reference.
//   ideal map  (Eq. "ideal-code-path"):  q = Q_E2M1(2^x),            x = y - E_B + log2 6
//   affine map (Eq. "affine-code-map"):  q = Q_E2M1(max(0, A x + B)), folded into one fused multiply-add
//                                        per element: u = s * fl32(A c) + fma(A, log2 6 - E_B, B)
// PMAP: 0 ideal map for every element, 1 affine map for every element, 2..4 mixed (the EX2-density control
// of Appendix "SM103 launch and EX2 controls"): element pair k of the block takes the ideal map where bit
// k of the pattern is set, the affine map elsewhere.
__host__ __device__ constexpr uint32_t exact_pairs_of(int pmap) {
  return pmap == 0 ? 0xFFFFu : pmap == 1 ? 0x0000u : pmap == 2 ? 0x1111u : pmap == 3 ? 0x5555u : 0x7777u;
}
// RULE: block exponent from the block maximum - 0 ceiling, 1 threshold rule, 2 the better of ceiling and ceiling - 1 by
// squared error of the 32 represented values (ideal map only; see direct_p_block_mse)
template <bool MASKED>
__device__ __forceinline__ void direct_p_block_mse(uint32_t* sraw, float c32, int visible, int& E, uint32_t* words);

template <int PMAP, bool MASKED, int RULE>
__device__ __forceinline__ void direct_p_block(uint32_t* sraw, float c32, float A, float B, int visible, int& E,
                                               uint32_t* words) {
  if (RULE == 2) { direct_p_block_mse<MASKED>(sraw, c32, visible, E, words); return; }
  constexpr bool THR16 = RULE == 1;
  constexpr uint32_t kExact = exact_pairs_of(PMAP);
  const float LOG2_6 = 2.5849625007211560f;
  if (MASKED) {                                                 // keys the row does not see (causal mask, padding) get -inf
#pragma unroll
    for (int i = 0; i < 32; ++i) sraw[i] = (i < visible) ? sraw[i] : 0xFF800000u;
  }
  // y is clamped to +-2^21 (scores beyond that are outside any softmax's range; a fully masked block,
  // max = -inf, lands on the lower clamp and becomes a zero block)
  const float ymax = fminf(fmaxf(__fmul_rn(max32(sraw), c32), -2097152.0f), 2097152.0f);
  // amplitude rule (Eq. "mx-scale" allows either neighbouring power of two): ceiling, or the threshold
  // rule alpha = 2^floor(log2(1.6 a)) under which values above the amplitude saturate at code 6.
  // Integer rounding on the FMA pipe (the conversion instructions share the SFU's issue slots with
  // ex2): for |y| < 2^22, y + 1.5*2^23 rounded up (down) is ceil(y) (floor(y)) + 1.5*2^23 exactly.
  const float M = 12582912.0f;
  const float t = THR16 ? __fadd_rd(__fadd_rn(ymax, 0.6780719161033630f), M) : __fadd_ru(ymax, M);
  E = (int)(__float_as_uint(t) - 0x4B400000u);
  const float bB = __fsub_rn(LOG2_6, __fsub_rn(t, M));          // t - M = (float)E, exact
  const float cA = __fmul_rn(A, c32), bA = __fmaf_rn(A, bB, B);  // affine pairs only
#pragma unroll
  for (int w = 0; w < 4; ++w) {
    float pv[8];
#pragma unroll
    for (int i = 0; i < 8; i += 2) {
      const int pair = 4 * w + i / 2;
      if ((kExact >> pair) & 1u) {
        float x0, x1;
        fma2(__uint_as_float(sraw[8 * w + i]), __uint_as_float(sraw[8 * w + i + 1]), c32, bB, x0, x1);
        if ((FP4ATTN_POLY_MASK >> pair) & 1u) {
          exp2_poly6(x0, x1, pv[i], pv[i + 1]);
        } else {
          pv[i] = ex2_approx(x0);
          pv[i + 1] = ex2_approx(x1);
        }
      } else {
        fma2(__uint_as_float(sraw[8 * w + i]), __uint_as_float(sraw[8 * w + i + 1]), cA, bA, pv[i], pv[i + 1]);
      }
    }
    // the conversion clamps negative inputs to +0 (affine pairs; exact pairs are positive anyway)
    words[w] = kExact == 0xFFFFu ? cvt_e2m1x8(pv) : cvt_e2m1x8_relu(pv);
  }
}

// Eq. "mx-scale" names both powers of two next to a block maximum.  Here every block takes, of E_c = ceil(max y) and
// E_c - 1, the one with the smaller squared error of its 32 represented probabilities.  Under E_c the code units are
// v = 6 * 2^(y - E_c) (every v through ex2.approx: the boundary polynomial is exact only where codes change); under
// E_c - 1 they are 2v, saturating at 6, in units half as large: the floor wins iff
//   sum (2v - q(2v))^2 < 4 sum (v - q(v))^2      (strictly; a block whose maximum is an integer has one candidate).
// Error sums in fp32: eight consecutive keys left to right, the four group sums as (g0 + g1) + (g2 + g3).
template <bool MASKED>
__device__ __forceinline__ void direct_p_block_mse(uint32_t* sraw, float c32, int visible, int& E, uint32_t* words) {
  const float LOG2_6 = 2.5849625007211560f;
  if (MASKED) {
#pragma unroll
    for (int i = 0; i < 32; ++i) sraw[i] = (i < visible) ? sraw[i] : 0xFF800000u;
  }
  const float ymax = fminf(fmaxf(__fmul_rn(max32(sraw), c32), -2097152.0f), 2097152.0f);
  const float M = 12582912.0f;
  const float t = __fadd_ru(ymax, M);
  const float Ec = __fsub_rn(t, M);                              // ceil(ymax), exact
  const float bB = __fsub_rn(LOG2_6, Ec);
  float gc[4], gf[4];
  uint32_t wc[4], wf[4];
#pragma unroll
  for (int w = 0; w < 4; ++w) {
    float v[8], v2[8];
#pragma unroll
    for (int i = 0; i < 8; i += 2) {
      float x0, x1;
      fma2(__uint_as_float(sraw[8 * w + i]), __uint_as_float(sraw[8 * w + i + 1]), c32, bB, x0, x1);
      v[i] = ex2_approx(x0);
      v[i + 1] = ex2_approx(x1);
      v2[i] = __fmul_rn(2.0f, v[i]);
      v2[i + 1] = __fmul_rn(2.0f, v[i + 1]);
    }
    wc[w] = cvt_e2m1x8(v);
    wf[w] = cvt_e2m1x8(v2);                                      // saturates at 6
    gc[w] = mx_error_x8(v, wc[w]);
    gf[w] = mx_error_x8(v2, wf[w]);
  }
  const float ec = __fadd_rn(__fadd_rn(gc[0], gc[1]), __fadd_rn(gc[2], gc[3]));
  const float ef = __fadd_rn(__fadd_rn(gf[0], gf[1]), __fadd_rn(gf[2], gf[3]));
  const bool take_f = (ymax != Ec) && (ef < __fmul_rn(4.0f, ec));
  E = (int)(__float_as_uint(t) - 0x4B400000u) - (take_f ? 1 : 0);
#pragma unroll
  for (int w = 0; w < 4; ++w) words[w] = take_f ? wf[w] : wc[w];
}

// Tensor maps of a launch (Q, K, V^T, O in that order) from the calling thread's cache; nullptr if the driver
// refuses to encode one.  Defined beside the one-query kernel.
const CUtensorMap* attention_tensor_maps(int D, const fp4attn_operands* ops, void* O, int B, int H, int Hkv, int N);
// The same with V^T held as E4M3 bytes [B, Hkv, d, N] (box: 128 keys x d rows, 128-byte swizzle).
const CUtensorMap* attention_tensor_maps_fp8v(int D, const fp4attn_operands* ops, void* O, int B, int H, int Hkv, int N);

}  // namespace fp4attn
