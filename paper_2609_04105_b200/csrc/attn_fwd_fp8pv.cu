// FP8 P/V route of the attention forward (Section "Training stability selects FP8 P/V"): Q and K stay block-scaled
// FP4 and S = Q K^T is the same product as in attn_fwd.cu, but probabilities and V are single E4M3 bytes without
// block scales, P V is a `tcgen05.mma kind::f8f6f4` product, and the row reference is the row maximum itself.
//
//   mu_i  = ceil(max_j y_ij)                         (integer, known before any probability is formed)
//   p8_ij = Q_E4M3(2^(y_ij - mu_i + 8))              (<= 256; round to nearest even; below 2^-10 it is 0)
//   O_i   = sum_j p8_ij V8_j / (G_V sum_j p8_ij),   LSE_i = ln2 (mu_i - 8 + log2 sum_j p8_ij)
//
// Without block scales a probability cannot be re-scaled after it has been rounded, so it must be formed against the
// final reference.  An online running maximum would make the rounded values depend on the tile order (E4M3 flushes
// and loses mantissa bits at the bottom of its range) and would put a reduction over the softmax teams on every
// stage.  The tensor pipe is three quarters idle in this kernel family, so the reference is taken by a first sweep
// instead: every work item walks its keys TWICE - sweep A computes S and reduces the row maxima only, sweep B
// computes S again, forms the bytes against the now final mu and feeds PV.  Nothing is ever rescaled, there is no
// correction pass, and the result equals the plain (not online) definition above.  The second sweep of one item
// and the first sweep of the CTA's next item run interleaved stage by stage (see the schedule comment in the
// kernel), so that SFU-heavy and SFU-free visits alternate on every team.
//
//   warp 0        TMA producer: Q tile per item; ring of {K, K scales} for A-steps and {K, V8^T, K scales} for B-steps
//   warp 1        QK issuer (both kinds of step; after an A-step it also hands the ring slot back)
//   warp 2        PV issuer (B-steps): four K32 products per 128-key stage, A operand from tensor memory
//   warps 3-6     epilogue: O = O_hw / (L_hw G_V), LSE
//   warps 7-22    softmax teams as in attn_fwd.cu (team 2p + h: h-th 64 keys of the steps with parity p)
//
// The row sum is column d of the accumulator: sixteen rows of E4M3 1.0 follow V8^T in every stage.
// Tensor memory: S slots 0..255 | O 256..399 | Q scales 400..415 | K scales 416..431 | P bytes 432..495 (per step
// parity 32 columns: 128 keys x 8 bits per row).
#include "attn_common.cuh"

namespace fp4attn {
using namespace ptx;

constexpr uint32_t k8ColP = 432;
constexpr float kP8Shift = 8.0f;

template <int D, bool NV>
struct Cfg8 {
  using C1 = Cfg<D, NV>;
  static constexpr int V_BYTES = D * BS;                              // V8^T: d rows x 128 bytes
  static constexpr int ONES_BYTES = kOnesRows * BS;                   // rows of E4M3 1.0
  static constexpr int OFF_KSF = C1::K_BYTES + V_BYTES + ONES_BYTES;  // within a stage
  static constexpr int STAGE_BYTES = (OFF_KSF + C1::KSF_BYTES + 1023) / 1024 * 1024;
  static constexpr int NST = (D == 128) ? 5 : 8;
  static constexpr int OFF_Q = 0;                                     // two buffers
  static constexpr int OFF_QSF = OFF_Q + 2 * C1::Q_BYTES;             // two buffers of 1 KB
  static constexpr int OFF_RMAX = OFF_QSF + 2048;                     // [item parity][first-sweep team][row] float
  static constexpr int OFF_MU = OFF_RMAX + 2 * 4 * BM * 4;            // [item parity][row] int
  static constexpr int OFF_STAGE = (OFF_MU + 2 * BM * 4 + 1023) / 1024 * 1024;
  static constexpr int OFF_OUT = OFF_STAGE + NST * STAGE_BYTES;
  static constexpr int OFF_BAR = OFF_OUT + C1::OUT_BYTES;
  static constexpr int SMEM_BYTES = OFF_BAR + 1024 + 1024;
  static_assert(OFF_STAGE % 1024 == 0 && OFF_OUT % 1024 == 0 && SMEM_BYTES <= 227 * 1024, "shared memory");
};

enum { B8_QFULL0 = 0, B8_QFREE0 = 2, B8_OFULL = 4, B8_OFREE = 5, B8_SFULL0 = 6, B8_SEMPTY0 = 8, B8_PFREE0 = 10,
       B8_SMDONE0 = 12, B8_DRAIN0 = 14, B8_MURDY0 = 16, B8_RING = 18 };

struct Fp8Params {
  AttnParams a;
  const float* v_G;        // one decode divisor per K/V unit: V^ = V8 / v_G[unit]
};

// D[tmem] (+)= A[tmem] * B[smem], E4M3 x E4M3, K = 32, fp32 accumulate
__device__ __forceinline__ void tc_mma_f8_ta(uint32_t d, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// Instruction descriptor of kind::f8f6f4: 4-5 accumulator format (1 = F32) | 7-9 A format, 10-12 B format (0 = E4M3) |
// 15/16 A/B major (0 = K-major) | 17-22 N >> 3 | 24-28 M >> 4
__host__ __device__ constexpr uint32_t make_idesc_f8(int M, int N) {
  return 1u << 4 | (uint32_t)(N >> 3) << 17 | (uint32_t)(M >> 4) << 24;
}
__device__ __forceinline__ uint32_t cvt_e4m3x4_pos(float a, float b, float c, float d) {   // a in bits 0-7 ... d in bits 24-31
  uint32_t w;
  asm("{\n\t.reg .b16 lo, hi;\n\t"
      "cvt.rn.satfinite.e4m3x2.f32 lo, %2, %1;\n\t"
      "cvt.rn.satfinite.e4m3x2.f32 hi, %4, %3;\n\t"
      "mov.b32 %0, {lo, hi};\n\t}"
      : "=r"(w) : "f"(a), "f"(b), "f"(c), "f"(d));
  return w;
}

// 32 scores of one row -> 32 E4M3 bytes (8 words) against the row's final reference: x = fma(s, c, 8 - mu)
template <bool MASKED>
__device__ __forceinline__ void fp8_p_block(const uint32_t* sraw, float c32, float b, int visible, uint32_t* words) {
#pragma unroll
  for (int w = 0; w < 8; ++w) {
    float pv[4];
#pragma unroll
    for (int i = 0; i < 4; i += 2) {
      float x0, x1;
      fma2(__uint_as_float(sraw[4 * w + i]), __uint_as_float(sraw[4 * w + i + 1]), c32, b, x0, x1);
      pv[i] = ex2_approx(x0);
      pv[i + 1] = ex2_approx(x1);
      if (MASKED) {
        if (4 * w + i >= visible) pv[i] = 0.f;
        if (4 * w + i + 1 >= visible) pv[i + 1] = 0.f;
      }
    }
    words[w] = cvt_e4m3x4_pos(pv[0], pv[1], pv[2], pv[3]);
  }
}

template <int D, int NV, bool CAUSAL>
__global__ void __launch_bounds__(kAttnThreads, 1)
attn_fwd_fp8pv_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                      const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmO,
                      const Fp8Params pp) {
  const AttnParams& p = pp.a;
  using C = Cfg<D, (NV != 0)>;
  using C8 = Cfg8<D, (NV != 0)>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* sgen = smem_raw + (sbase - smem_u32(smem_raw));
  uint32_t* tslot = reinterpret_cast<uint32_t*>(sgen + C8::OFF_BAR + 768);
  volatile int* abortf = reinterpret_cast<volatile int*>(sgen + C8::OFF_BAR + 776);
  auto bar = [&](int i) { return sbase + C8::OFF_BAR + 8u * i; };
  auto bar_full = [&](int s) { return bar(B8_RING + s); };
  auto bar_empty = [&](int s) { return bar(B8_RING + C8::NST + s); };
  constexpr uint64_t kDescSF = (uint64_t)(16 >> 4) << 16 | (uint64_t)(128 >> 4) << 32 | 1ull << 46;
  constexpr uint64_t kDescQK = (uint64_t)(16 >> 4) << 16 | (uint64_t)((8 * C::ROW_BYTES) >> 4) << 32 | 1ull << 46 | C::SWZ_QK << 61;
  constexpr uint64_t kDescV = (uint64_t)(16 >> 4) << 16 | (uint64_t)(1024 >> 4) << 32 | 1ull << 46 | kSwz128 << 61;   // 128-byte rows
  auto at = [](uint64_t tmpl, uint32_t addr) { return tmpl | (uint64_t)((addr & 0x3FFFFu) >> 4); };

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int qtiles = p.N / BM;
  // this CTA's work items are item(k) = blockIdx.x + k * gridDim.x, k = 0 .. n_my - 1
  const int n_my = p.n_items > (int)blockIdx.x ? (p.n_items - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;
  auto item_of = [&](int k) { return (int)blockIdx.x + k * (int)gridDim.x; };

  if (threadIdx.x == 0) {
    for (int b = 0; b < 2; ++b) {
      mbar_init(bar(B8_QFULL0 + b), 1);
      mbar_init(bar(B8_QFREE0 + b), 1);
      mbar_init(bar(B8_SFULL0 + b), 1);
      mbar_init(bar(B8_SEMPTY0 + b), 8);       // the two teams of the pair, four warps each
      mbar_init(bar(B8_SMDONE0 + b), 8);
      mbar_init(bar(B8_PFREE0 + b), 1);
      mbar_init(bar(B8_MURDY0 + b), 4 * kTeams);   // every softmax warp, once per item (slot by item parity)
      mbar_init(bar(B8_DRAIN0 + b), 1);
    }
    mbar_init(bar(B8_OFULL), 1);
    mbar_init(bar(B8_OFREE), 4);
    for (int s = 0; s < C8::NST; ++s) { mbar_init(bar_full(s), 1); mbar_init(bar_empty(s), 1); }
    *abortf = 0;
    fence_barrier_init();
    prefetch_tensormap(&tmQ);
    prefetch_tensormap(&tmK);
    prefetch_tensormap(&tmV);
    prefetch_tensormap(&tmO);
  }
  if (warp == 1) { tmem_alloc(sbase + C8::OFF_BAR + 768, kTmemCols); tmem_relinquish(); }
  // constant operand rows: E4M3 1.0 (0x38) in every byte
  for (int i = threadIdx.x; i < C8::NST * (C8::ONES_BYTES / 4); i += kAttnThreads)
    reinterpret_cast<uint32_t*>(sgen + C8::OFF_STAGE + (i / (C8::ONES_BYTES / 4)) * C8::STAGE_BYTES + C::K_BYTES + C8::V_BYTES)[i % (C8::ONES_BYTES / 4)] = 0x38383838u;
  fence_proxy_async_smem();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tslot;

  // Every role walks the same schedule.  Phase ph (0 .. n_my) carries the first sweep ("A": scores -> row maxima) of
  // item ph and the second sweep ("B": scores -> bytes -> PV) of item ph - 1, stage by stage, in the order
  // A B | B A | A B | ... ; the first phase has no B part, the last no A part.  Steps are numbered g = 0, 1, 2 ... in
  // that order; step g uses score slot g & 1 and is served by the team pair g & 1 (teams 2p, 2p + 1), so each pair
  // alternates between the SFU-heavy second sweep of one item and the SFU-free first sweep of the next, and the four
  // warps of a scheduler are never all in the same kind of work.
  if (warp == 0) {
    // ===================================================================== TMA producer
    int s = 0, ph = 0;
    uint32_t gs = 0;
    uint32_t st = sbase + C8::OFF_STAGE;
    bool ok = true;
    for (int phs = 0; ok && phs <= n_my; ++phs) {
      WorkItem wa = {}, wb = {};
      int TA = 0, TB = 0;
      if (phs < n_my) { wa = decode_item<CAUSAL>(item_of(phs), p, qtiles); TA = wa.T2; }
      if (phs >= 1) { wb = decode_item<CAUSAL>(item_of(phs - 1), p, qtiles); TB = wb.T2; }
      if (phs < n_my) {
        const int qb = phs & 1;
        if (phs >= 2) ok = __all_sync(0xffffffffu, mbar_wait(bar(B8_QFREE0 + qb), ((phs >> 1) - 1) & 1, abortf));
        if (!ok) break;
        if (elect_one()) {
          mbar_arrive_expect_tx(bar(B8_QFULL0 + qb), C::Q_BYTES + C::QSF_BYTES);
          tma_load_2d(sbase + C8::OFF_Q + qb * C::Q_BYTES, &tmQ, 0, wa.qrow0, bar(B8_QFULL0 + qb));
          bulk_load_1d(sbase + C8::OFF_QSF + qb * 1024, p.q_sf + (size_t)wa.qtile_lin * C::QSF_BYTES, C::QSF_BYTES, bar(B8_QFULL0 + qb));
        }
      }
      const int TM = TA > TB ? TA : TB;
      for (int s2 = 0; ok && s2 < TM; ++s2) {
#pragma unroll
        for (int j = 0; j < 2; ++j) {
          const int kind = j ^ (s2 & 1);                            // 0: A-step of item phs, 1: B-step of item phs - 1
          if (s2 >= (kind ? TB : TA)) continue;
          const WorkItem& wi = kind ? wb : wa;
          if (gs >= (uint32_t)C8::NST) ok = __all_sync(0xffffffffu, mbar_wait(bar_empty(s), ph ^ 1, abortf));
          if (!ok) break;
          const uint32_t fb = bar_full(s);
          if (elect_one()) {
            mbar_arrive_expect_tx(fb, C::K_BYTES + C::KSF_BYTES + (kind ? C8::V_BYTES : 0));
            tma_load_2d(st, &tmK, 0, wi.kvh * p.N + s2 * BS, fb);
            if (kind) tma_load_2d(st + C::K_BYTES, &tmV, s2 * BS, wi.kvh * D, fb);
            bulk_load_1d(st + C8::OFF_KSF, p.k_sf + ((size_t)wi.kvh * qtiles + s2) * C::KSF_BYTES, C::KSF_BYTES, fb);
          }
          ++gs;
          st += C8::STAGE_BYTES;
          if (++s == C8::NST) { s = 0; ph ^= 1; st = sbase + C8::OFF_STAGE; }
        }
      }
    }
    if (*abortf && lane == 0) {
      for (int r = 0; r < C8::NST; ++r)
        for (int spin = 0; spin < (1 << 12) && !mbar_try_wait(bar_full(r), 0) && !mbar_try_wait(bar_full(r), 1); ++spin) {}
    }
    __syncwarp();
  } else if (warp == 1) {
    // ===================================================================== QK issuer (both sweeps)
    constexpr uint32_t kIdQK0 = NV ? make_idesc_fp4(BM, BS, false, 0, 0) : make_idesc_fp4(BM, BS, true, 0, 0);
    constexpr uint32_t kIdQK1 = NV ? make_idesc_fp4(BM, BS, false, 0, 0) : make_idesc_fp4(BM, BS, true, 2, 2);
    int sq = 0, phq = 0;
    uint32_t stq = sbase + C8::OFF_STAGE;
    uint32_t g = 0;                                             // steps issued so far (both kinds, all items)
    bool ok = true;
    for (int phs = 0; ok && phs <= n_my; ++phs) {
      int TA = 0, TB = 0;
      if (phs < n_my) TA = decode_item<CAUSAL>(item_of(phs), p, qtiles).T2;
      if (phs >= 1) TB = decode_item<CAUSAL>(item_of(phs - 1), p, qtiles).T2;
      if (phs < n_my) {
        const int qb = phs & 1;
        ok = __all_sync(0xffffffffu, mbar_wait(bar(B8_QFULL0 + qb), (phs >> 1) & 1, abortf));
        if (!ok) break;
        tc_fence_after();
        if (elect_one()) {
#pragma unroll
          for (int a = 0; a < C::CTQ; ++a)
            tc_cp_32x128b_warpx4(tmem + kColSFQ + 8 * qb + 4 * a, at(kDescSF, sbase + C8::OFF_QSF + qb * 1024 + 512 * a));
        }
        __syncwarp();
      }
      const int TM = TA > TB ? TA : TB;
      for (int s2 = 0; ok && s2 < TM; ++s2) {
#pragma unroll
        for (int j = 0; j < 2; ++j) {
          const int kind = j ^ (s2 & 1);
          if (s2 >= (kind ? TB : TA)) continue;
          const int qb = (kind ? phs - 1 : phs) & 1;              // the Q buffer of the step's item
          const int pr = g & 1;
          const uint32_t m = g >> 1;
          ok = __all_sync(0xffffffffu, mbar_wait(bar_full(sq), phq, abortf));
          if (ok && m > 0) ok = __all_sync(0xffffffffu, mbar_wait(bar(B8_SEMPTY0 + pr), (m - 1) & 1, abortf));   // both teams have read the slot
          if (!ok) break;
          tc_fence_after();
          const uint32_t tSFQ = tmem + kColSFQ + 8 * qb;
          const uint32_t tSFK = tmem + kColSFK + 8 * pr;
          const uint32_t tS = tmem + kColS + BS * pr;
          const uint64_t dQ0 = at(kDescQK, sbase + C8::OFF_Q + qb * C::Q_BYTES);
          const uint64_t dK0 = at(kDescQK, stq);
          if (elect_one()) {
#pragma unroll
            for (int a = 0; a < C::CTQ; ++a) tc_cp_32x128b_warpx4(tSFK + 4 * a, at(kDescSF, stq + C8::OFF_KSF + 512 * a));
            if (NV) {
              tc_mma_fp4_4x(tS, dQ0, dK0, kIdQK0, tSFQ, tSFK, 0);
              if (C::KBLK == 2) tc_mma_fp4_4x(tS, dQ0 + 2, dK0 + 2, kIdQK1, tSFQ + 4, tSFK + 4, 1);
            } else {
              tc_mma_fp4_2x(tS, dQ0, dK0, kIdQK0, tSFQ, tSFK, 0);
              if (C::KBLK == 2) tc_mma_fp4_2x(tS, dQ0 + 2, dK0 + 2, kIdQK1, tSFQ, tSFK, 1);
            }
            tc_commit(bar(B8_SFULL0 + pr));
            if (kind == 0) tc_commit(bar_empty(sq));              // first sweep: nothing else reads the stage
            if (kind == 1 && s2 == TB - 1) tc_commit(bar(B8_QFREE0 + qb));   // the item's Q buffer may take the item after next
          }
          __syncwarp();
          ++g;
          stq += C8::STAGE_BYTES;
          if (++sq == C8::NST) { sq = 0; phq ^= 1; stq = sbase + C8::OFF_STAGE; }
        }
      }
    }
    if (*abortf && elect_one()) tc_commit(bar(B8_DRAIN0));
    __syncwarp();
  } else if (warp == 2) {
    // ===================================================================== PV issuer (B-steps)
    constexpr uint32_t kIdPV = make_idesc_f8(BM, C::DN);
    const uint32_t tO = tmem + kColO;
    uint32_t g = 0;                                             // steps so far (both kinds): ring slot and team pair of a step
    uint32_t nb[2] = {0, 0};                                    // B-steps served so far, per team pair
    bool ok = true;
    for (int phs = 0; ok && phs <= n_my; ++phs) {
      int TA = 0, TB = 0;
      if (phs < n_my) TA = decode_item<CAUSAL>(item_of(phs), p, qtiles).T2;
      if (phs >= 1) TB = decode_item<CAUSAL>(item_of(phs - 1), p, qtiles).T2;
      if (phs >= 2) ok = __all_sync(0xffffffffu, mbar_wait(bar(B8_OFREE), (phs - 2) & 1, abortf));   // epilogue of item phs - 2 has read O
      const int TM = TA > TB ? TA : TB;
      for (int s2 = 0; ok && s2 < TM; ++s2) {
#pragma unroll
        for (int j = 0; j < 2; ++j) {
          const int kind = j ^ (s2 & 1);
          if (s2 >= (kind ? TB : TA)) continue;
          if (kind == 0) { ++g; continue; }                       // an A-step: only its slot is counted
          const int pr = g & 1;
          ok = __all_sync(0xffffffffu, mbar_wait(bar(B8_SMDONE0 + pr), (pr ? nb[1] : nb[0]) & 1, abortf));   // bytes of both tiles are in tensor memory
          if (!ok) break;
          if (pr) ++nb[1]; else ++nb[0];
          tc_fence_after();
          const uint32_t sp = g % C8::NST;
          const uint32_t stp = sbase + C8::OFF_STAGE + sp * C8::STAGE_BYTES;
          const uint64_t dV = at(kDescV, stp + C::K_BYTES);
          if (elect_one()) {
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)                         // 32 keys per product: 8 columns of P, 32 bytes along V8^T's rows
              tc_mma_f8_ta(tO, tmem + k8ColP + 32 * pr + 8 * kk, dV + 2 * kk, kIdPV, (s2 > 0 || kk > 0) ? 1u : 0u);
            tc_commit(bar_empty(sp));
            tc_commit(bar(B8_PFREE0 + pr));
            if (s2 == TB - 1) tc_commit(bar(B8_OFULL));
          }
          __syncwarp();
          ++g;
        }
      }
    }
    if (*abortf && elect_one()) tc_commit(bar(B8_DRAIN0 + 1));
    __syncwarp();
  } else if (warp < kFirstSoftmaxWarp) {
    // ===================================================================== epilogue warps
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;
    const uint32_t tO = tmem + ((uint32_t)(quarter * 32) << 16) + kColO;
    bool ok = true;
    for (int k = 0; ok && k < n_my; ++k) {
      const WorkItem wi = decode_item<CAUSAL>(item_of(k), p, qtiles);
      ok = __all_sync(0xffffffffu, mbar_wait(bar(B8_OFULL), k & 1, abortf));
      if (!ok) break;
      tc_fence_after();
      const int mu = reinterpret_cast<const int*>(sgen + C8::OFF_MU)[(k & 1) * BM + row];   // written before any PV of the item
      float Lhw;
      {
        uint32_t r16[16];
        tmem_ld_32x32b_x16(tO + D, r16);
        tmem_wait_ld();
        Lhw = __uint_as_float(r16[0]);
      }
      const float inv = __frcp_rn(Lhw * __ldg(pp.v_G + wi.kvh));
      if (lane == 0) bulk_wait_read_all();
      __syncwarp();
#pragma unroll
      for (int c0 = 0; c0 < D; c0 += 16) {
        uint32_t o[16];
        tmem_ld_32x32b_x16(tO + c0, o);
        tmem_wait_ld();
        if (c0 + 16 == D) {                                     // last read of O
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar(B8_OFREE));
        }
        uint8_t* half = sgen + C8::OFF_OUT + (c0 >> 6) * (BM * 128) + row * 128;
#pragma unroll
        for (int c = 0; c < 16; c += 8) {
          uint32_t pk[4];
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const __nv_bfloat162 hh = __floats2bfloat162_rn(__uint_as_float(o[c + 2 * q]) * inv, __uint_as_float(o[c + 2 * q + 1]) * inv);
            pk[q] = *reinterpret_cast<const uint32_t*>(&hh);
          }
          const int chunk = ((c0 & 63) + c) >> 3;
          *reinterpret_cast<uint4*>(half + ((chunk ^ (row & 7)) << 4)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
        }
      }
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) {
#pragma unroll
        for (int hf = 0; hf < D / 64; ++hf)
          tma_store_2d(&tmO, hf * 128, wi.qrow0 + quarter * 32, sbase + C8::OFF_OUT + hf * (BM * 128) + quarter * 32 * 128);
        bulk_commit_group();
      }
      if (p.LSE) p.LSE[(size_t)wi.qrow0 + row] = 0.69314718055994531f * ((float)mu - kP8Shift + log2f(Lhw));
    }
  } else {
    // ===================================================================== softmax teams
    const int team = (warp - kFirstSoftmaxWarp) >> 2;
    const int pr = team >> 1;                                   // the steps with g & 1 == pr are this pair's
    const int h = team & 1;                                     // which 64 keys of a stage
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;
    const uint32_t tS = tmem + ((uint32_t)(quarter * 32) << 16) + kColS + BN * team;
    const uint32_t sfull = bar(B8_SFULL0 + pr), sempty = bar(B8_SEMPTY0 + pr);
    const uint32_t smdone = bar(B8_SMDONE0 + pr), pfree = bar(B8_PFREE0 + pr);
    const uint32_t tP = tmem + ((uint32_t)(quarter * 32) << 16) + k8ColP + 32 * pr + 16 * h;
    float c32;
    if (NV) c32 = __fdiv_rn(p.c_base, __fmul_rn(__ldg(p.q_G), __ldg(p.k_G)));
    else    c32 = __fdiv_rn(p.c_base, 36.0f);
    bool ok = true;
    uint32_t g = 0;                                             // steps so far (both kinds, all pairs)
    uint32_t nbt = 0;                                           // B-visits of this team so far
    // keys of the team's tile that this row sees in an item's last stage, the masked one (causal: keys 0..i of row
    // i = qt * 128 + row; padded sequence: keys 0..len-1; both: the fewer)
    auto tile_keys = [&](const WorkItem& w) {
      const int seen = p.causal ? min(w.len, w.qt * BM + row + 1) : w.len;
      return seen - (w.T2 - 1) * BS - 64 * h;
    };
    float b = 0.f;                                              // 8 - mu of the item in its second sweep
    for (int phs = 0; ok && phs <= n_my; ++phs) {
      WorkItem wa = {}, wb = {};
      int TA = 0, TB = 0;
      if (phs < n_my) { wa = decode_item<CAUSAL>(item_of(phs), p, qtiles); TA = wa.T2; }
      if (phs >= 1) { wb = decode_item<CAUSAL>(item_of(phs - 1), p, qtiles); TB = wb.T2; }
      const int va = CAUSAL ? tile_keys(wa) : 64, vb = CAUSAL ? tile_keys(wb) : 64;
      float smax = -INFINITY;                                   // this team's share of the maxima of item phs
      const int TM = TA > TB ? TA : TB;
      for (int s2 = 0; ok && s2 < TM; ++s2) {
#pragma unroll
        for (int j = 0; j < 2; ++j) {
          const int kind = j ^ (s2 & 1);
          if (s2 >= (kind ? TB : TA)) continue;
          if ((int)(g & 1) != pr) { ++g; continue; }              // the other pair's step
          ok = __all_sync(0xffffffffu, mbar_wait(sfull, (g >> 1) & 1, abortf));
          if (!ok) break;
          tc_fence_after();
          uint32_t sraw[32];
          if (kind == 0) {
            // ---- first sweep of item phs: maxima only
            const bool diag = CAUSAL && s2 == TA - 1;
            tmem_ld_32x32b_x32(tS, sraw);
            tmem_wait_ld();
            if (diag) {
#pragma unroll
              for (int e = 0; e < 32; ++e) sraw[e] = (e < va) ? sraw[e] : 0xFF800000u;
            }
            smax = fmaxf(smax, max32(sraw));
            tmem_ld_32x32b_x32(tS + 32, sraw);
            tmem_wait_ld();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(sempty);
            if (diag) {
#pragma unroll
              for (int e = 0; e < 32; ++e) sraw[e] = (e < va - 32) ? sraw[e] : 0xFF800000u;
            }
            smax = fmaxf(smax, max32(sraw));
          } else {
            // ---- second sweep of item phs - 1: bytes against its final reference
            uint32_t w[16];
            const bool diag = CAUSAL && s2 == TB - 1;
            tmem_ld_32x32b_x32(tS, sraw);
            tmem_wait_ld();
            if (diag) fp8_p_block<true>(sraw, c32, b, vb, w);
            else      fp8_p_block<false>(sraw, c32, b, 32, w);
            tmem_ld_32x32b_x32(tS + 32, sraw);
            tmem_wait_ld();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(sempty);
            if (diag) fp8_p_block<true>(sraw, c32, b, vb - 32, w + 8);
            else      fp8_p_block<false>(sraw, c32, b, 32, w + 8);
            // the pair's probability slot was last read by the PV product of this team's previous B-visit
            if (nbt > 0) ok = __all_sync(0xffffffffu, mbar_wait(pfree, (nbt - 1) & 1, abortf));
            if (!ok) break;
            tmem_st_32x32b_x16(tP, w);
            tmem_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smdone);
            ++nbt;
          }
          ++g;
        }
      }
      if (!ok) break;
      if (phs < n_my) {
        // ---- the sixteen softmax warps meet: mu of item phs = ceil(c * max over all its keys), on the FMA pipe
        float* rmax = reinterpret_cast<float*>(sgen + C8::OFF_RMAX) + (phs & 1) * 4 * BM;
        rmax[team * BM + row] = smax;                           // (-inf from a team that served none of the item's A-steps)
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(B8_MURDY0 + (phs & 1)));
        ok = __all_sync(0xffffffffu, mbar_wait(bar(B8_MURDY0 + (phs & 1)), (phs >> 1) & 1, abortf));
        if (!ok) break;
        const float mall = fmaxf(fmaxf(rmax[row], rmax[BM + row]), fmaxf(rmax[2 * BM + row], rmax[3 * BM + row]));
        const float ymax = fminf(fmaxf(__fmul_rn(mall, c32), -2097152.0f), 2097152.0f);
        const float tt = __fadd_ru(ymax, 12582912.0f);          // ceil, exact for |y| < 2^22
        b = __fsub_rn(kP8Shift, __fsub_rn(tt, 12582912.0f));
        if (team == 0) reinterpret_cast<int*>(sgen + C8::OFF_MU)[(phs & 1) * BM + row] = (int)(__float_as_uint(tt) - 0x4B400000u);
      }
    }
  }
  if (warp >= 3 && warp < kFirstSoftmaxWarp && lane == 0) bulk_wait_all();
  __syncthreads();
  if (*abortf && threadIdx.x == 0 && p.status) *p.status = FP4ATTN_ERR_TIMEOUT;
  if (warp == 1) {
    if (*abortf && lane == 0) {
      for (int r = 0; r < 2; ++r)
        for (int spin = 0; spin < (1 << 14) && !mbar_try_wait(bar(B8_DRAIN0 + r), 0); ++spin) {}
    }
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem, kTmemCols);
  }
}

template <int D, int NV, bool CAUSAL>
static int launch_fp8(const fp4attn_operands* ops, int B, int H, int N, const Fp8Params& prm, cudaStream_t st) {
  using C8 = Cfg8<D, (NV != 0)>;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return FP4ATTN_ERR_CUDA;
  static std::atomic<bool> attr_set[kMaxDevices];
  if (dev < 0 || dev >= kMaxDevices) return FP4ATTN_ERR_CUDA;
  if (!attr_set[dev].load(std::memory_order_acquire)) {
    if (cudaFuncSetAttribute(attn_fwd_fp8pv_kernel<D, NV, CAUSAL>, cudaFuncAttributeMaxDynamicSharedMemorySize, C8::SMEM_BYTES) != cudaSuccess)
      return FP4ATTN_ERR_CUDA;
    attr_set[dev].store(true, std::memory_order_release);
  }
  const CUtensorMap* tm = attention_tensor_maps_fp8v(D, ops, prm.a.O, B, H, prm.a.Hkv, N);
  if (!tm) return FP4ATTN_ERR_CUDA;
  const unsigned grid = (unsigned)(prm.a.n_items < sms ? prm.a.n_items : sms);
  attn_fwd_fp8pv_kernel<D, NV, CAUSAL><<<grid, kAttnThreads, C8::SMEM_BYTES, st>>>(tm[0], tm[1], tm[2], tm[3], prm);
  return cudaGetLastError() == cudaSuccess ? FP4ATTN_OK : FP4ATTN_ERR_CUDA;
}

// Entry used by fp4attn_fwd for pv_fmt = FP4ATTN_PV_E4M3; `prm` is filled as for the one-query FP4 kernel.
int launch_attn_fp8pv(const fp4attn_operands* ops, int B, int H, int N, int d, AttnParams prm, cudaStream_t st) {
  if (!ops->v_G) return FP4ATTN_ERR_INVALID_ARG;
  if (ops->p_map != FP4ATTN_PMAP_IDEAL || ops->p_scale_rule != FP4ATTN_PSCALE_CEIL || ops->g_per_head ||
      ops->schedule != FP4ATTN_SCHEDULE_ONE_QUERY)
    return FP4ATTN_ERR_INVALID_ARG;                               // the code maps and block rules belong to the FP4 probability path
  Fp8Params pp{prm, ops->v_G};
  const bool nv = ops->qk_fmt == FP4ATTN_FMT_NVFP4;
  const int sel = (d == 128 ? 4 : 0) | (nv ? 2 : 0) | ((prm.causal || prm.seq_len) ? 1 : 0);   // masked instances
  switch (sel) {
    case 0: return launch_fp8<64, 0, false>(ops, B, H, N, pp, st);
    case 1: return launch_fp8<64, 0, true>(ops, B, H, N, pp, st);
    case 2: return launch_fp8<64, 1, false>(ops, B, H, N, pp, st);
    case 3: return launch_fp8<64, 1, true>(ops, B, H, N, pp, st);
    case 4: return launch_fp8<128, 0, false>(ops, B, H, N, pp, st);
    case 5: return launch_fp8<128, 0, true>(ops, B, H, N, pp, st);
    case 6: return launch_fp8<128, 1, false>(ops, B, H, N, pp, st);
    default: return launch_fp8<128, 1, true>(ops, B, H, N, pp, st);
  }
}

}  // namespace fp4attn
