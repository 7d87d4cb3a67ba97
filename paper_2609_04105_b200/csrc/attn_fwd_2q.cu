// Two-query schedule of the Direct-P attention forward (Section "Two-query execution model"): one CTA owns TWO
// 128-row query tiles of the same (batch, head) and walks the keys once for both, so every K / V^T stage that
// TMA brings into shared memory feeds two score products and two PV products, and the SM carries two
// independent score -> code -> PV chains, one per query tile, each with its own accumulator.
//
// Tensor memory decides where this schedule exists.  Two accumulators of d + 16 columns (the sixteen extra
// columns hold the represented row sum, see attn_fwd.cu) need 288 of the 512 columns at d = 128; together with
// the 256 score columns that hide the latency of the QK product (two 64-key slots per chain) that is already
// more than an SM has, before any scale page or probability slot.  The paper's own layout fits at d = 128 only
// by giving up the separate columns: probability codes and every scale page are overlaid on retired score
// columns (Eq. "score-overlay") and the row sum is taken in the softmax threads.  At d = 64 the accumulators
// take 160 columns and everything fits side by side, so this file provides the schedule for d = 64:
//
//   S  0..255 (query q: columns 128q.., two 64-key slots) | O  256 + 80q (q = 0, 1) | Q scales 416..431 (item
//   parity x query, 4 columns each) | K scales 432..439 (stage parity) | V scales 440..447 (stage parity) |
//   P scales 448 + 4q | P codes 456 + 16q + 8h
//
// Roles are those of the one-query kernel; what was indexed by the parity of the stage there is indexed by the
// query here: softmax team 2q + h serves the h-th 64 keys of EVERY stage for query q, the correction warps keep
// one integer row reference per query (two rows per thread), and the issuers run q = 0, 1 inside every stage.
// The K / V^T ring advances once per stage, i.e. once per two score tiles.
#include "attn_common.cuh"

namespace fp4attn {
using namespace ptx;

constexpr uint32_t k2ColO = 256, k2ColSFQ = 416, k2ColSFK = 432, k2ColSFV = 440, k2ColSFP = 448, k2ColP = 456;
constexpr int k2OCols = 64 + kOnesRows;          // accumulator columns per query

template <bool NV>
struct Cfg2 {
  using C1 = Cfg<64, NV>;
  static constexpr int OFF_Q = 0;                                      // four buffers: item parity x query
  static constexpr int OFF_QSF = OFF_Q + 4 * C1::Q_BYTES;              // four buffers of 1 KB
  static constexpr int OFF_PSF = OFF_QSF + 4096;                       // one atom per query
  static constexpr int OFF_META = OFF_PSF + 2 * C1::PSF_BYTES;         // per query and row: {E_0, E_1} of tile 0, of tile 1
  static constexpr int OFF_STAGE = (OFF_META + 2 * C1::META_BYTES + 1023) / 1024 * 1024;
  static constexpr int OFF_OUT = (OFF_STAGE + C1::NST * C1::STAGE_BYTES + 1023) / 1024 * 1024;   // one bf16 tile [128][128 B]
  static constexpr int OFF_BAR = OFF_OUT + C1::OUT_BYTES;
  static constexpr int SMEM_BYTES = OFF_BAR + 1024 + 1024;
  static_assert(OFF_STAGE % 1024 == 0 && OFF_OUT % 1024 == 0 && SMEM_BYTES <= 227 * 1024, "shared memory");
};

enum { B2_QFULL0 = 0, B2_QFREE0 = 2, B2_OFULL0 = 4, B2_OFREE0 = 6, B2_SFULL0 = 8, B2_SEMPTY0 = 10, B2_PFULL0 = 12,
       B2_PFREE0 = 14, B2_SMDONE0 = 16, B2_DRAIN0 = 18, B2_RING = 20 };

struct WorkItem2 {
  int qrow0;               // first row of query tile 0 (tile 1 follows) in the [B*H*N] row space
  int qtile_lin;           // index of tile 0's Q scale atom
  int kvh;                 // K/V head
};
__device__ __forceinline__ WorkItem2 decode_item2(int item, const AttnParams& p, int pairs) {
  WorkItem2 w;
  const int bh = fast_div(item, p.recip_qtiles);               // here the reciprocal of the number of tile pairs
  const int pair = item - bh * pairs;
  w.qrow0 = bh * p.N + pair * (2 * BM);
  w.qtile_lin = bh * (2 * pairs) + 2 * pair;
  w.kvh = bh;
  if (p.H != p.Hkv) {
    const int b = bh / p.H, h = bh - b * p.H;
    w.kvh = b * p.Hkv + h / (p.H / p.Hkv);
  }
  return w;
}

// NV: 0 - MXFP4 Q, K; 1 - NVFP4 with one encode factor per tensor
template <int NV, int PMAP, bool THR16>
__global__ void __launch_bounds__(kAttnThreads, 1)
attn_fwd_2q_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                   const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmO,
                   const AttnParams p) {
  constexpr int D = 64;
  using C = Cfg<64, (NV != 0)>;
  using C2 = Cfg2<(NV != 0)>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* sgen = smem_raw + (sbase - smem_u32(smem_raw));
  uint32_t* tslot = reinterpret_cast<uint32_t*>(sgen + C2::OFF_BAR + 768);
  volatile int* abortf = reinterpret_cast<volatile int*>(sgen + C2::OFF_BAR + 776);
  auto bar = [&](int i) { return sbase + C2::OFF_BAR + 8u * i; };
  auto bar_full = [&](int s) { return bar(B2_RING + s); };
  auto bar_empty = [&](int s) { return bar(B2_RING + C::NST + s); };
  constexpr uint64_t kDescSF = (uint64_t)(16 >> 4) << 16 | (uint64_t)(128 >> 4) << 32 | 1ull << 46;
  constexpr uint64_t kDescQK = (uint64_t)(16 >> 4) << 16 | (uint64_t)((8 * C::ROW_BYTES) >> 4) << 32 | 1ull << 46 | C::SWZ_QK << 61;
  constexpr uint64_t kDescV = (uint64_t)(16 >> 4) << 16 | (uint64_t)(512 >> 4) << 32 | 1ull << 46 | kSwz64 << 61;
  auto at = [](uint64_t tmpl, uint32_t addr) { return tmpl | (uint64_t)((addr & 0x3FFFFu) >> 4); };

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int T2 = p.stages;                                     // 128-key stages per item (noncausal)
  const int pairs = p.N / (2 * BM);

  if (threadIdx.x == 0) {
    for (int b = 0; b < 2; ++b) {
      mbar_init(bar(B2_QFULL0 + b), 1);
      mbar_init(bar(B2_QFREE0 + b), 1);
      mbar_init(bar(B2_OFULL0 + b), 1);
      mbar_init(bar(B2_OFREE0 + b), 4);
      mbar_init(bar(B2_SFULL0 + b), 1);
      mbar_init(bar(B2_SEMPTY0 + b), 8);       // both teams of the query, four warps each
      mbar_init(bar(B2_PFULL0 + b), 4);        // the four correction warps, once per stage and query
      mbar_init(bar(B2_SMDONE0 + b), 8);
      mbar_init(bar(B2_PFREE0 + b), 1);
      mbar_init(bar(B2_DRAIN0 + b), 1);
    }
    for (int s = 0; s < C::NST; ++s) { mbar_init(bar_full(s), 1); mbar_init(bar_empty(s), 1); }
    *abortf = 0;
    fence_barrier_init();
    prefetch_tensormap(&tmQ);
    prefetch_tensormap(&tmK);
    prefetch_tensormap(&tmV);
    prefetch_tensormap(&tmO);
  }
  if (warp == 1) { tmem_alloc(sbase + C2::OFF_BAR + 768, kTmemCols); tmem_relinquish(); }
  // constant operand rows: E2M1 code 2 (= 1.0) in every nibble (their scale bytes are set per stage by the PV issuer)
  for (int i = threadIdx.x; i < C::NST * (C::ONES_BYTES / 4); i += kAttnThreads)
    reinterpret_cast<uint32_t*>(sgen + C2::OFF_STAGE + (i / (C::ONES_BYTES / 4)) * C::STAGE_BYTES + C::K_BYTES + C::V_BYTES)[i % (C::ONES_BYTES / 4)] = 0x22222222u;
  fence_proxy_async_smem();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tslot;

  if (warp == 0) {
    // ===================================================================== TMA producer
    int s = 0, ph = 0;
    uint32_t gs = 0;
    uint32_t st = sbase + C2::OFF_STAGE;
    bool ok = true;
    int i = 0;
    for (int item = blockIdx.x; ok && item < p.n_items; item += gridDim.x, ++i) {
      const WorkItem2 wi = decode_item2(item, p, pairs);
      const int ib = i & 1;
      if (i >= 2) ok = __all_sync(0xffffffffu, mbar_wait(bar(B2_QFREE0 + ib), ((i >> 1) - 1) & 1, abortf));
      if (!ok) break;
      if (elect_one()) {
        mbar_arrive_expect_tx(bar(B2_QFULL0 + ib), 2 * (C::Q_BYTES + C::QSF_BYTES));
#pragma unroll
        for (int q = 0; q < 2; ++q) {
          tma_load_2d(sbase + C2::OFF_Q + (2 * ib + q) * C::Q_BYTES, &tmQ, 0, wi.qrow0 + q * BM, bar(B2_QFULL0 + ib));
          bulk_load_1d(sbase + C2::OFF_QSF + (2 * ib + q) * 1024, p.q_sf + (size_t)(wi.qtile_lin + q) * C::QSF_BYTES, C::QSF_BYTES,
                       bar(B2_QFULL0 + ib));
        }
      }
      const uint8_t* ksf = p.k_sf + (size_t)wi.kvh * T2 * C::KSF_BYTES;
      const uint8_t* vsf = p.v_sf + (size_t)wi.kvh * T2 * C::VSF_BYTES;
      const int krow0 = wi.kvh * p.N, vrow0 = wi.kvh * D;
      for (int s2 = 0; s2 < T2; ++s2, ++gs) {
        if (gs >= (uint32_t)C::NST) ok = __all_sync(0xffffffffu, mbar_wait(bar_empty(s), ph ^ 1, abortf));
        if (!ok) break;
        const uint32_t fb = bar_full(s);
        if (elect_one()) {
          mbar_arrive_expect_tx(fb, C::K_BYTES + C::V_BYTES + C::KSF_BYTES + C::VSF_BYTES);
          tma_load_2d(st, &tmK, 0, krow0 + s2 * BS, fb);
          tma_load_2d(st + C::K_BYTES, &tmV, s2 * (BS / 2), vrow0, fb);
          bulk_load_1d(st + C::OFF_KSF, ksf + (size_t)s2 * C::KSF_BYTES, C::KSF_BYTES, fb);
          bulk_load_1d(st + C::OFF_VSF, vsf + (size_t)s2 * C::VSF_BYTES, C::VSF_BYTES, fb);
        }
        st += C::STAGE_BYTES;
        if (++s == C::NST) { s = 0; ph ^= 1; st = sbase + C2::OFF_STAGE; }
      }
    }
    if (*abortf && lane == 0) {
      for (int r = 0; r < C::NST; ++r)
        for (int spin = 0; spin < (1 << 12) && !mbar_try_wait(bar_full(r), 0) && !mbar_try_wait(bar_full(r), 1); ++spin) {}
    }
    __syncwarp();
  } else if (warp == 1) {
    // ===================================================================== QK issuer: per stage S_q = Q_q K^T for q = 0, 1
    constexpr uint32_t kIdQK = NV ? make_idesc_fp4(BM, BS, false, 0, 0) : make_idesc_fp4(BM, BS, true, 0, 0);
    int sq = 0, phq = 0;
    uint32_t stq = sbase + C2::OFF_STAGE;
    uint32_t ms = 0;                                            // stages issued so far (all items)
    bool ok = true;
    int i = 0;
    for (int item = blockIdx.x; ok && item < p.n_items; item += gridDim.x, ++i) {
      const int ib = i & 1;
      ok = __all_sync(0xffffffffu, mbar_wait(bar(B2_QFULL0 + ib), (i >> 1) & 1, abortf));
      if (!ok) break;
      tc_fence_after();
      if (elect_one()) {
#pragma unroll
        for (int q = 0; q < 2; ++q)
          tc_cp_32x128b_warpx4(tmem + k2ColSFQ + 4 * (2 * ib + q), at(kDescSF, sbase + C2::OFF_QSF + (2 * ib + q) * 1024));
      }
      for (int s2 = 0; s2 < T2; ++s2, ++ms) {
        ok = __all_sync(0xffffffffu, mbar_wait(bar_full(sq), phq, abortf));
        if (!ok) break;
        tc_fence_after();
        const uint32_t tSFK = tmem + k2ColSFK + 4 * (ms & 1);
        const uint64_t dK0 = at(kDescQK, stq);
        if (elect_one()) tc_cp_32x128b_warpx4(tSFK, at(kDescSF, stq + C::OFF_KSF));
#pragma unroll
        for (int q = 0; q < 2; ++q) {
          if (ms > 0) ok = __all_sync(0xffffffffu, mbar_wait(bar(B2_SEMPTY0 + q), (ms - 1) & 1, abortf));   // both teams of the query have read S_q
          if (!ok) break;
          tc_fence_after();
          if (elect_one()) {
            const uint64_t dQ0 = at(kDescQK, sbase + C2::OFF_Q + (2 * ib + q) * C::Q_BYTES);
            const uint32_t tSFQ = tmem + k2ColSFQ + 4 * (2 * ib + q);
            if (NV) tc_mma_fp4_4x(tmem + kColS + BS * q, dQ0, dK0, kIdQK, tSFQ, tSFK, 0);
            else    tc_mma_fp4_2x(tmem + kColS + BS * q, dQ0, dK0, kIdQK, tSFQ, tSFK, 0);
            tc_commit(bar(B2_SFULL0 + q));
            if (s2 == T2 - 1 && q == 1) tc_commit(bar(B2_QFREE0 + ib));
          }
          __syncwarp();
        }
        if (!ok) break;
        stq += C::STAGE_BYTES;
        if (++sq == C::NST) { sq = 0; phq ^= 1; stq = sbase + C2::OFF_STAGE; }
      }
    }
    if (*abortf && elect_one()) tc_commit(bar(B2_DRAIN0));
    __syncwarp();
  } else if (warp == 2) {
    // ===================================================================== PV issuer: per stage O_q += P_q V for q = 0, 1
    constexpr uint32_t kIdPV0 = make_idesc_fp4(BM, C::DN, true, 0, 0), kIdPV1 = make_idesc_fp4(BM, C::DN, true, 2, 2);
    int sp = 0;
    uint32_t stp = sbase + C2::OFF_STAGE;
    uint32_t ms = 0;
    bool ok = true;
    int i = 0;
    for (int item = blockIdx.x; ok && item < p.n_items; item += gridDim.x, ++i) {
      for (int s2 = 0; ok && s2 < T2; ++s2, ++ms) {
        const uint32_t tSFV = tmem + k2ColSFV + 4 * (ms & 1);
        const uint64_t dV = at(kDescV, stp + C::K_BYTES);
#pragma unroll
        for (int q = 0; q < 2; ++q) {
          if (s2 == 0 && i >= 1) ok = __all_sync(0xffffffffu, mbar_wait(bar(B2_OFREE0 + q), (i - 1) & 1, abortf));   // epilogue has read O_q
          if (ok) ok = __all_sync(0xffffffffu, mbar_wait(bar(B2_PFULL0 + q), ms & 1, abortf));
          if (!ok) break;
          tc_fence_after();
          if (q == 0) {
            // B rows 64..79 (the ones) take their scales from the V atom's padding rows: set them to 2^0
            if (lane < kOnesRows) *reinterpret_cast<uint32_t*>(sgen + (stp - sbase) + C::OFF_VSF + lane * 16 + 8) = 0x7F7F7F7Fu;
            fence_proxy_async_smem();
            __syncwarp();
          }
          const uint32_t tSFP = tmem + k2ColSFP + 4 * q, tO = tmem + k2ColO + k2OCols * q;
          if (elect_one()) {
            tc_cp_32x128b_warpx4(tSFP, at(kDescSF, sbase + C2::OFF_PSF + 512 * q));
            if (q == 0) tc_cp_32x128b_warpx4(tSFV, at(kDescSF, stp + C::OFF_VSF));
            tc_mma_fp4_2x_ta(tO, tmem + k2ColP + 16 * q, dV, kIdPV0, tSFP, tSFV, s2 > 0);
            tc_mma_fp4_2x_ta(tO, tmem + k2ColP + 16 * q + 8, dV + 2, kIdPV1, tSFP, tSFV, 1);
            tc_commit(bar(B2_PFREE0 + q));
            if (q == 1) tc_commit(bar_empty(sp));               // stage back to the producer
            if (s2 == T2 - 1) tc_commit(bar(B2_OFULL0 + q));
          }
          __syncwarp();
        }
        stp += C::STAGE_BYTES;
        if (++sp == C::NST) { sp = 0; stp = sbase + C2::OFF_STAGE; }
      }
    }
    if (*abortf && elect_one()) tc_commit(bar(B2_DRAIN0 + 1));
    __syncwarp();
  } else if (warp < kFirstSoftmaxWarp) {
    // ===================================================================== correction warps: two rows per thread
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;
    const uint32_t tObase = tmem + ((uint32_t)(quarter * 32) << 16) + k2ColO;
    uint32_t ms0 = 0;
    bool ok = true;
    int i = 0;
    for (int item = blockIdx.x; ok && item < p.n_items; item += gridDim.x, ++i, ms0 += T2) {
      const WorkItem2 wi = decode_item2(item, p, pairs);
      int mu[2] = {-(1 << 28), -(1 << 28)}, runmax[2] = {-(1 << 28), -(1 << 28)};
      for (uint32_t ms = ms0; ok && ms < ms0 + (uint32_t)T2; ++ms) {
#pragma unroll
        for (int q = 0; q < 2; ++q) {
          ok = __all_sync(0xffffffffu, mbar_wait(bar(B2_SMDONE0 + q), ms & 1, abortf));
          if (!ok) break;
          const int4 me = *reinterpret_cast<const int4*>(sgen + C2::OFF_META + C::META_BYTES * q + row * 16);
          const int Emax = max(max(me.x, me.y), max(me.z, me.w));
          runmax[q] = max(runmax[q], Emax);
          const bool need = Emax > mu[q] + kLazyShift;
          if (__any_sync(0xffffffffu, need)) {
            // same policy as the one-query kernel: the whole warp re-centres its references when one row asks
            int delta = runmax[q] + kRefHeadroom - mu[q];
            if (delta > 126 && runmax[q] <= mu[q] + 126 + kLazyShift) delta = 126;
            const float f = (delta > 126) ? 0.f : __uint_as_float((uint32_t)(127 - delta) << 23);
            mu[q] = (delta > 126) ? runmax[q] + kRefHeadroom : mu[q] + delta;
            if (ms != ms0) {
              ok = __all_sync(0xffffffffu, mbar_wait(bar(B2_PFREE0 + q), (ms - 1) & 1, abortf));   // PV of the previous stage has landed
              if (!ok) break;
              tc_fence_after();
#pragma unroll 1
              for (int c0 = 0; c0 < k2OCols; c0 += 16) {
                uint32_t o[16];
                tmem_ld_32x32b_x16(tObase + k2OCols * q + c0, o);
                tmem_wait_ld();
#pragma unroll
                for (int k = 0; k < 16; ++k) o[k] = __float_as_uint(__uint_as_float(o[k]) * f);
                tmem_st_32x32b_x16(tObase + k2OCols * q + c0, o);
              }
              tmem_wait_st();
              tc_fence_before();
            }
          }
          const uint32_t u0 = (uint32_t)max(me.x - mu[q] + 127, 0), u1 = (uint32_t)max(me.y - mu[q] + 127, 0);
          const uint32_t u2 = (uint32_t)max(me.z - mu[q] + 127, 0), u3 = (uint32_t)max(me.w - mu[q] + 127, 0);
          *reinterpret_cast<uint32_t*>(sgen + C2::OFF_PSF + 512 * q + lane * 16 + quarter * 4) = u0 | (u1 << 8) | (u2 << 16) | (u3 << 24);
          fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar(B2_PFULL0 + q));
        }
      }
      if (!ok) break;
      // ---- epilogue, query 0 then query 1: O = O_hw / (6 L_hw), LSE = ln2 (mu + log2(L_hw / 6))
#pragma unroll
      for (int q = 0; q < 2; ++q) {
        ok = __all_sync(0xffffffffu, mbar_wait(bar(B2_OFULL0 + q), i & 1, abortf));
        if (!ok) break;
        tc_fence_after();
        const uint32_t tO = tObase + k2OCols * q;
        float Lhw;
        {
          uint32_t r16[16];
          tmem_ld_32x32b_x16(tO + D, r16);
          tmem_wait_ld();
          Lhw = __uint_as_float(r16[0]);
        }
        const float inv = __frcp_rn(6.0f * Lhw);
        if (lane == 0) bulk_wait_read_all();                    // this warp's previous store has read the buffer
        __syncwarp();
        uint8_t* orow = sgen + C2::OFF_OUT + row * 128;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          uint32_t o[16];
          tmem_ld_32x32b_x16(tO + 16 * c, o);
          tmem_wait_ld();
          if (c == 3) {                                         // last read of O_q: the next item's PV may overwrite it
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(B2_OFREE0 + q));
          }
#pragma unroll
          for (int k = 0; k < 16; k += 8) {
            uint32_t pk[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const __nv_bfloat162 hh = __floats2bfloat162_rn(__uint_as_float(o[k + 2 * j]) * inv, __uint_as_float(o[k + 2 * j + 1]) * inv);
              pk[j] = *reinterpret_cast<const uint32_t*>(&hh);
            }
            const int chunk = (16 * c + k) >> 3;
            *reinterpret_cast<uint4*>(orow + ((chunk ^ (row & 7)) << 4)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
          }
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
          tma_store_2d(&tmO, 0, wi.qrow0 + q * BM + quarter * 32, sbase + C2::OFF_OUT + quarter * 32 * 128);
          bulk_commit_group();
        }
        if (p.LSE) p.LSE[(size_t)wi.qrow0 + q * BM + row] = 0.69314718055994531f * ((float)mu[q] + (log2f(Lhw) - 2.5849625007211560f));
      }
    }
  } else {
    // ===================================================================== softmax teams: team 2q + h, every stage of query q
    const int team = (warp - kFirstSoftmaxWarp) >> 2;
    const int q = team >> 1;
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;
    const uint32_t tS = tmem + ((uint32_t)(quarter * 32) << 16) + kColS + BN * team;
    const uint32_t sfull = bar(B2_SFULL0 + q), sempty = bar(B2_SEMPTY0 + q);
    const uint32_t smdone = bar(B2_SMDONE0 + q), pfree = bar(B2_PFREE0 + q);
    const uint32_t tP = tmem + ((uint32_t)(quarter * 32) << 16) + k2ColP + 8 * team;
    int2* meta = reinterpret_cast<int2*>(sgen + C2::OFF_META + C::META_BYTES * q + row * 16 + 8 * (team & 1));
    float c32;
    if (NV) c32 = __fdiv_rn(p.c_base, __fmul_rn(__ldg(p.q_G), __ldg(p.k_G)));
    else    c32 = __fdiv_rn(p.c_base, 36.0f);
    bool ok = true;
    uint32_t ms = 0;
    for (int item = blockIdx.x; ok && item < p.n_items; item += gridDim.x) {
      for (int s2 = 0; s2 < T2; ++s2, ++ms) {
        ok = __all_sync(0xffffffffu, mbar_wait(sfull, ms & 1, abortf));
        if (!ok) break;
        tc_fence_after();
        uint32_t sraw[32], w0[4], w1[4];
        int E0, E1;
        tmem_ld_32x32b_x32(tS, sraw);
        tmem_wait_ld();
        direct_p_block<PMAP, false, THR16>(sraw, c32, p.aff_a, p.aff_b, 32, E0, w0);
        tmem_ld_32x32b_x32(tS + 32, sraw);
        tmem_wait_ld();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(sempty);                     // S_q may take the next stage
        direct_p_block<PMAP, false, THR16>(sraw, c32, p.aff_a, p.aff_b, 32, E1, w1);
        if (ms > 0) ok = __all_sync(0xffffffffu, mbar_wait(pfree, (ms - 1) & 1, abortf));   // PV of the query's previous stage is done
        if (!ok) break;
        {
          const uint32_t pw[8] = {w0[0], w0[1], w0[2], w0[3], w1[0], w1[1], w1[2], w1[3]};
          tmem_st_32x32b_x8(tP, pw);
        }
        *meta = make_int2(E0, E1);
        tmem_wait_st();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smdone);
      }
    }
  }
  if (warp >= 3 && warp < kFirstSoftmaxWarp && lane == 0) bulk_wait_all();
  __syncthreads();
  if (*abortf && threadIdx.x == 0 && p.status) *p.status = FP4ATTN_ERR_TIMEOUT;
  if (warp == 1) {
    if (*abortf && lane == 0) {
      for (int r = 0; r < 2; ++r)
        for (int spin = 0; spin < (1 << 14) && !mbar_try_wait(bar(B2_DRAIN0 + r), 0); ++spin) {}
    }
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem, kTmemCols);
  }
}

template <int NV, int PMAP, bool THR16>
static int launch_2q(const fp4attn_operands* ops, int B, int H, int N, AttnParams prm, cudaStream_t st) {
  using C2 = Cfg2<(NV != 0)>;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return FP4ATTN_ERR_CUDA;
  static std::atomic<bool> attr_set[kMaxDevices];
  if (dev < 0 || dev >= kMaxDevices) return FP4ATTN_ERR_CUDA;
  if (!attr_set[dev].load(std::memory_order_acquire)) {
    if (cudaFuncSetAttribute(attn_fwd_2q_kernel<NV, PMAP, THR16>, cudaFuncAttributeMaxDynamicSharedMemorySize, C2::SMEM_BYTES) != cudaSuccess)
      return FP4ATTN_ERR_CUDA;
    attr_set[dev].store(true, std::memory_order_release);
  }
  const CUtensorMap* tm = attention_tensor_maps(64, ops, prm.O, B, H, prm.Hkv, N);
  if (!tm) return FP4ATTN_ERR_CUDA;
  const unsigned grid = (unsigned)(prm.n_items < sms ? prm.n_items : sms);
  attn_fwd_2q_kernel<NV, PMAP, THR16><<<grid, kAttnThreads, C2::SMEM_BYTES, st>>>(tm[0], tm[1], tm[2], tm[3], prm);
  return cudaGetLastError() == cudaSuccess ? FP4ATTN_OK : FP4ATTN_ERR_CUDA;
}

// Entry used by fp4attn_fwd for schedule = FP4ATTN_SCHEDULE_TWO_QUERY; the caller has validated everything that
// does not depend on the schedule and filled `prm` for the one-query kernel.
int launch_attn_two_query(const fp4attn_operands* ops, int B, int H, int N, int d, int pmap, AttnParams prm, cudaStream_t st) {
  if (d != 64 || N % (2 * BM) != 0 || ops->causal || ops->g_per_head) return FP4ATTN_ERR_UNSUPPORTED_SHAPE;
  const int pairs = N / (2 * BM);
  prm.n_items = B * H * pairs;
  prm.recip_qtiles = pairs > 1 ? ~0ull / (unsigned long long)pairs + 1 : 0;
  const bool nv = ops->qk_fmt == FP4ATTN_FMT_NVFP4;
#define FP4ATTN_2Q(PM_)                                                                  \
  if (prm.thr16) return nv ? launch_2q<1, PM_, true>(ops, B, H, N, prm, st) : launch_2q<0, PM_, true>(ops, B, H, N, prm, st); \
  return nv ? launch_2q<1, PM_, false>(ops, B, H, N, prm, st) : launch_2q<0, PM_, false>(ops, B, H, N, prm, st);
  switch (pmap) {
    case 0: FP4ATTN_2Q(0)
    case 1: FP4ATTN_2Q(1)
    case 2: FP4ATTN_2Q(2)
    case 3: FP4ATTN_2Q(3)
    default: FP4ATTN_2Q(4)
  }
#undef FP4ATTN_2Q
}

}  // namespace fp4attn
