// Full-FP4 attention forward with Direct-P for sm_100a (noncausal or causal, optional grouped K/V heads, optional
// per-batch token counts for padded sequences).
//
// Persistent kernel, one CTA per SM.  A CTA takes work items (one 128-row query tile of one
// (batch, head)) round-robin and walks the keys of an item in stages of 128 (two 64-key tiles, four
// N32 probability blocks).  Score tiles live in a ring of four 64-column TMEM slots (two per stage),
// each served by its own team of four softmax warps, so four independent score->code streams share
// every SM sub-partition; everything that is sequential in the key index (row reference, rescale of O,
// scale bytes of P) is done by separate correction warps on four numbers per row and stage.  All roles
// keep running counters across items, so the next item's loads, QK products and softmax overlap the
// previous item's epilogue.
//
//   warp 0        TMA producer: Q tile per item (two buffers), ring of {K, V^T, K scales, V scales}
//   warp 1        tensor-core issuer for S = Q K^T, one 128-key stage (two score slots) per issue
//   warp 2        tensor-core issuer for O += P V, one stage (two K64 products) per issue
//   warps 3-6     correction: integer row reference, E8M0 bytes of P, exact power-of-two rescale of
//                 O, epilogue; one pass per stage
//   warps 7-22    softmax teams 0..3, one thread per query row; team 2p+h serves the h-th 64 keys of
//                 the stages with parity p: Algorithm "direct-p-pack" up to the codes (written
//                 straight into tensor memory, PV's A operand) and the block exponents; codes do not
//                 depend on the row reference, so teams never wait for one another
//
// The represented row sum (the denominator of Eq. "represented-output") is produced by the same PV
// instruction as the numerator: sixteen constant rows of ones follow V^T in every stage, so column d
// of the accumulator is sum_j 2^(u_B-127) q_j over exactly the codes and scale bytes PV consumed.
//
// Tensor memory (512 columns): S slots 0..255 | O 256..399 (d + 16 columns) | Q scales 400..415 (two
// buffers) | K scales 416..431 (two slots) | V scales 432..447 (two slots of 8) | P scales 448..455 |
// P codes 456..487 (per stage parity and 64-key tile 8 columns: 64 keys x 4 bits per row).
#include "attn_common.cuh"

namespace fp4attn {
using namespace ptx;

// CAUSAL: the instances that mask the last stage of an item.  They serve the causal mask (p.causal), padded
// sequences (p.seq_len) and both together; the other instances never look at either field.
// NV: 0 - MXFP4 Q, K; 1 - NVFP4 with one encode factor per tensor; 2 - NVFP4 with one factor per (batch, head)
// unit (an instance of its own: a score constant that changes per work item costs the tensor-wide variant
// 2-8 % when it is only a run-time branch)
// FIXREF: the row reference is the constant p.ref_fixed (the shiftless path): the teams publish the E8M0 bytes of
// their blocks themselves, the PV issuer waits for the teams, nothing is ever rescaled, and the correction warps are
// left with the epilogue.
template <int D, int NV, int PMAP, bool CAUSAL, int THR16, bool FIXREF = false>
__global__ void __launch_bounds__(kAttnThreads, 1)
attn_fwd_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmO,
                const AttnParams p) {
  using C = Cfg<D, (NV != 0)>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* sgen = smem_raw + (sbase - smem_u32(smem_raw));
  uint32_t* tslot = reinterpret_cast<uint32_t*>(sgen + C::OFF_BAR + 768);
  volatile int* abortf = reinterpret_cast<volatile int*>(sgen + C::OFF_BAR + 776);
  auto bar = [&](int i) { return sbase + C::OFF_BAR + 8u * i; };
  auto bar_full = [&](int s) { return bar(BAR_RING + s); };
  auto bar_empty = [&](int s) { return bar(BAR_RING + C::NST + s); };
  // descriptor templates: everything but the 14 address bits is loop-invariant
  constexpr uint64_t kDescSF = (uint64_t)(16 >> 4) << 16 | (uint64_t)(128 >> 4) << 32 | 1ull << 46;
  constexpr uint64_t kDescQK = (uint64_t)(16 >> 4) << 16 | (uint64_t)((8 * C::ROW_BYTES) >> 4) << 32 | 1ull << 46 | C::SWZ_QK << 61;
  constexpr uint64_t kDescV = (uint64_t)(16 >> 4) << 16 | (uint64_t)(512 >> 4) << 32 | 1ull << 46 | kSwz64 << 61;
  auto at = [](uint64_t tmpl, uint32_t addr) { return tmpl | (uint64_t)((addr & 0x3FFFFu) >> 4); };

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int qtiles = p.N / BM;

  if (threadIdx.x == 0) {
    for (int b = 0; b < 2; ++b) {
      mbar_init(bar(BAR_QFULL0 + b), 1);
      mbar_init(bar(BAR_QFREE0 + b), 1);
      mbar_init(bar(BAR_SFULL0 + b), 1);
      mbar_init(bar(BAR_SEMPTY0 + b), 8);      // both teams of the pair, four warps each
      mbar_init(bar(BAR_PFULL0 + b), 4);       // the four correction warps, once per stage
      mbar_init(bar(BAR_SMDONE0 + b), 8);      // both teams of the pair, four warps each
      mbar_init(bar(BAR_PFREE0 + b), 1);
    }
    mbar_init(bar(BAR_OFULL), 1);
    mbar_init(bar(BAR_OFREE), 4);
    mbar_init(bar(BAR_DRAIN0), 1);             // time-out path only: one per tensor-core issuer
    mbar_init(bar(BAR_DRAIN0 + 1), 1);
    for (int s = 0; s < C::NST; ++s) { mbar_init(bar_full(s), 1); mbar_init(bar_empty(s), 1); }
    *abortf = 0;
    fence_barrier_init();
    prefetch_tensormap(&tmQ);
    prefetch_tensormap(&tmK);
    prefetch_tensormap(&tmV);
    prefetch_tensormap(&tmO);
  }
  if (warp == 1) { tmem_alloc(sbase + C::OFF_BAR + 768, kTmemCols); tmem_relinquish(); }
  // constant operand rows: E2M1 code 2 (= 1.0) in every nibble, E8M0 byte 127 (= 2^0) as their scale
  for (int i = threadIdx.x; i < C::NST * (C::ONES_BYTES / 4); i += kAttnThreads)
    reinterpret_cast<uint32_t*>(sgen + C::OFF_STAGE + (i / (C::ONES_BYTES / 4)) * C::STAGE_BYTES + C::K_BYTES + C::V_BYTES)[i % (C::ONES_BYTES / 4)] = 0x22222222u;
  for (int i = threadIdx.x; i < 128; i += kAttnThreads) reinterpret_cast<uint32_t*>(sgen + C::OFF_ONESF)[i] = 0x7F7F7F7Fu;
  fence_proxy_async_smem();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tslot;

  if (warp == 0) {
    // ===================================================================== TMA producer
    // The whole warp runs the loop (addresses and waits stay warp-uniform); one elected lane issues.
    int s = 0, ph = 0;
    uint32_t gs = 0;                                            // stages issued so far (all items)
    uint32_t st = sbase + C::OFF_STAGE;
    bool ok = true;
    int i = 0;
    for (int item = blockIdx.x; ok && item < p.n_items; item += gridDim.x, ++i) {
      const WorkItem wi = decode_item<CAUSAL>(item, p, qtiles);
      const int T2 = wi.T2;
      const int qb = i & 1;
      if (i >= 2) ok = __all_sync(0xffffffffu, mbar_wait(bar(BAR_QFREE0 + qb), ((i >> 1) - 1) & 1, abortf));
      if (!ok) break;
      if (elect_one()) {
        mbar_arrive_expect_tx(bar(BAR_QFULL0 + qb), C::Q_BYTES + C::QSF_BYTES);
        tma_load_2d(sbase + C::OFF_Q + qb * C::Q_BYTES, &tmQ, 0, wi.qrow0, bar(BAR_QFULL0 + qb));
        bulk_load_1d(sbase + C::OFF_QSF + qb * 1024, p.q_sf + (size_t)wi.qtile_lin * C::QSF_BYTES, C::QSF_BYTES, bar(BAR_QFULL0 + qb));
      }
      const uint8_t* ksf = p.k_sf + (size_t)wi.kvh * qtiles * C::KSF_BYTES;
      const uint8_t* vsf = p.v_sf + (size_t)wi.kvh * qtiles * C::VSF_BYTES;
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
        if (++s == C::NST) { s = 0; ph ^= 1; st = sbase + C::OFF_STAGE; }
      }
    }
    if (*abortf && lane == 0) {
      // bounded drain: give copies still in flight time to land before the CTA retires
      for (int r = 0; r < C::NST; ++r)
        for (int spin = 0; spin < (1 << 12) && !mbar_try_wait(bar_full(r), 0) && !mbar_try_wait(bar_full(r), 1); ++spin) {}
    }
    __syncwarp();
  } else if (warp == 1) {
    // ===================================================================== QK issuer: S = Q K^T, one stage per issue
    // Warp-uniform control flow; tcgen05 instructions are issued by one elected lane.
    constexpr uint32_t kIdQK0 = NV ? make_idesc_fp4(BM, BS, false, 0, 0) : make_idesc_fp4(BM, BS, true, 0, 0);
    constexpr uint32_t kIdQK1 = NV ? make_idesc_fp4(BM, BS, false, 0, 0) : make_idesc_fp4(BM, BS, true, 2, 2);
    int sq = 0, phq = 0;
    uint32_t stq = sbase + C::OFF_STAGE;
    uint32_t g = 0;                                             // stages issued so far (all items)
    bool ok = true;
    int i = 0;
    for (int item = blockIdx.x; ok && item < p.n_items; item += gridDim.x, ++i) {
      const int T2 = decode_item<CAUSAL>(item, p, qtiles).T2;
      const int qb = i & 1;
      ok = __all_sync(0xffffffffu, mbar_wait(bar(BAR_QFULL0 + qb), (i >> 1) & 1, abortf));
      if (!ok) break;
      tc_fence_after();
      const uint32_t tSFQ = tmem + kColSFQ + 8 * qb;
      if (elect_one()) {
#pragma unroll
        for (int a = 0; a < C::CTQ; ++a) tc_cp_32x128b_warpx4(tSFQ + 4 * a, at(kDescSF, sbase + C::OFF_QSF + qb * 1024 + 512 * a));
      }
      const uint64_t dQ0 = at(kDescQK, sbase + C::OFF_Q + qb * C::Q_BYTES);
      for (int s2 = 0; s2 < T2; ++s2, ++g) {
        const int pr = g & 1;
        const uint32_t m = g >> 1;
        ok = __all_sync(0xffffffffu, mbar_wait(bar_full(sq), phq, abortf));
        if (ok && m > 0) ok = __all_sync(0xffffffffu, mbar_wait(bar(BAR_SEMPTY0 + pr), (m - 1) & 1, abortf));   // both teams have read the pair
        if (!ok) break;
        tc_fence_after();
        const uint32_t tSFK = tmem + kColSFK + 8 * pr;
        const uint32_t tS = tmem + kColS + BS * pr;
        const uint64_t dK0 = at(kDescQK, stq);
        if (elect_one()) {
#pragma unroll
          for (int a = 0; a < C::CTQ; ++a) tc_cp_32x128b_warpx4(tSFK + 4 * a, at(kDescSF, stq + C::OFF_KSF + 512 * a));
          if (NV) {
            tc_mma_fp4_4x(tS, dQ0, dK0, kIdQK0, tSFQ, tSFK, 0);
            if (C::KBLK == 2) tc_mma_fp4_4x(tS, dQ0 + 2, dK0 + 2, kIdQK1, tSFQ + 4, tSFK + 4, 1);
          } else {
            tc_mma_fp4_2x(tS, dQ0, dK0, kIdQK0, tSFQ, tSFK, 0);
            if (C::KBLK == 2) tc_mma_fp4_2x(tS, dQ0 + 2, dK0 + 2, kIdQK1, tSFQ, tSFK, 1);
          }
          tc_commit(bar(BAR_SFULL0 + pr));
          if (s2 == T2 - 1) tc_commit(bar(BAR_QFREE0 + qb));    // Q buffer may take the item after next
        }
        __syncwarp();
        stq += C::STAGE_BYTES;
        if (++sq == C::NST) { sq = 0; phq ^= 1; stq = sbase + C::OFF_STAGE; }
      }
    }
    if (*abortf && elect_one()) tc_commit(bar(BAR_DRAIN0));      // completes when this warp's products and copies have
    __syncwarp();
  } else if (warp == 2) {
    // ===================================================================== PV issuer: O += P V, one stage per issue
    constexpr uint32_t kIdPV0 = make_idesc_fp4(BM, C::DN, true, 0, 0), kIdPV1 = make_idesc_fp4(BM, C::DN, true, 2, 2);
    const uint32_t tO = tmem + kColO;
    if (D == 128) {
      // B rows 128..143 (the ones) read their scales from a fifth column group: constant, set once per slot
      if (elect_one()) {
        tc_cp_32x128b_warpx4(tmem + kColSFV + 4, at(kDescSF, sbase + C::OFF_ONESF));
        tc_cp_32x128b_warpx4(tmem + kColSFV + 12, at(kDescSF, sbase + C::OFF_ONESF));
      }
      __syncwarp();
    }
    int sp = 0;
    uint32_t stp = sbase + C::OFF_STAGE;
    uint32_t g = 0;
    bool ok = true;
    int i = 0;
    for (int item = blockIdx.x; ok && item < p.n_items; item += gridDim.x, ++i) {
      const int T2 = decode_item<CAUSAL>(item, p, qtiles).T2;
      if (i >= 1) ok = __all_sync(0xffffffffu, mbar_wait(bar(BAR_OFREE), (i - 1) & 1, abortf));   // epilogue has read O
      for (int s2 = 0; ok && s2 < T2; ++s2, ++g) {
        const int pr = g & 1;
        const uint32_t m = g >> 1;
        // codes of both tiles are in tensor memory, their scale bytes in shared memory (written by the correction
        // warps, or with a fixed reference by the teams themselves)
        ok = __all_sync(0xffffffffu, mbar_wait(bar((FIXREF ? BAR_SMDONE0 : BAR_PFULL0) + pr), m & 1, abortf));
        if (!ok) break;
        tc_fence_after();
        const uint32_t tSFP = tmem + kColSFP + 4 * pr, tSFV = tmem + kColSFV + 8 * pr;
        if (D == 64) {
          // B rows 64..79 (the ones) take their scales from the V atom's padding rows: set them to 2^0
          if (lane < kOnesRows) *reinterpret_cast<uint32_t*>(sgen + (stp - sbase) + C::OFF_VSF + lane * 16 + 8) = 0x7F7F7F7Fu;
          fence_proxy_async_smem();
          __syncwarp();
        }
        const uint64_t dV = at(kDescV, stp + C::K_BYTES);
        if (elect_one()) {
          tc_cp_32x128b_warpx4(tSFP, at(kDescSF, sbase + C::OFF_PSF + 512 * pr));
          tc_cp_32x128b_warpx4(tSFV, at(kDescSF, stp + C::OFF_VSF));
          // tile h of the stage: P codes from tensor memory (the A operand; written there by the teams, so
          // no shared-memory round trip and no proxy fence), keys 64h..64h+63 of V^T (32 bytes on), scale
          // bytes {2h, 2h+1}
          tc_mma_fp4_2x_ta(tO, tmem + kColP + 16 * pr, dV, kIdPV0, tSFP, tSFV, s2 > 0);
          tc_mma_fp4_2x_ta(tO, tmem + kColP + 16 * pr + 8, dV + 2, kIdPV1, tSFP, tSFV, 1);
          tc_commit(bar_empty(sp));                             // stage back to the producer
          tc_commit(bar(BAR_PFREE0 + pr));                      // the stage's P columns reusable; O holds this stage
          if (s2 == T2 - 1) tc_commit(bar(BAR_OFULL));
        }
        __syncwarp();
        stp += C::STAGE_BYTES;
        if (++sp == C::NST) { sp = 0; stp = sbase + C::OFF_STAGE; }
      }
    }
    if (*abortf && elect_one()) tc_commit(bar(BAR_DRAIN0 + 1));
    __syncwarp();
  } else if (warp < kFirstSoftmaxWarp) {
    // ===================================================================== correction warps
    // One thread per query row, stages in key order.  Owns the integer row reference mu and the O
    // accumulator's scale (numerator and row-sum columns alike); turns the teams' absolute block exponents
    // into the E8M0 bytes the PV instruction reads.
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;
    const uint32_t tO = tmem + ((uint32_t)(quarter * 32) << 16) + kColO;
    uint32_t g0 = 0;                                            // stages completed in earlier items
    bool ok = true;
    int i = 0;
    int T2 = 0;
    int mu_next = -(1 << 28);                                   // reference of the item whose first stage was served ahead
    bool first_served = false;
    for (int item = blockIdx.x; ok && item < p.n_items; item += gridDim.x, ++i, g0 += T2) {
      const WorkItem wi = decode_item<CAUSAL>(item, p, qtiles);
      T2 = wi.T2;
      const bool has_next = item + (int)gridDim.x < p.n_items;
      int mu = FIXREF ? p.ref_fixed : (first_served ? mu_next : -(1 << 28));
      int runmax = first_served ? mu_next - kRefHeadroom : -(1 << 28);   // largest block exponent of the row so far
      // One pass per 128-key stage (both of its tiles).  The item's first stage may already have been served
      // from inside the previous item's epilogue.
      for (uint32_t g = FIXREF ? g0 + (uint32_t)T2 : g0 + (first_served ? 1u : 0u); g < g0 + (uint32_t)T2; ++g) {
        const bool first_of_item = g == g0;
        const int pr = g & 1;
        ok = __all_sync(0xffffffffu, mbar_wait(bar(BAR_SMDONE0 + pr), (g >> 1) & 1, abortf));
        if (!ok) break;
        const int4 me = *reinterpret_cast<const int4*>(sgen + C::OFF_META + C::META_BYTES * pr + row * 16);
        const int Emax = max(max(me.x, me.y), max(me.z, me.w));
        runmax = max(runmax, Emax);
        const bool need = Emax > mu + kLazyShift;
        if (__any_sync(0xffffffffu, need)) {
          // New reference: kRefHeadroom above the row's largest block exponent so far, but never more than 126
          // octaves above the old one while the old contributions can still matter (they reach up to
          // mu + kLazyShift); only when even that is out of reach are they dropped (f = 0).  The pass over O is
          // paid for by the whole warp, so the rows that did not ask for it re-centre as well (for them
          // 0 <= delta <= kLazyShift + kRefHeadroom): every row has its full span again afterwards, which keeps
          // passes rare for the warp as a whole (with outlier channels one raise per row would otherwise mean
          // a pass in every few stages).
          int delta = runmax + kRefHeadroom - mu;
          if (delta > 126 && runmax <= mu + 126 + kLazyShift) delta = 126;
          const float f = (delta > 126) ? 0.f : __uint_as_float((uint32_t)(127 - delta) << 23);
          mu = (delta > 126) ? runmax + kRefHeadroom : mu + delta;
          if (!first_of_item) {
            // O holds the item's earlier stages once their PV has landed (an item's first stage never
            // touches O: it may still belong to the previous item)
            const uint32_t gprev = g - 1;
            ok = __all_sync(0xffffffffu, mbar_wait(bar(BAR_PFREE0 + (gprev & 1)), (gprev >> 1) & 1, abortf));
            if (!ok) break;
            tc_fence_after();
#pragma unroll 1
            for (int c0 = 0; c0 < C::DN; c0 += 16) {             // numerator columns and the row-sum columns
              uint32_t o[16];
              tmem_ld_32x32b_x16(tO + c0, o);
              tmem_wait_ld();
#pragma unroll
              for (int q = 0; q < 16; ++q) o[q] = __float_as_uint(__uint_as_float(o[q]) * f);
              tmem_st_32x32b_x16(tO + c0, o);
            }
            tmem_wait_st();
            tc_fence_before();
          }
        }
        // A block more than 126 octaves below the reference is a zero block: it gets the smallest
        // byte (2^-127, below 2^-60 of the row's mass by construction) in numerator and row sum alike.
        const uint32_t u0 = (uint32_t)max(me.x - mu + 127, 0), u1 = (uint32_t)max(me.y - mu + 127, 0);
        const uint32_t u2 = (uint32_t)max(me.z - mu + 127, 0), u3 = (uint32_t)max(me.w - mu + 127, 0);
        *reinterpret_cast<uint32_t*>(sgen + C::OFF_PSF + 512 * pr + lane * 16 + quarter * 4) = u0 | (u1 << 8) | (u2 << 16) | (u3 << 24);
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(BAR_PFULL0 + pr));
      }
      if (!ok) break;
      first_served = false;
      // ---- epilogue: with L_hw = column d of the accumulator, O = O_hw / (6 L_hw), LSE = ln2 (mu + log2(L_hw / 6))
      ok = __all_sync(0xffffffffu, mbar_wait(bar(BAR_OFULL), i & 1, abortf));
      if (!ok) break;
      tc_fence_after();
      float Lhw;
      {
        uint32_t r16[16];
        tmem_ld_32x32b_x16(tO + D, r16);
        tmem_wait_ld();
        Lhw = __uint_as_float(r16[0]);
      }
      const float inv = __frcp_rn(6.0f * Lhw);
      if (FIXREF && !(Lhw > 0.f && Lhw < INFINITY) && p.status) *p.status = FP4ATTN_ERR_RANGE;   // nothing of the row is inside the byte range
      const size_t grow = (size_t)wi.qrow0 + row;
      // stage the bf16 tile in shared memory (128-byte rows, 128B-swizzled like the tensor map) and
      // let TMA write it out, so O is released after four TMEM reads instead of after 16 global stores
      if (lane == 0) bulk_wait_read_all();                      // this warp's previous stores have read the buffer
      __syncwarp();
      // 16-column chunks, the next one in flight from tensor memory while this one is normalised and stored
      uint32_t oa[16], ob[16];
      tmem_ld_32x32b_x16(tO, oa);
      tmem_wait_ld();
#pragma unroll
      for (int c0 = 0; c0 < D; c0 += 16) {
        uint32_t* o = ((c0 >> 4) & 1) ? ob : oa;
        uint32_t* nx = ((c0 >> 4) & 1) ? oa : ob;
        if (c0 + 16 < D) tmem_ld_32x32b_x16(tO + c0 + 16, nx);
        uint8_t* half = sgen + C::OFF_OUT + (c0 >> 6) * (BM * 128) + row * 128;
#pragma unroll
        for (int c = 0; c < 16; c += 8) {
          uint32_t pk[4];
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const __nv_bfloat162 hh = __floats2bfloat162_rn(__uint_as_float(o[c + 2 * q]) * inv, __uint_as_float(o[c + 2 * q + 1]) * inv);
            pk[q] = *reinterpret_cast<const uint32_t*>(&hh);
          }
          const int chunk = ((c0 & 63) + c) >> 3;               // 16-byte chunk of the 128-byte row
          *reinterpret_cast<uint4*>(half + ((chunk ^ (row & 7)) << 4)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
        }
        if (c0 + 16 < D) {
          tmem_wait_ld();
          if (c0 + 32 == D) {                                   // last read of O: the next item's PV may overwrite it
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(BAR_OFREE));
          }
        }
      }
      if (!FIXREF && PMAP != 1 && has_next) {
        // O is released; before the stores go out, serve the next item's first stage (the teams run ahead and
        // have it encoded, or will shortly - nothing they need depends on this epilogue), so that its PV waits
        // for neither the rest of this epilogue nor a pass after it.  A first stage starts a fresh reference,
        // kRefHeadroom above its largest block exponent, and never touches O.  (Measured against serving it
        // before the epilogue: +1 % with exponentials in the map; the pure affine map loses 1 % at long
        // sequences either way and serves the stage in its own loop, after the epilogue.)
        const uint32_t g = g0 + (uint32_t)T2;
        const int pr = g & 1;
        ok = __all_sync(0xffffffffu, mbar_wait(bar(BAR_SMDONE0 + pr), (g >> 1) & 1, abortf));
        if (!ok) break;
        const int4 me = *reinterpret_cast<const int4*>(sgen + C::OFF_META + C::META_BYTES * pr + row * 16);
        mu_next = max(max(me.x, me.y), max(me.z, me.w)) + kRefHeadroom;
        const uint32_t u0 = (uint32_t)max(me.x - mu_next + 127, 0), u1 = (uint32_t)max(me.y - mu_next + 127, 0);
        const uint32_t u2 = (uint32_t)max(me.z - mu_next + 127, 0), u3 = (uint32_t)max(me.w - mu_next + 127, 0);
        *reinterpret_cast<uint32_t*>(sgen + C::OFF_PSF + 512 * pr + lane * 16 + quarter * 4) = u0 | (u1 << 8) | (u2 << 16) | (u3 << 24);
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(BAR_PFULL0 + pr));
        first_served = true;
      }
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) {                                          // this warp's 32 rows, one box per 128-byte half
#pragma unroll
        for (int hf = 0; hf < D / 64; ++hf)
          tma_store_2d(&tmO, hf * 128, wi.qrow0 + quarter * 32, sbase + C::OFF_OUT + hf * (BM * 128) + quarter * 32 * 128);
        bulk_commit_group();
      }
      if (p.LSE) p.LSE[grow] = 0.69314718055994531f * ((float)mu + (log2f(Lhw) - 2.5849625007211560f));
    }
  } else {
    // ===================================================================== softmax teams
    const int team = (warp - kFirstSoftmaxWarp) >> 2;
    const int pr = team >> 1;                                   // stage parity this team serves (keys 64*(team&1)..)
    const int quarter = warp & 3;                               // TMEM lane quarter this warp may touch
    const int row = quarter * 32 + lane;
    const uint32_t tS = tmem + ((uint32_t)(quarter * 32) << 16) + kColS + BN * team;
    const uint32_t sfull = bar(BAR_SFULL0 + pr), sempty = bar(BAR_SEMPTY0 + pr);
    const uint32_t smdone = bar(BAR_SMDONE0 + pr), pfree = bar(BAR_PFREE0 + pr);
    const uint32_t tP = tmem + ((uint32_t)(quarter * 32) << 16) + kColP + 8 * team;
    int2* meta = reinterpret_cast<int2*>(sgen + C::OFF_META + C::META_BYTES * pr + row * 16 + 8 * (team & 1));
    float c32;
    if (NV) c32 = __fdiv_rn(p.c_base, __fmul_rn(__ldg(p.q_G), __ldg(p.k_G)));
    else    c32 = __fdiv_rn(p.c_base, 36.0f);
    uint32_t g0 = 0;
    bool ok = true;
    int T2 = 0;
    for (int item = blockIdx.x; ok && item < p.n_items; item += gridDim.x, g0 += T2) {
      uint32_t gdiag;                                           // global index of the item's masked stage, its last (none: ~0)
      int vis;                                                  // keys of that stage this row sees
      {
        const WorkItem wi = decode_item<CAUSAL>(item, p, qtiles);
        T2 = wi.T2;
        gdiag = CAUSAL ? g0 + (uint32_t)(T2 - 1) : 0xFFFFFFFFu;
        // causal: keys 0..i of row i = qt * 128 + row; padded sequence: keys 0..len-1; both: the fewer
        const int seen = (CAUSAL && p.causal) ? min(wi.len, wi.qt * BM + row + 1) : wi.len;
        vis = seen - (T2 - 1) * BS;
        if (NV == 2)                                            // this unit's own pair of encode factors
          c32 = __fdiv_rn(p.c_base, __fmul_rn(__ldg(p.q_G + wi.bh), __ldg(p.k_G + wi.kvh)));
      }
      for (uint32_t g = g0 + ((g0 & 1) != (uint32_t)pr); g < g0 + T2; g += 2) {   // this team's stages of the item
        const uint32_t m = g >> 1;
        ok = __all_sync(0xffffffffu, mbar_wait(sfull, m & 1, abortf));
        if (!ok) break;
        tc_fence_after();
        uint32_t sraw[32], w0[4], w1[4];
        int E0, E1;
        tmem_ld_32x32b_x32(tS, sraw);
        tmem_wait_ld();
        if (!CAUSAL || g != gdiag) {
          direct_p_block<PMAP, false, THR16>(sraw, c32, p.aff_a, p.aff_b, 32, E0, w0);
          tmem_ld_32x32b_x32(tS + 32, sraw);
          tmem_wait_ld();
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(sempty);                   // pair may take the stage after next
          direct_p_block<PMAP, false, THR16>(sraw, c32, p.aff_a, p.aff_b, 32, E1, w1);
        } else {
          // masked stage: this row sees the first `vis` keys of the stage; the team's tile starts at key 64*(team&1)
          const int v0 = vis - 64 * (team & 1);
          direct_p_block<PMAP, true, THR16>(sraw, c32, p.aff_a, p.aff_b, v0, E0, w0);
          tmem_ld_32x32b_x32(tS + 32, sraw);
          tmem_wait_ld();
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(sempty);
          direct_p_block<PMAP, true, THR16>(sraw, c32, p.aff_a, p.aff_b, v0 - 32, E1, w1);
        }
        if (m > 0) ok = __all_sync(0xffffffffu, mbar_wait(pfree, (m - 1) & 1, abortf));   // PV of the pair's previous stage is done
        if (!ok) break;
        // fixed reference: E8M0 bytes of the two blocks against the constant; below the range a zero block (no codes,
        // so that a row without any live block shows as a zero row sum), above it an error
        const int b0 = FIXREF ? E0 - p.ref_fixed + 127 : 0, b1 = FIXREF ? E1 - p.ref_fixed + 127 : 0;
        if (FIXREF && __any_sync(0xffffffffu, min(b0, b1) < 1)) {    // rare: some row of the warp has a block below the range
          if (b0 < 1) w0[0] = w0[1] = w0[2] = w0[3] = 0u;
          if (b1 < 1) w1[0] = w1[1] = w1[2] = w1[3] = 0u;
        }
        {
          const uint32_t pw[8] = {w0[0], w0[1], w0[2], w0[3], w1[0], w1[1], w1[2], w1[3]};
          tmem_st_32x32b_x8(tP, pw);
        }
        if (FIXREF) {
          if (max(b0, b1) > 254 && p.status) *p.status = FP4ATTN_ERR_RANGE;      // (the byte written below is then meaningless)
          const uint32_t u0 = (uint32_t)max(b0, 0) & 0xFFu, u1 = (uint32_t)max(b1, 0) & 0xFFu;
          *reinterpret_cast<uint16_t*>(sgen + C::OFF_PSF + 512 * pr + lane * 16 + quarter * 4 + 2 * (team & 1)) = (uint16_t)(u0 | (u1 << 8));
          fence_proxy_async_smem();
        } else {
          *meta = make_int2(E0, E1);
        }
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
      // time-out path: the issuers may have left with products or scale copies in flight; give them a bounded
      // time to finish before tensor memory and shared memory are given up
      for (int r = 0; r < 2; ++r)
        for (int spin = 0; spin < (1 << 14) && !mbar_try_wait(bar(BAR_DRAIN0 + r), 0); ++spin) {}
    }
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem, kTmemCols);
  }
}

// ------------------------------------------------------------------ dense FP4 issue-rate probe
__global__ void __launch_bounds__(128, 1) mma_peak_kernel(int iters, unsigned long long* cycles_out) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* sgen = smem_raw + (sbase - smem_u32(smem_raw));
  // A: 128 rows x 32 B, B: 128 rows x 32 B (one K64 slice each), scale atoms 2 x 512 B, all zero
  for (int i = threadIdx.x; i < (4096 + 4096 + 1024) / 4; i += 128) reinterpret_cast<uint32_t*>(sgen)[i] = 0;
  uint32_t* tslot = reinterpret_cast<uint32_t*>(sgen + 9216 + 64);
  volatile int* abortf = reinterpret_cast<volatile int*>(sgen + 9216 + 72);
  if (threadIdx.x == 0) { mbar_init(sbase + 9216, 1); *abortf = 0; fence_barrier_init(); }
  fence_proxy_async_smem();
  if ((threadIdx.x >> 5) == 0) { tmem_alloc(sbase + 9216 + 64, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tslot;
  if (threadIdx.x == 32) {
    tc_cp_32x128b_warpx4(tmem + 480, make_smem_desc(sbase + 8192, 16, 128, kSwzNone));
    tc_cp_32x128b_warpx4(tmem + 484, make_smem_desc(sbase + 8192 + 512, 16, 128, kSwzNone));
    const uint64_t ad = make_smem_desc(sbase, 16, 256, kSwz32), bd = make_smem_desc(sbase + 4096, 16, 256, kSwz32);
    const uint32_t idesc = make_idesc_fp4(128, 128, true, 0, 0);
    const long long t0 = clock64();
    for (int i = 0; i < iters; ++i) tc_mma_fp4_2x(tmem + 128 * (i & 1), ad, bd, idesc, tmem + 480, tmem + 484, 1);
    tc_commit(sbase + 9216);
    const bool ok = mbar_wait(sbase + 9216, 0, abortf);
    const long long t1 = clock64();
    if (ok) atomicMax(cycles_out, (unsigned long long)(t1 - t0));
  }
  tc_fence_before();
  __syncthreads();
  if ((threadIdx.x >> 5) == 0) { tc_fence_after(); tmem_dealloc(tmem, 512); }
}

// ------------------------------------------------------------------ bounded-wait self-test
// One warp waits on an mbarrier that nothing will ever complete, with a short limit, and must come
// back through the same time-out path the attention kernel uses (abort flag -> status word).
__global__ void __launch_bounds__(32, 1) bounded_wait_selftest_kernel(long long limit_cycles, int* status) {
  __shared__ __align__(8) uint64_t never;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) { mbar_init(smem_u32(&never), 1); abort_flag = 0; fence_barrier_init(); }
  __syncwarp();
  const bool ok = __all_sync(0xffffffffu, mbar_wait_limit(smem_u32(&never), 0, &abort_flag, limit_cycles));
  if (threadIdx.x == 0) *status = (!ok && abort_flag) ? FP4ATTN_ERR_TIMEOUT : FP4ATTN_OK;
}

// ------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static std::atomic<EncodeTiledFn> cached{nullptr};
  EncodeTiledFn fn = cached.load(std::memory_order_acquire);
  if (!fn) {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
    cached.store(fn, std::memory_order_release);
  }
  return fn;
}

// 2-D byte tensor [rows][row_bytes], box [box_rows][box_bytes], swizzle matching the box width
static bool make_map(CUtensorMap* m, const void* base, uint64_t row_bytes, uint64_t rows, uint32_t box_bytes,
                     uint32_t box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {row_bytes, rows};
  const cuuint64_t strides[1] = {row_bytes};
  const cuuint32_t box[2] = {box_bytes, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  const CUtensorMapSwizzle swz = box_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : box_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B;
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The four tensor maps of a launch depend only on the operand and output addresses and the shape, and encoding
// them costs more host time than launching a short kernel, so each host thread remembers the maps of its last
// few distinct calls (a map holds addresses and extents, no reference to the memory: a stale entry is harmless
// and is simply never matched again).
struct MapKey {
  const void *q, *k, *v, *o;
  int B, H, Hkv, N, D, v8;              // v8: V^T is E4M3 bytes (FP8 P/V route), not packed E2M1
  bool operator==(const MapKey& r) const {
    return q == r.q && k == r.k && v == r.v && o == r.o && B == r.B && H == r.H && Hkv == r.Hkv && N == r.N && D == r.D && v8 == r.v8;
  }
};
struct MapEntry {
  MapKey key;
  unsigned long long epoch;             // value of g_map_epoch when the entry was made; 0 = empty
  alignas(64) CUtensorMap tm[4];
};
constexpr int kMapCacheEntries = 8;
static std::atomic<unsigned long long> g_map_epoch{1};          // bumped by fp4attn_release: older entries are dead
static thread_local MapEntry t_maps[kMapCacheEntries];
static thread_local unsigned t_map_next = 0;
void drop_tensor_map_cache() { g_map_epoch.fetch_add(1, std::memory_order_acq_rel); }

template <int D>
static const CUtensorMap* tensor_maps(const fp4attn_operands* ops, void* O, int B, int H, int Hkv, int N, bool v8 = false) {
  constexpr int ROW_BYTES = D / 2;
  const MapKey key{ops->q, ops->k, ops->v, O, B, H, Hkv, N, D, v8 ? 1 : 0};
  const unsigned long long epoch = g_map_epoch.load(std::memory_order_acquire);
  for (int i = 0; i < kMapCacheEntries; ++i)
    if (t_maps[i].epoch == epoch && t_maps[i].key == key) return t_maps[i].tm;
  MapEntry& e = t_maps[t_map_next];
  e.epoch = 0;
  const uint64_t rows = (uint64_t)B * H * N, kv_rows = (uint64_t)B * Hkv * N;
  if (!make_map(&e.tm[0], ops->q, ROW_BYTES, rows, ROW_BYTES, BM) ||
      !make_map(&e.tm[1], ops->k, ROW_BYTES, kv_rows, ROW_BYTES, BS) ||
      !(v8 ? make_map(&e.tm[2], ops->v, (uint64_t)N, (uint64_t)B * Hkv * D, BS, D)
           : make_map(&e.tm[2], ops->v, (uint64_t)N / 2, (uint64_t)B * Hkv * D, BS / 2, D)) ||
      !make_map(&e.tm[3], O, (uint64_t)D * 2, rows, 128, 32))
    return nullptr;
  e.key = key;
  e.epoch = epoch;
  t_map_next = (t_map_next + 1) % kMapCacheEntries;
  return e.tm;
}

const CUtensorMap* attention_tensor_maps(int D, const fp4attn_operands* ops, void* O, int B, int H, int Hkv, int N) {
  return D == 128 ? tensor_maps<128>(ops, O, B, H, Hkv, N) : tensor_maps<64>(ops, O, B, H, Hkv, N);
}

const CUtensorMap* attention_tensor_maps_fp8v(int D, const fp4attn_operands* ops, void* O, int B, int H, int Hkv, int N) {
  return D == 128 ? tensor_maps<128>(ops, O, B, H, Hkv, N, true) : tensor_maps<64>(ops, O, B, H, Hkv, N, true);
}

template <int D, int NV, int PMAP, bool CAUSAL, int THR16, bool FIXREF = false>
static int launch_attn(const fp4attn_operands* ops, int B, int H, int N, AttnParams prm, cudaStream_t st) {
  const int Hkv = prm.Hkv;
  using C = Cfg<D, (NV != 0)>;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return FP4ATTN_ERR_CUDA;
  // the shared-memory opt-in is a per-device property of the function: set it once on every device used
  static std::atomic<bool> attr_set[kMaxDevices];
  if (dev < 0 || dev >= kMaxDevices) return FP4ATTN_ERR_CUDA;
  if (!attr_set[dev].load(std::memory_order_acquire)) {
    if (cudaFuncSetAttribute(attn_fwd_kernel<D, NV, PMAP, CAUSAL, THR16, FIXREF>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES) != cudaSuccess)
      return FP4ATTN_ERR_CUDA;
    attr_set[dev].store(true, std::memory_order_release);
  }
  const CUtensorMap* tm = tensor_maps<D>(ops, prm.O, B, H, Hkv, N);
  if (!tm) return FP4ATTN_ERR_CUDA;
  const unsigned grid = (unsigned)(prm.n_items < sms ? prm.n_items : sms);     // persistent: one CTA per SM
  attn_fwd_kernel<D, NV, PMAP, CAUSAL, THR16, FIXREF><<<grid, kAttnThreads, C::SMEM_BYTES, st>>>(tm[0], tm[1], tm[2], tm[3], prm);
  return cudaGetLastError() == cudaSuccess ? FP4ATTN_OK : FP4ATTN_ERR_CUDA;
}

int launch_attn_two_query(const fp4attn_operands* ops, int B, int H, int N, int d, int pmap, AttnParams prm, cudaStream_t st);
int launch_attn_fp8pv(const fp4attn_operands* ops, int B, int H, int N, int d, AttnParams prm, cudaStream_t st);

}  // namespace fp4attn

using namespace fp4attn;

extern "C" int fp4attn_fwd(const fp4attn_operands* ops, int B, int H, int N, int d, void* O, float* LSE,
                           int* device_status, fp4attn_stream_t stream) {
  if (!ops || !O || !ops->q || !ops->k || !ops->v || !ops->q_sf || !ops->k_sf) return FP4ATTN_ERR_INVALID_ARG;
  if (ops->pv_fmt != FP4ATTN_PV_E4M3 && !ops->v_sf) return FP4ATTN_ERR_INVALID_ARG;   // E4M3 V carries no block scales
  if (ops->qk_fmt != FP4ATTN_FMT_MXFP4 && ops->qk_fmt != FP4ATTN_FMT_NVFP4) return FP4ATTN_ERR_INVALID_ARG;
  if (ops->qk_fmt == FP4ATTN_FMT_NVFP4 && (!ops->q_G || !ops->k_G)) return FP4ATTN_ERR_INVALID_ARG;
  if (B <= 0 || H <= 0 || N <= 0 || d <= 0) return FP4ATTN_ERR_INVALID_ARG;
  if (!(d == 64 || d == 128) || N < 128 || N % 128 != 0) return FP4ATTN_ERR_UNSUPPORTED_SHAPE;
  if ((uint64_t)B * H * N >= (1ull << 31)) return FP4ATTN_ERR_UNSUPPORTED_SHAPE;
  if (!(ops->softmax_scale >= 0.f)) return FP4ATTN_ERR_INVALID_ARG;
  if (ops->p_map != FP4ATTN_PMAP_IDEAL && ops->p_map != FP4ATTN_PMAP_AFFINE && ops->p_map != FP4ATTN_PMAP_HYBRID)
    return FP4ATTN_ERR_INVALID_ARG;
  int pmap = ops->p_map;                                          // kernel instance: 0 ideal, 1 affine, 2..4 mixed patterns
  if (ops->p_map == FP4ATTN_PMAP_HYBRID) {
    pmap = ops->exact_pairs == 0x1111 ? 2 : ops->exact_pairs == 0x5555 ? 3 : ops->exact_pairs == 0x7777 ? 4 : -1;
    if (pmap < 0 || ops->causal || ops->seq_len) return FP4ATTN_ERR_INVALID_ARG;    // three patterns, no masks
  }
  if (ops->p_scale_rule != FP4ATTN_PSCALE_CEIL && ops->p_scale_rule != FP4ATTN_PSCALE_THR16 && ops->p_scale_rule != FP4ATTN_PSCALE_MSE)
    return FP4ATTN_ERR_INVALID_ARG;
  if (ops->p_scale_rule == FP4ATTN_PSCALE_MSE &&
      (ops->p_map != FP4ATTN_PMAP_IDEAL || ops->g_per_head || ops->schedule != FP4ATTN_SCHEDULE_ONE_QUERY || ops->pv_fmt != FP4ATTN_PV_MXFP4))
    return FP4ATTN_ERR_INVALID_ARG;                                 // ideal map, one factor per tensor, one-query schedule
  if (ops->g_per_head != 0 && ops->g_per_head != 1) return FP4ATTN_ERR_INVALID_ARG;
  if (ops->g_per_head && ops->p_map == FP4ATTN_PMAP_HYBRID) return FP4ATTN_ERR_INVALID_ARG;   // ideal and affine maps only
  if (ops->kv_heads < 0 || (ops->kv_heads > 0 && H % ops->kv_heads != 0) || (ops->causal != 0 && ops->causal != 1))
    return FP4ATTN_ERR_INVALID_ARG;
  if (ops->p_map != FP4ATTN_PMAP_IDEAL && !(ops->affine_a >= 0.f && ops->affine_a < 16.f && fabsf(ops->affine_b) < 16.f))
    return FP4ATTN_ERR_INVALID_ARG;
  const uintptr_t a128 = (uintptr_t)ops->q | (uintptr_t)ops->k | (uintptr_t)ops->v | (uintptr_t)ops->q_sf |
                         (uintptr_t)ops->k_sf | (uintptr_t)ops->v_sf;
  if ((a128 & 127) || ((uintptr_t)O & 15) || ((uintptr_t)LSE & 3)) return FP4ATTN_ERR_ALIGNMENT;
  int rc = check_device_sm100();
  if (rc != FP4ATTN_OK) return rc;
  AttnParams prm;
  prm.q_sf = (const uint8_t*)ops->q_sf; prm.k_sf = (const uint8_t*)ops->k_sf; prm.v_sf = (const uint8_t*)ops->v_sf;
  prm.q_G = ops->q_G; prm.k_G = ops->k_G;
  prm.O = (__nv_bfloat16*)O; prm.LSE = LSE; prm.status = device_status;
  prm.N = N; prm.stages = N / BS; prm.n_items = B * H * (N / BM);
  prm.BH = B * H;
  prm.recip_qtiles = (N / BM) > 1 ? ~0ull / (unsigned long long)(N / BM) + 1 : 0;
  prm.recip_bh = prm.BH > 1 ? ~0ull / (unsigned long long)prm.BH + 1 : 0;
  prm.causal = ops->causal ? 1 : 0;
  prm.seq_len = ops->seq_len;
  prm.recip_h = H > 1 ? ~0ull / (unsigned long long)H + 1 : 0;
  const bool masked = prm.causal || prm.seq_len;                  // kernels that mask an item's last stage
  prm.H = H;
  prm.Hkv = ops->kv_heads > 0 ? ops->kv_heads : H;
  const float scale = ops->softmax_scale > 0.f ? ops->softmax_scale : (float)(1.0 / sqrt((double)d));
  prm.c_base = 1.4426950408889634f * scale;                        // fl32(log2e_32 * scale_32)
  cudaStream_t st = (cudaStream_t)stream;
  const bool nv = ops->qk_fmt == FP4ATTN_FMT_NVFP4;
  prm.aff_a = ops->affine_a != 0.f ? ops->affine_a : 1.5f;         // the paper's generic `fast` fit
  prm.aff_b = ops->affine_a != 0.f ? ops->affine_b : 1.2f;
  prm.thr16 = ops->p_scale_rule == FP4ATTN_PSCALE_THR16;
  if (ops->schedule != FP4ATTN_SCHEDULE_ONE_QUERY && ops->schedule != FP4ATTN_SCHEDULE_TWO_QUERY) return FP4ATTN_ERR_INVALID_ARG;
  if (ops->pv_fmt != FP4ATTN_PV_MXFP4 && ops->pv_fmt != FP4ATTN_PV_E4M3) return FP4ATTN_ERR_INVALID_ARG;
  if (ops->seq_len && ops->schedule != FP4ATTN_SCHEDULE_ONE_QUERY) return FP4ATTN_ERR_INVALID_ARG;
  if (((uintptr_t)ops->seq_len & 3) != 0) return FP4ATTN_ERR_ALIGNMENT;
  if (ops->row_reference != FP4ATTN_REFERENCE_RUNNING && ops->row_reference != FP4ATTN_REFERENCE_FIXED) return FP4ATTN_ERR_INVALID_ARG;
  prm.ref_fixed = ops->fixed_reference;
  if (ops->row_reference == FP4ATTN_REFERENCE_FIXED) {
    // the shiftless path: ideal or affine map, ceiling rule, one factor per tensor, one query tile, FP4 P and V
    if (pmap > 1 || ops->p_scale_rule != FP4ATTN_PSCALE_CEIL || ops->g_per_head || ops->schedule != FP4ATTN_SCHEDULE_ONE_QUERY ||
        ops->pv_fmt != FP4ATTN_PV_MXFP4 || ops->fixed_reference < -1000 || ops->fixed_reference > 1000)
      return FP4ATTN_ERR_INVALID_ARG;
    const int sel = (d == 128 ? 8 : 0) | (nv ? 4 : 0) | (pmap ? 2 : 0) | (masked ? 1 : 0);
    switch (sel) {
      case 0: return launch_attn<64, 0, 0, false, 0, true>(ops, B, H, N, prm, st);
      case 1: return launch_attn<64, 0, 0, true, 0, true>(ops, B, H, N, prm, st);
      case 2: return launch_attn<64, 0, 1, false, 0, true>(ops, B, H, N, prm, st);
      case 3: return launch_attn<64, 0, 1, true, 0, true>(ops, B, H, N, prm, st);
      case 4: return launch_attn<64, 1, 0, false, 0, true>(ops, B, H, N, prm, st);
      case 5: return launch_attn<64, 1, 0, true, 0, true>(ops, B, H, N, prm, st);
      case 6: return launch_attn<64, 1, 1, false, 0, true>(ops, B, H, N, prm, st);
      case 7: return launch_attn<64, 1, 1, true, 0, true>(ops, B, H, N, prm, st);
      case 8: return launch_attn<128, 0, 0, false, 0, true>(ops, B, H, N, prm, st);
      case 9: return launch_attn<128, 0, 0, true, 0, true>(ops, B, H, N, prm, st);
      case 10: return launch_attn<128, 0, 1, false, 0, true>(ops, B, H, N, prm, st);
      case 11: return launch_attn<128, 0, 1, true, 0, true>(ops, B, H, N, prm, st);
      case 12: return launch_attn<128, 1, 0, false, 0, true>(ops, B, H, N, prm, st);
      case 13: return launch_attn<128, 1, 0, true, 0, true>(ops, B, H, N, prm, st);
      case 14: return launch_attn<128, 1, 1, false, 0, true>(ops, B, H, N, prm, st);
      default: return launch_attn<128, 1, 1, true, 0, true>(ops, B, H, N, prm, st);
    }
  }
  if (ops->pv_fmt == FP4ATTN_PV_E4M3) return launch_attn_fp8pv(ops, B, H, N, d, prm, st);
  if (ops->schedule == FP4ATTN_SCHEDULE_TWO_QUERY) return launch_attn_two_query(ops, B, H, N, d, pmap, prm, st);
  if (ops->p_scale_rule == FP4ATTN_PSCALE_MSE) {
    const int sel = (d == 128 ? 4 : 0) | (nv ? 2 : 0) | (masked ? 1 : 0);
    switch (sel) {
      case 0: return launch_attn<64, 0, 0, false, 2>(ops, B, H, N, prm, st);
      case 1: return launch_attn<64, 0, 0, true, 2>(ops, B, H, N, prm, st);
      case 2: return launch_attn<64, 1, 0, false, 2>(ops, B, H, N, prm, st);
      case 3: return launch_attn<64, 1, 0, true, 2>(ops, B, H, N, prm, st);
      case 4: return launch_attn<128, 0, 0, false, 2>(ops, B, H, N, prm, st);
      case 5: return launch_attn<128, 0, 0, true, 2>(ops, B, H, N, prm, st);
      case 6: return launch_attn<128, 1, 0, false, 2>(ops, B, H, N, prm, st);
      default: return launch_attn<128, 1, 0, true, 2>(ops, B, H, N, prm, st);
    }
  }
  // one kernel instance per (d, Q/K format, P map, mask, P scale rule): nothing of these is decided at run time
  const bool per_head = nv && ops->g_per_head;
  const int shape = (d == 128 ? 2 : 0) | (nv ? 1 : 0);
#define FP4ATTN_SHAPES(PM_, CAU_, THR_)                                                  \
  if (per_head && PM_ <= 1) {                                                            \
    if (d == 64) return launch_attn<64, 2, (PM_ <= 1 ? PM_ : 0), CAU_, THR_>(ops, B, H, N, prm, st);   \
    return launch_attn<128, 2, (PM_ <= 1 ? PM_ : 0), CAU_, THR_>(ops, B, H, N, prm, st); \
  }                                                                                      \
  switch (shape) {                                                                       \
    case 0: return launch_attn<64, 0, PM_, CAU_, THR_>(ops, B, H, N, prm, st);           \
    case 1: return launch_attn<64, 1, PM_, CAU_, THR_>(ops, B, H, N, prm, st);           \
    case 2: return launch_attn<128, 0, PM_, CAU_, THR_>(ops, B, H, N, prm, st);          \
    default: return launch_attn<128, 1, PM_, CAU_, THR_>(ops, B, H, N, prm, st);         \
  }
#define FP4ATTN_MASKS(PM_)                                         \
  if (masked) {                                                    \
    if (prm.thr16) { FP4ATTN_SHAPES(PM_, true, true) }             \
    else           { FP4ATTN_SHAPES(PM_, true, false) }            \
  } else {                                                         \
    if (prm.thr16) { FP4ATTN_SHAPES(PM_, false, true) }            \
    else           { FP4ATTN_SHAPES(PM_, false, false) }           \
  }
#define FP4ATTN_NONCAUSAL(PM_)                                     \
  if (prm.thr16) { FP4ATTN_SHAPES(PM_, false, true) }              \
  else           { FP4ATTN_SHAPES(PM_, false, false) }
  switch (pmap) {
    case 0: FP4ATTN_MASKS(0)
    case 1: FP4ATTN_MASKS(1)
    case 2: FP4ATTN_NONCAUSAL(2)
    case 3: FP4ATTN_NONCAUSAL(3)
    default: FP4ATTN_NONCAUSAL(4)
  }
#undef FP4ATTN_SHAPES
#undef FP4ATTN_MASKS
#undef FP4ATTN_NONCAUSAL
}

extern "C" int fp4attn_mma_peak_probe(int iters, unsigned long long* cycles_out, fp4attn_stream_t stream) {
  if (iters <= 0 || !cycles_out) return FP4ATTN_ERR_INVALID_ARG;
  int rc = check_device_sm100();
  if (rc != FP4ATTN_OK) return rc;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return FP4ATTN_ERR_CUDA;
  // > 114 KB of dynamic shared memory keeps it at one CTA per SM
  const int smem = 120 * 1024;
  if (cudaFuncSetAttribute(mma_peak_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)
    return FP4ATTN_ERR_CUDA;
  if (cudaMemsetAsync(cycles_out, 0, sizeof(unsigned long long), (cudaStream_t)stream) != cudaSuccess) return FP4ATTN_ERR_CUDA;
  mma_peak_kernel<<<sms, 128, smem, (cudaStream_t)stream>>>(iters, cycles_out);
  return cudaGetLastError() == cudaSuccess ? FP4ATTN_OK : FP4ATTN_ERR_CUDA;
}

extern "C" int fp4attn_selftest_bounded_wait(long long limit_cycles, int* device_status, fp4attn_stream_t stream) {
  if (!device_status || limit_cycles <= 0 || limit_cycles > (1ll << 31)) return FP4ATTN_ERR_INVALID_ARG;
  int rc = check_device_sm100();
  if (rc != FP4ATTN_OK) return rc;
  bounded_wait_selftest_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(limit_cycles, device_status);
  return cudaGetLastError() == cudaSuccess ? FP4ATTN_OK : FP4ATTN_ERR_CUDA;
}
