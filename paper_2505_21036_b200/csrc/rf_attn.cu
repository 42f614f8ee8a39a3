// Pattern-masked FlashAttention forward on tcgen05 / TMEM / TMA (Eq. 1-2 with the masks of Sec. 3.2).
//
// One CTA owns two adjacent 128-row query tiles of one head (two "streams") and walks the union of
// their KV-tile lists, so every K/V tile fetched by TMA feeds up to two S = Q K^T and two O += P V
// contractions.  Warp roles:
//   warps 0-3  softmax of stream 0   (one thread per query row, TMEM lane = row)
//   warps 4-7  softmax of stream 1
//   warp  8    TMA producer: Q once, then K and V tiles into two shared-memory rings (V of tile u and K of
//              tile u + 1 as a pair under one full / one empty mbarrier)
//   warp  9    MMA issuer: tcgen05.mma, accumulators in TMEM (S0, S1, O0, O1)
//   (warps 10-11 only fill the third warpgroup, which hands its registers to the softmax warpgroups)
// Per listed tile and stream: S lands in TMEM, the softmax warps read their rows (tcgen05.ld), keep a
// running maximum and sum in fp32, write P as packed bf16 back into TMEM (tcgen05.st: on top of the S
// columns at D = 96 / 128, into spare columns at D = 64) and the MMA warp multiplies it with V straight
// from TMEM.  The running maximum is raised lazily (see kSumLimit), in which case the softmax warp itself
// rescales its rows of O in TMEM; the final O / l and the log-sum-exp do not depend on it.
// PARTIAL tiles apply the exact element mask of the head's pattern; FULL tiles skip it.
#include "rf_attn_common.cuh"

namespace {

using namespace sm100;
using namespace rf_attn;

constexpr int kThreads = kWsThreads;        // 3 warpgroups: softmax 0, softmax 1, {TMA, MMA, 2 idle warps}
constexpr int kTmaWarp = 8, kMmaWarp = 9;
// Lazy rescaling of the running maximum.  A tile's weights are taken as 2^(score - running maximum) and accepted
// while their row sum stays within kSumLimit; beyond it the row's maximum is raised.  bf16 P and the fp32 sums
// carry the same relative precision at every exponent and 2^32 times the longest row is far from overflow, so
// O / l and the log-sum-exp do not depend on how stale the running maximum is.
constexpr float kSumLimit = 4294967296.0f;  // 2^32
constexpr float kRaiseMargin = 8.0f;        // log2 units: on the slow path, rows this far above their maximum raise it
constexpr float kLazyRaise = 32.0f;         // log2 units: where the exact tile maximum is at hand (D = 64)

struct Maps { CUtensorMap m[8]; };

template <int D>
struct Cfg {
  static constexpr int KB = (D + 63) / 64;            // 64-column (128-byte) blocks per row
  // first column of the second block.  D = 96 is fetched as columns [0,64) and [64,128): the TMA box
  // reaches past the tensor's 96 columns and the missing ones arrive as zeros; they are never read
  // (Q K^T runs 6 k-steps, P V is one N = 96 MMA per k-step over one and a half 64-column blocks)
  static constexpr int COL1 = 64;
  static constexpr uint32_t BLK = 128 * 128;          // bytes of one 128-row x 64-col bf16 block
  static constexpr uint32_t TILE = KB * BLK;          // bytes of one 128-row tile
  // D = 64 leaves 128 TMEM columns unused (O is only 64 wide), room for P of both streams in columns of its
  // own: the S accumulator is then free again as soon as the softmax warps have read it, and the next tile's
  // scores are computed during the softmax of the current one.  At D = 96 / 128 TMEM is full and P lives on
  // top of the S columns it was computed from.
  static constexpr bool S_EARLY = D == 64;
  static constexpr int NK = D == 64 ? 3 : 2;          // K ring depth
  static constexpr int NV = D == 64 ? 3 : 2;          // V ring depth
  // byte offset, inside a tile, of the 16 columns of k-step ks of the Q K^T contraction
  static __host__ __device__ constexpr uint32_t koff(int ks) {
    return ks < 4 ? (uint32_t)ks * 32u : BLK + (uint32_t)(ks - 4) * 32u;
  }
  static constexpr uint32_t Q = 0;
  static constexpr uint32_t K0 = Q + 2 * TILE;
  static constexpr uint32_t V0 = K0 + NK * TILE;
  static constexpr uint32_t BAR = V0 + NV * TILE;
  // barrier slots (8 bytes each)
  // V of tile u and K of tile u + 1 travel as a pair: they are wanted in the same iteration of the MMA warp and
  // released by it together, so one full and one empty barrier per pair (B_F, B_E) serve both; K of the first
  // tile has its own two (B_K0 landed, B_K0E consumed).
  static_assert(NK == NV, "K and V rings advance together");
  static constexpr int NP = NV;
  static constexpr int B_Q = 0, B_K0 = 1, B_K0E = 2, B_F = 3, B_E = B_F + NP, B_SF = B_E + NP,
                       B_PF = B_SF + 2, B_OF = B_PF + 2, B_SE = B_OF + 2 /* S read, S_EARLY only */, B_COUNT = B_SE + 2;
  static constexpr uint32_t MISC = BAR + 8 * ((B_COUNT + 7) / 8 * 8);
  static constexpr uint32_t TOTAL = MISC + 64;
  static constexpr uint32_t ALLOC = TOTAL + 1024;     // slack for manual 1024-byte alignment
  // TMEM columns
  static constexpr uint32_t S_COL0 = 0, S_COL1 = 128, O_COL0 = 256, O_COL1 = S_EARLY ? 320 : 384, TMEM_COLS = 512;
  static constexpr uint32_t P_COL0 = S_EARLY ? 384 : S_COL0, P_COL1 = S_EARLY ? 448 : S_COL1;   // packed bf16, 64 columns
};

template <int D>
__global__ void __launch_bounds__(kThreads, 1) rf_attn_kernel(const __grid_constant__ Maps maps, const RfAttnArgs a) {
  using C = Cfg<D>;
  constexpr int KB = C::KB;
  constexpr uint32_t IDESC_S = idesc_bf16(BM, BN, 0);
  constexpr uint32_t IDESC_PV = idesc_bf16(BM, D, 1);

  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
  auto bar = [&](int slot) -> uint32_t { return base + C::BAR + 8u * slot; };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + C::MISC);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + C::MISC + 8);

  RfGeom g = a.g;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int bh = blockIdx.y;
  const int qt0 = 2 * blockIdx.x, qt1 = qt0 + 1;

  int cls = RF_DENSE;
  if (a.head_class != nullptr) {
    cls = a.head_class[bh];
    if (cls < 0 || cls > 3) {
      if (tid == 0) rf_report(a.dev_status, RF_ERR_INVALID_ARG);
      cls = RF_DENSE;
    }
  }
  if (a.head_window != nullptr) {   // dynamic bandwidth: this head's own window
    const int w = a.head_window[bh];
    if (cls == RF_SPATIAL && w >= 0) g.wf = min(w, g.T);     // past the extent: same mask, no overflow
    if (cls == RF_TEMPORAL && w >= 0) g.ws = min(w, g.S);
  }
  const bool perm = cls == RF_TEMPORAL && g.permute;
  const bool tex = cls == RF_TEXTURAL;
  const CUtensorMap* map_q = &maps.m[perm ? 3 : 0];
  const CUtensorMap* map_k = &maps.m[perm ? 4 : (tex ? 6 : 1)];
  const CUtensorMap* map_v = &maps.m[perm ? 5 : (tex ? 7 : 2)];

  Lists L;
  L.lkv = rf_kv_len(g, cls);
  L.listed = a.head_class != nullptr;
  if (L.listed) {
    L.n0 = a.count[(size_t)bh * g.nQ + qt0];
    L.n1 = qt1 < g.nQ ? a.count[(size_t)bh * g.nQ + qt1] : 0;
    // a schedule that was not built for this shape could hold any count: the checking build refuses to walk past a row
    if (!rf_in_bounds(L.n0, g.nKmax + 1, a.dev_status)) L.n0 = 0;
    if (!rf_in_bounds(L.n1, g.nKmax + 1, a.dev_status)) L.n1 = 0;
    L.l0 = a.kv_tile + ((size_t)bh * g.nQ + qt0) * g.nKmax;
    L.l1 = a.kv_tile + ((size_t)bh * g.nQ + min(qt1, g.nQ - 1)) * g.nKmax;
  } else {
    L.n0 = rf_cdiv(L.lkv, BN);
    L.n1 = qt1 < g.nQ ? L.n0 : 0;
    L.l0 = L.l1 = nullptr;
  }

  if (tid == 0) {
    mbar_init(bar(C::B_Q), 1);
    mbar_init(bar(C::B_K0), 1);
    mbar_init(bar(C::B_K0E), 1);
    for (int s = 0; s < C::NP; ++s) { mbar_init(bar(C::B_F + s), 1); mbar_init(bar(C::B_E + s), 1); }
    for (int j = 0; j < 2; ++j) {
      mbar_init(bar(C::B_SF + j), 1);
      mbar_init(bar(C::B_PF + j), 4);   // one arrival per softmax warp
      mbar_init(bar(C::B_OF + j), 1);
      mbar_init(bar(C::B_SE + j), 4);
    }
    *abort_flag = 0;
    mbar_init_fence();
  }
  if (warp == kTmaWarp) {
    if (lane == 0) { prefetch_tmap(map_q); prefetch_tmap(map_k); prefetch_tmap(map_v); }
    __syncwarp();
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), C::TMEM_COLS);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const WaitCtx wc{abort_flag, a.dev_status};

  if (warp >= 8) {
  RF_SETMAXNREG_DEC();
  if (warp == kTmaWarp) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      mbar_expect_tx(bar(C::B_Q), 2 * C::TILE);
#pragma unroll
      for (int j = 0; j < 2; ++j)
#pragma unroll
        for (int kb = 0; kb < KB; ++kb)
          tma_load_3d(base + C::Q + j * C::TILE + kb * C::BLK, map_q, kb * C::COL1, (qt0 + j) * BM, bh, bar(C::B_Q));
      Merge mg;
      mg.start(L);
      int tile, uses, ntile = 0;
      bool has = mg.next(L, tile, uses);
      if (has) {
        mbar_expect_tx(bar(C::B_K0), C::TILE);
#pragma unroll
        for (int kb = 0; kb < KB; ++kb)
          tma_load_3d(base + C::K0 + kb * C::BLK, map_k, kb * C::COL1, tile * BN, bh, bar(C::B_K0));
      }
      for (int u = 0; has; ++u) {
        const bool has_nxt = mg.next(L, ntile, uses);
        const int ps = u % C::NP, ksn = (u + 1) % C::NK;
        // pair u reuses the V slot of pair u - NP and the K slot that pair filled; the first tile's K slot
        // comes round at u = NK - 1
        if (u >= C::NP) mbar_wait(bar(C::B_E + ps), ((u / C::NP) - 1) & 1, wc);
        else if (has_nxt && ksn == 0) mbar_wait(bar(C::B_K0E), 0, wc);
        mbar_expect_tx(bar(C::B_F + ps), has_nxt ? 2 * C::TILE : C::TILE);
#pragma unroll
        for (int kb = 0; kb < KB; ++kb)
          tma_load_3d(base + C::V0 + ps * C::TILE + kb * C::BLK, map_v, kb * C::COL1, tile * BN, bh, bar(C::B_F + ps));
        if (has_nxt) {
#pragma unroll
          for (int kb = 0; kb < KB; ++kb)
            tma_load_3d(base + C::K0 + ksn * C::TILE + kb * C::BLK, map_k, kb * C::COL1, ntile * BN, bh, bar(C::B_F + ps));
        }
        has = has_nxt;
        tile = ntile;
      }
    }
  } else if (warp == kMmaWarp) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      // Descriptors differ only in their 14-bit start-address field: keep the constant words in
      // registers and add the byte offset (>> 4) per k-step.
      constexpr uint32_t DESC_HI = (1024u >> 4) | (1u << 14) | (2u << 29);      // SBO 1024 B, version 1, 128B swizzle
      constexpr uint32_t LO_KMAJOR = 1u << 16;                                    // LBO field unused for K-major
      constexpr uint32_t LO_VMAJOR = (C::BLK >> 4) << 16;                         // LBO = one 64-column block
      auto desc = [](uint32_t lo) -> uint64_t { return ((uint64_t)DESC_HI << 32) | lo; };
      const uint32_t q_lo = ((base + C::Q) >> 4) | LO_KMAJOR, k_lo = ((base + C::K0) >> 4) | LO_KMAJOR;
      const uint32_t v_lo = ((base + C::V0) >> 4) | LO_VMAJOR;
      auto issue_s = [&](int j, int ks) {
        const uint32_t a0 = q_lo + j * (C::TILE >> 4), b0 = k_lo + ks * (C::TILE >> 4);
        // the accumulate flag is a compile-time constant: the issuing thread blocks on every MMA, so each
        // instruction between two of them is idle tensor time
        const uint32_t t_d = tmem_base + (j ? C::S_COL1 : C::S_COL0);
        mma_ss_c<false>(t_d, desc(a0), desc(b0), IDESC_S);
#pragma unroll
        for (int k = 1; k < D / 16; ++k)
          mma_ss_c<true>(t_d, desc(a0 + (C::koff(k) >> 4)), desc(b0 + (C::koff(k) >> 4)), IDESC_S);
        tc_commit(bar(C::B_SF + j));
      };
      auto issue_pv = [&](int j, int vs, bool first) {
        const uint32_t b0 = v_lo + vs * (C::TILE >> 4);
        const uint32_t t_p = tmem_base + (j ? C::P_COL1 : C::P_COL0), t_o = tmem_base + (j ? C::O_COL1 : C::O_COL0);
        mma_ts(t_o, t_p, desc(b0), IDESC_PV, !first);
#pragma unroll
        for (int k = 1; k < BN / 16; ++k)
          mma_ts_c<true>(t_o, t_p + k * 8, desc(b0 + k * (2048 >> 4)), IDESC_PV);
        tc_commit(bar(C::B_OF + j));
      };
      Merge mg;
      mg.start(L);
      int cur_tile, cur_uses, nxt_tile = 0, nxt_uses = 0;
      bool has_cur = mg.next(L, cur_tile, cur_uses);
      int pv_cnt[2] = {0, 0};
      int s_cnt[2] = {0, 0};   // S_EARLY: S tiles issued per stream
      mbar_wait(bar(C::B_Q), 0, wc);
      if (has_cur) {
        mbar_wait(bar(C::B_K0), 0, wc);
        tc_fence_after();
        if (cur_uses & 1) { issue_s(0, 0); ++s_cnt[0]; }
        if (cur_uses & 2) { issue_s(1, 0); ++s_cnt[1]; }
        tc_commit(bar(C::B_K0E));
      }
      for (int u = 0; has_cur; ++u) {
        const bool has_nxt = mg.next(L, nxt_tile, nxt_uses);
        const int vs = u % C::NV, ksn = (u + 1) % C::NK;
        // the TMA barrier first (V of this tile and K of the next): the data has normally landed long ago, and
        // checking here keeps it out of the gap between a stream's P arriving and its MMAs being issued
        mbar_wait(bar(C::B_F + vs), (u / C::NP) & 1, wc);
        if constexpr (C::S_EARLY) {
          // Per stream: the next tile's scores (S is free as soon as the softmax warps have read the current
          // one), then O += P V of the current tile.  Stream 1's next scores are thus only issued once stream 0
          // has delivered its P: the two streams settle half a tile apart and take turns at the MUFU unit
          // instead of sitting in their exponentials at the same time.
#pragma unroll
          for (int j = 0; j < 2; ++j) {
            if (has_nxt && (nxt_uses & (1 << j))) {
              mbar_wait(bar(C::B_SE + j), (s_cnt[j] - 1) & 1, wc);
              tc_fence_after();
              issue_s(j, ksn);
              ++s_cnt[j];
            }
            if (cur_uses & (1 << j)) {
              mbar_wait(bar(C::B_PF + j), pv_cnt[j] & 1, wc);
              tc_fence_after();
              issue_pv(j, vs, pv_cnt[j] == 0);
              ++pv_cnt[j];
            }
          }
        } else {
#pragma unroll
          for (int j = 0; j < 2; ++j) {
            if (cur_uses & (1 << j)) {
              mbar_wait(bar(C::B_PF + j), pv_cnt[j] & 1, wc);
              tc_fence_after();
              issue_pv(j, vs, pv_cnt[j] == 0);
              ++pv_cnt[j];
            }
            if (has_nxt && (nxt_uses & (1 << j))) issue_s(j, ksn);
          }
        }
        tc_commit(bar(C::B_E + vs));
        has_cur = has_nxt;
        cur_tile = nxt_tile;
        cur_uses = nxt_uses;
      }
    }
  }
  } else {
    RF_SETMAXNREG_INC();
    // ------------------------------------------------------------ softmax + epilogue, one thread per query row
    const int j = warp >> 2;                       // stream
    const int row_in_tile = tid & 127;
    const int r = (qt0 + j) * BM + row_in_tile;    // query slot in the head's coordinate space
    const int n = j == 0 ? L.n0 : L.n1;
    const uint32_t lane_sel = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t t_s = tmem_base + lane_sel + (j ? C::S_COL1 : C::S_COL0);
    const uint32_t t_o = tmem_base + lane_sel + (j ? C::O_COL1 : C::O_COL0);
    const RowMask rmask = make_row_mask(g, cls, min(r, g.N - 1));
    const float sc = a.scale_log2;
    float m_run = -INFINITY;   // running maximum, log2 domain (score * sc)
    float l_run = 0.f;         // sum of the weights as rounded to bf16, the ones P V multiplies: normalises O
    float l_exact = 0.f;       // sum of the unrounded weights: the log-sum-exp

    for (int it = 0; it < n; ++it) {
      const uint32_t entry = L.entry(j, it);
      const bool partial = (entry & RF_PARTIAL_BIT) != 0;
      const int u0 = (int)(entry & ~RF_PARTIAL_BIT) * BN;
      mbar_wait(bar(C::B_SF + j), it & 1, wc);
      tc_fence_after();
      if constexpr (C::S_EARLY) {
        // S into registers and the accumulator handed back at once; P goes to TMEM columns of its own.
        uint32_t s[128];
        {
          uint32_t(&s0)[32] = *reinterpret_cast<uint32_t(*)[32]>(&s[0]);
          uint32_t(&s1)[32] = *reinterpret_cast<uint32_t(*)[32]>(&s[32]);
          uint32_t(&s2)[32] = *reinterpret_cast<uint32_t(*)[32]>(&s[64]);
          uint32_t(&s3)[32] = *reinterpret_cast<uint32_t(*)[32]>(&s[96]);
          tmem_ld32(t_s, s0);
          tmem_ld32(t_s + 32, s1);
          tmem_ld32(t_s + 64, s2);
          tmem_ld32(t_s + 96, s3);
          tc_wait_ld();
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(C::B_SE + j));
        if (partial) {
          uint32_t w[4];
          rmask.tile_bits(u0, w);
#pragma unroll
          for (int c = 0; c < 128; ++c)
            if (!((w[c >> 5] >> (c & 31)) & 1u)) s[c] = 0xff800000u;  // -inf
        }
        // The scores are gone from TMEM, so the exact row maximum comes first and the exponentials are
        // taken once; the running maximum is raised only when the tile exceeds it by kLazyRaise.
        float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
        for (int c = 0; c < 128; c += 4) {
          mx0 = fmaxf(mx0, fmaxf(__uint_as_float(s[c]), __uint_as_float(s[c + 1])));
          mx1 = fmaxf(mx1, fmaxf(__uint_as_float(s[c + 2]), __uint_as_float(s[c + 3])));
        }
        const float m_tile = fmaxf(mx0, mx1) * sc;
        const bool raise = m_tile > m_run + kLazyRaise || (m_run == -INFINITY && m_tile > -INFINITY);
        const bool any_raise = __any_sync(0xffffffffu, raise);
        float alpha = 1.f;
        if (raise) {
          alpha = ex2(m_run - m_tile);   // 0 when m_run = -inf
          m_run = m_tile;
          l_run *= alpha;
          l_exact *= alpha;
        }
        // P V of the previous tile reads the P columns this tile is about to overwrite, and O may only be
        // rescaled once everything issued into it has landed.  The wait sits in front of the P store (the
        // exponentials of this tile run under the previous tile's P V); it also keeps this stream at most
        // one tile ahead of the MMA warp, which tracks the P barrier by phase parity.
        bool o_landed = it == 0;
        if (it > 0 && any_raise) {
          mbar_wait(bar(C::B_OF + j), (it - 1) & 1, wc);
          o_landed = true;
          {
            tc_fence_after();
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
              uint32_t v[32];
              tmem_ld32(t_o + c * 32, v);
              tc_wait_ld();
#pragma unroll
              for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(__uint_as_float(v[i]) * alpha);
              tmem_st32(t_o + c * 32, v);
            }
            tc_wait_st();
            tc_fence_before();
          }
        }
        const float m_use = m_run == -INFINITY ? 0.f : m_run;
        const float2 sc2 = make_float2(sc, sc), mneg = make_float2(-m_use, -m_use);
        float2 la = make_float2(0.f, 0.f), lb = make_float2(0.f, 0.f);
        uint32_t pk[64];
#pragma unroll
        for (int c = 0; c < 128; c += 4) {
          float2 e0 = __ffma2_rn(make_float2(__uint_as_float(s[c]), __uint_as_float(s[c + 1])), sc2, mneg);
          float2 e1 = __ffma2_rn(make_float2(__uint_as_float(s[c + 2]), __uint_as_float(s[c + 3])), sc2, mneg);
          e0.x = ex2(e0.x); e0.y = ex2(e0.y);
          e1.x = ex2(e1.x); e1.y = ex2(e1.y);
          pk[c / 2] = pack_bf16(e0.x, e0.y);
          pk[c / 2 + 1] = pack_bf16(e1.x, e1.y);
          la = __fadd2_rn(la, __fadd2_rn(e0, e1));
          lb = __fadd2_rn(lb, __fadd2_rn(unpack_bf16(pk[c / 2]), unpack_bf16(pk[c / 2 + 1])));
        }
        l_exact += la.x + la.y;
        l_run += lb.x + lb.y;
        if (!o_landed) mbar_wait(bar(C::B_OF + j), (it - 1) & 1, wc);
        {
          const uint32_t t_p = tmem_base + lane_sel + (j ? C::P_COL1 : C::P_COL0);
          uint32_t(&p0)[32] = *reinterpret_cast<uint32_t(*)[32]>(&pk[0]);
          uint32_t(&p1)[32] = *reinterpret_cast<uint32_t(*)[32]>(&pk[32]);
          tmem_st32(t_p, p0);
          tmem_st32(t_p + 32, p1);
          tc_wait_st();
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(C::B_PF + j));
        continue;
      }
      // Exponentials are taken against the running maximum of the previous tiles, without looking at the
      // tile's own maximum: all weights are non-negative, so a row sum within kSumLimit proves that none
      // of them left the safe range.  Only if some row's sum does not (its maximum grew by more than
      // ~2^25; rare after a row's first tile) is the exact tile maximum taken from the scores, which are
      // still in TMEM because P has not been stored yet, the running maximum raised, O rescaled and the
      // pass repeated.
      uint32_t pk[64];
#pragma unroll 1
      for (int pass = 0; pass < 2; ++pass) {
        uint32_t s[128];
        {
          uint32_t(&s0)[32] = *reinterpret_cast<uint32_t(*)[32]>(&s[0]);
          uint32_t(&s1)[32] = *reinterpret_cast<uint32_t(*)[32]>(&s[32]);
          uint32_t(&s2)[32] = *reinterpret_cast<uint32_t(*)[32]>(&s[64]);
          uint32_t(&s3)[32] = *reinterpret_cast<uint32_t(*)[32]>(&s[96]);
          tmem_ld32(t_s, s0);
          tmem_ld32(t_s + 32, s1);
          tmem_ld32(t_s + 64, s2);
          tmem_ld32(t_s + 96, s3);
          tc_wait_ld();
        }
        if (partial) {
          uint32_t w[4];
          rmask.tile_bits(u0, w);
#pragma unroll
          for (int c = 0; c < 128; ++c)
            if (!((w[c >> 5] >> (c & 31)) & 1u)) s[c] = 0xff800000u;  // -inf
        }
        const float m_use = m_run == -INFINITY ? 0.f : m_run;
        const float2 sc2 = make_float2(sc, sc), mneg = make_float2(-m_use, -m_use);
        // several partial sums, so that the chain of dependent additions left after the last exponential is
        // short (the sum of the rounded weights gates the P store)
        float2 la[2], lb[4];
        la[0] = la[1] = lb[0] = lb[1] = lb[2] = lb[3] = make_float2(0.f, 0.f);
#pragma unroll
        for (int c = 0; c < 128; c += 4) {
          float2 e0 = __ffma2_rn(make_float2(__uint_as_float(s[c]), __uint_as_float(s[c + 1])), sc2, mneg);
          float2 e1 = __ffma2_rn(make_float2(__uint_as_float(s[c + 2]), __uint_as_float(s[c + 3])), sc2, mneg);
          e0.x = ex2(e0.x); e0.y = ex2(e0.y);
          e1.x = ex2(e1.x); e1.y = ex2(e1.y);
          pk[c / 2] = pack_bf16(e0.x, e0.y);
          pk[c / 2 + 1] = pack_bf16(e1.x, e1.y);
          la[(c >> 2) & 1] = __fadd2_rn(la[(c >> 2) & 1], __fadd2_rn(e0, e1));
          lb[(c >> 2) & 3] = __fadd2_rn(lb[(c >> 2) & 3], __fadd2_rn(unpack_bf16(pk[c / 2]), unpack_bf16(pk[c / 2 + 1])));
        }
        la[0] = __fadd2_rn(la[0], la[1]);
        lb[0] = __fadd2_rn(__fadd2_rn(lb[0], lb[1]), __fadd2_rn(lb[2], lb[3]));
        const float l_tile = lb[0].x + lb[0].y, l_tile_exact = la[0].x + la[0].y;
        if (pass == 1) { l_run += l_tile; l_exact += l_tile_exact; break; }
        const bool bad = !(l_tile <= kSumLimit) || m_run == -INFINITY;
        if (!__any_sync(0xffffffffu, bad)) { l_run += l_tile; l_exact += l_tile_exact; break; }
        const float m_tile = tile_row_max(t_s, partial, rmask, u0) * sc;
        const bool raise = m_tile > m_run + kRaiseMargin || (m_run == -INFINITY && m_tile > -INFINITY);
        float alpha = 1.f;
        if (raise) {
          alpha = ex2(m_run - m_tile);   // 0 when m_run = -inf
          m_run = m_tile;
          l_run *= alpha;
          l_exact *= alpha;
        }
        if (it > 0) {
          // O of the previous tiles must be complete before it is rescaled
          mbar_wait(bar(C::B_OF + j), (it - 1) & 1, wc);
          tc_fence_after();
#pragma unroll
          for (int c = 0; c < D / 32; ++c) {
            uint32_t v[32];
            tmem_ld32(t_o + c * 32, v);
            tc_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(__uint_as_float(v[i]) * alpha);
            tmem_st32(t_o + c * 32, v);
          }
          tc_wait_st();
        }
      }
      {
        uint32_t(&p0)[32] = *reinterpret_cast<uint32_t(*)[32]>(&pk[0]);
        uint32_t(&p1)[32] = *reinterpret_cast<uint32_t(*)[32]>(&pk[32]);
        tmem_st32(t_s, p0);
        tmem_st32(t_s + 32, p1);
        tc_wait_st();
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(C::B_PF + j));
    }

    if (n > 0) {
      mbar_wait(bar(C::B_OF + j), (n - 1) & 1, wc);
      tc_fence_after();
      int tok = r;
      if (perm && r < g.Nv) tok = (r % g.T) * g.S + r / g.T;
      const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
      uint4* dst = reinterpret_cast<uint4*>(a.o + ((size_t)bh * g.N + min(tok, g.N - 1)) * D);
#pragma unroll
      for (int c = 0; c < D / 32; ++c) {
        uint32_t v[32];
        tmem_ld32(t_o + c * 32, v);   // warp-collective: rows past N take part, they just do not store
        tc_wait_ld();
        if (r < g.N && rf_in_bounds(tok, g.N, a.dev_status)) {
#pragma unroll
          for (int i = 0; i < 32; i += 8) {
            uint4 w;
            w.x = pack_bf16(__uint_as_float(v[i]) * inv, __uint_as_float(v[i + 1]) * inv);
            w.y = pack_bf16(__uint_as_float(v[i + 2]) * inv, __uint_as_float(v[i + 3]) * inv);
            w.z = pack_bf16(__uint_as_float(v[i + 4]) * inv, __uint_as_float(v[i + 5]) * inv);
            w.w = pack_bf16(__uint_as_float(v[i + 6]) * inv, __uint_as_float(v[i + 7]) * inv);
            dst[(c * 32 + i) / 8] = w;
          }
        }
      }
      if (r < g.N && a.lse != nullptr && rf_in_bounds(tok, g.N, a.dev_status)) a.lse[(size_t)bh * g.N + tok] = (m_run + log2f(l_exact)) * 0.6931471805599453f;
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == kTmaWarp) {
    if (*abort_flag) __nanosleep(20000);  // let abandoned copies land before shared memory is released
    __syncwarp();
    tmem_dealloc(tmem_base, C::TMEM_COLS);
  }
}

template <int D>
rf_status launch(const RfAttnArgs& a, const CUtensorMap* maps, cudaStream_t st) {
  static bool configured[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return RF_ERR_CUDA;
  if (dev >= 0 && dev < 64 && !configured[dev]) {
    if (!rf_regs_ok(rf_attn_kernel<D>)) return RF_ERR_UNSUPPORTED;   // setmaxnreg.inc could never be granted
    if (cudaFuncSetAttribute(rf_attn_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Cfg<D>::ALLOC) != cudaSuccess)
      return RF_ERR_CUDA;
    configured[dev] = true;
  }
  Maps m;
  for (int i = 0; i < 8; ++i) m.m[i] = maps[i];
  dim3 grid(rf_cdiv(a.g.nQ, 2), a.g.B * a.g.H);
  rf_attn_kernel<D><<<grid, kThreads, Cfg<D>::ALLOC, st>>>(m, a);
  return cudaGetLastError() == cudaSuccess ? RF_OK : RF_ERR_CUDA;
}

}  // namespace

// Self-test of the bounded-wait machinery every kernel here relies on: one warp waits on an mbarrier that
// nothing ever arrives at.  The wait must give up after limit_ns, raise the CTA's abort flag, report
// RF_ERR_TIMEOUT to *dev_status, let a second wait return at once, and the kernel must exit normally.
__global__ void rf_selftest_timeout_kernel(int32_t* dev_status, uint64_t limit_ns, int32_t* waits_returned) {
  __shared__ __align__(8) uint64_t barrier;
  __shared__ int abort_flag;
  const uint32_t bar = sm100::smem_u32(&barrier);
  if (threadIdx.x == 0) {
    sm100::mbar_init(bar, 1);
    abort_flag = 0;
    sm100::mbar_init_fence();
  }
  __syncthreads();
  sm100::WaitCtx wc{&abort_flag, dev_status, limit_ns};
  const bool first = sm100::mbar_wait(bar, 0, wc);    // runs out
  const bool second = sm100::mbar_wait(bar, 0, wc);   // returns at once: the CTA has given up
  if (threadIdx.x == 0) *waits_returned = (first ? 1 : 0) + (second ? 2 : 0) + (abort_flag ? 4 : 0);
}

rf_status rf_launch_selftest_timeout(int32_t* dev_status, uint64_t limit_ns, int32_t* waits_returned, cudaStream_t st) {
  rf_selftest_timeout_kernel<<<1, 32, 0, st>>>(dev_status, limit_ns, waits_returned);
  return cudaGetLastError() == cudaSuccess ? RF_OK : RF_ERR_CUDA;
}

rf_status rf_launch_attention(const RfAttnArgs& a, const CUtensorMap* maps, cudaStream_t st) {
  switch (a.g.D) {
    case 64: return launch<64>(a, maps, st);
    case 96: return launch<96>(a, maps, st);
    case 128: return launch<128>(a, maps, st);
  }
  return RF_ERR_UNSUPPORTED;
}
