// Pattern-masked FlashAttention forward on CTA pairs (Eq. 1-2 with the masks of Sec. 3.2): tcgen05.mma with
// cta_group::2, M = 256 over a cluster of two CTAs.
//
// A pair owns two adjacent 128-row query tiles of one head, one tile per CTA, and walks the union of their KV-tile
// lists.  One thread of the leader CTA (cluster rank 0) issues every MMA for both SMs:
//     S = Q K^T   M = 256 (128 rows per CTA), N = 128 keys; each CTA holds 64 of the tile's keys in shared memory
//     O += P V    M = 256, N = 128 columns;  each CTA holds 64 columns of the V tile (all 128 keys)
// so a CTA fetches and keeps only half of every K and V tile and an instruction does twice the work.  Columns of O
// past D (D = 64, 96) multiply zero-filled parts of the V boxes and are never stored.
// Per CTA, TMEM holds two score buffers, two P buffers and one O accumulator:
//     S0 [0,128)  S1 [128,256)  O [256,384)  P0 [384,448)  P1 [448,512)
// and the two softmax warpgroups take alternate tiles of the SAME 128 query rows: while warpgroup A turns S(u) into
// P(u), the tensor cores compute S(u+2) into the buffer A has just read and O += P(u-1) V(u-1) for warpgroup B.
// A score buffer is handed back as soon as it is in registers, so the exact row maximum of the tile is taken first
// and the exponentials once.  The row's running maximum is shared by the two warpgroups through shared memory and
// raised lazily (only when a tile exceeds it by 2^kLazyRaise): decisions are handed from tile u to tile u+1 through
// a per-warp mbarrier, and the warpgroup that raises rescales the O rows in TMEM after O += P(u-1) V(u-1) has landed.
// Warp roles per CTA: warps 0-3 / 4-7 softmax warpgroups A / B (thread = query row = TMEM lane), warp 8 TMA
// producer (this CTA's halves; completion is counted on the leader's barriers), warp 9 MMA issuer (leader only),
// warps 10-11 fill the third warpgroup, whose registers go to the softmax warpgroups.
// Barriers that the other CTA must reach are addressed through mapa; completion of MMAs is committed once to each
// CTA's barrier.  No load uses cluster multicast.  Every wait is bounded (mbar_wait*).
#include "rf_attn_common.cuh"

namespace {

using namespace sm100;
using namespace rf_attn;

constexpr int kThreads = kWsThreads;
constexpr int kTmaWarp = 8, kMmaWarp = 9;
constexpr float kLazyRaise = 32.0f;   // log2 units: the running maximum is raised when a tile exceeds it by this much
#ifndef RF_PAIR_MIXED_ADD
#define RF_PAIR_MIXED_ADD 0
#endif
#ifndef RF_PAIR_POLY
#define RF_PAIR_POLY 0
#endif
constexpr int kPolyEighths = RF_PAIR_POLY;   // of every eight pairs of exponentials, this many run on the FMA pipe

struct PairMaps { CUtensorMap m[11]; };   // [0..7] as for the single-CTA kernel; [8..10] K with 64-row boxes:
                                          // original order, position-major workspace, compacted workspace

template <int D>
struct PCfg {
  static constexpr int KB = (D + 63) / 64;             // 64-column (128-byte) blocks per Q / K row
  static constexpr uint32_t QBLK = 128 * 128;          // 128 rows x 128 bytes
  static constexpr uint32_t QTILE = KB * QBLK;
  static constexpr uint32_t KBLK = 64 * 128;           // this CTA's 64 keys x 128 bytes
  static constexpr uint32_t KTILE = KB * KBLK;
  static constexpr uint32_t VTILE = 128 * 128;         // 128 keys x this CTA's 64 columns
  static constexpr int NK = 4, NV = 4;                 // ring depths; the slot-reuse waits rely on NK, NV <= 4
  static constexpr uint32_t Q = 0;
  static constexpr uint32_t K0 = Q + QTILE;
  static constexpr uint32_t V0 = K0 + NK * KTILE;
  static constexpr uint32_t BAR = V0 + NV * VTILE;
  // barrier slots (8 bytes each).  QF / KF / SE / PF are used in the leader CTA only.
  static constexpr int B_QF = 0, B_KF = 1 /* K of tiles 0 and 1 */, B_SF = B_KF + 2 /* S(u) ready, by u % 4 */,
                       B_OD = B_SF + 4 /* O += P(u) V(u) landed, by u % 4; last three tiles only */,
                       B_SE = B_OD + 4 /* S(u) read by every softmax warp of the pair and K(u + 2) landed, by u % 4 */,
                       B_PF = B_SE + 4 /* P(u) stored by every softmax warp of the pair and V(u) landed, by u % 4 */,
                       B_DEC = B_PF + 4 /* [warpgroup][warp] decision published */,
                       B_INF = B_DEC + 8 /* tile record u % 8 written */, B_COUNT = B_INF + 8;
  static constexpr uint32_t MISC = BAR + 8 * ((B_COUNT + 7) / 8 * 8);   // +0 TMEM base, +8 abort flag, +12 tile count, +32 tile records
  static constexpr uint32_t MSH = MISC + 64;           // float m_sh[128]: the rows' shared running maximum
  static constexpr uint32_t FIN = MSH + 512;           // float fin[2][3][128]: per warpgroup (m, l_rounded, l_exact)
  static constexpr uint32_t TOTAL = FIN + 2 * 3 * 512;
  static constexpr uint32_t ALLOC = TOTAL + 1024;      // slack for manual 1024-byte alignment
  static_assert(ALLOC <= 227 * 1024, "exceeds the shared memory a CTA can opt in to");
  static constexpr uint32_t S_COL = 0, O_COL = 256, P_COL = 384, TMEM_COLS = 512;
  static __host__ __device__ constexpr uint32_t koff_q(int ks) { return ks < 4 ? (uint32_t)ks * 32u : QBLK + (uint32_t)(ks - 4) * 32u; }
  static __host__ __device__ constexpr uint32_t koff_k(int ks) { return ks < 4 ? (uint32_t)ks * 32u : KBLK + (uint32_t)(ks - 4) * 32u; }
};

// Tile record of the union's tile u, written by the TMA warp (the only role that walks the lists) into a ring of
// eight words and read by the MMA issuer and the softmax warps: tile index, which of the two query tiles list it,
// and whether their entries are PARTIAL.  kEnd follows the last tile (twice, one per warpgroup parity).
constexpr uint32_t kEnd = 0xffffffffu;
constexpr uint32_t kTileMask = 0x00ffffffu;
// bits 0-23 tile, 24-25 how many tiles follow this one (3 = three or more), 28-29 uses, 30-31 PARTIAL flags
__device__ __forceinline__ uint32_t make_record(int tile, int uses, int part) {
  return (uint32_t)tile | ((uint32_t)uses << 28) | ((uint32_t)part << 30);
}
__device__ __forceinline__ int rec_more(uint32_t rec) { return (int)((rec >> 24) & 3u); }

// The pair's merged walk over the two tiles' ascending lists.
struct Walk {
  int i0 = 0, i1 = 0;
  uint32_t raw0 = 0, raw1 = 0;
  __device__ __forceinline__ void start(const Lists& L) {
    if (L.n0 > 0) raw0 = L.entry(0, 0);
    if (L.n1 > 0) raw1 = L.entry(1, 0);
  }
  // Next tile of the union; bit j of `uses` set when query tile j lists it, bit j of `part` when its entry is PARTIAL.
  __device__ __forceinline__ bool next(const Lists& L, int& tile, int& uses, int& part) {
    const int h0 = i0 < L.n0 ? (int)(raw0 & ~RF_PARTIAL_BIT) : 0x7fffffff;
    const int h1 = i1 < L.n1 ? (int)(raw1 & ~RF_PARTIAL_BIT) : 0x7fffffff;
    tile = min(h0, h1);
    if (tile == 0x7fffffff) return false;
    uses = (h0 == tile ? 1 : 0) | (h1 == tile ? 2 : 0);
    part = ((uses & 1) && (raw0 & RF_PARTIAL_BIT) ? 1 : 0) | ((uses & 2) && (raw1 & RF_PARTIAL_BIT) ? 2 : 0);
    if ((uses & 1) && ++i0 < L.n0) raw0 = L.entry(0, i0);
    if ((uses & 2) && ++i1 < L.n1) raw1 = L.entry(1, i1);
    return true;
  }
};

template <int D>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
rf_attn_pair_kernel(const __grid_constant__ PairMaps maps, const RfAttnArgs a) {
  using C = PCfg<D>;
  constexpr int KB = C::KB;
  constexpr uint32_t IDESC_S = idesc_bf16(256, BN, 0);
  constexpr uint32_t IDESC_PV = idesc_bf16(256, 128, 1);

  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
  auto bar = [&](int slot) -> uint32_t { return base + C::BAR + 8u * slot; };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + C::MISC);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + C::MISC + 8);
  volatile int* n_sh = reinterpret_cast<volatile int*>(base_ptr + C::MISC + 12);
  volatile uint32_t* rec_sh = reinterpret_cast<volatile uint32_t*>(base_ptr + C::MISC + 32);
  volatile float* m_sh = reinterpret_cast<volatile float*>(base_ptr + C::MSH);
  volatile float* fin = reinterpret_cast<volatile float*>(base_ptr + C::FIN);

  RfGeom g = a.g;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t rank = cluster_ctarank();          // 0: leader
  const int bh = blockIdx.y;
  const int qt0 = 2 * (blockIdx.x >> 1), qt1 = qt0 + 1;
  const int qt_own = qt0 + (int)rank;

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
    if (cls == RF_SPATIAL && w >= 0) g.wf = min(w, g.T);
    if (cls == RF_TEMPORAL && w >= 0) g.ws = min(w, g.S);
  }
  const bool perm = cls == RF_TEMPORAL && g.permute;
  const bool tex = cls == RF_TEXTURAL;
  const CUtensorMap* map_q = &maps.m[perm ? 3 : 0];
  const CUtensorMap* map_k = &maps.m[perm ? 9 : (tex ? 10 : 8)];
  const CUtensorMap* map_v = &maps.m[perm ? 5 : (tex ? 7 : 2)];

  Lists L;
  L.lkv = rf_kv_len(g, cls);
  L.listed = a.head_class != nullptr;
  if (L.listed) {
    L.n0 = a.count[(size_t)bh * g.nQ + qt0];
    L.n1 = qt1 < g.nQ ? a.count[(size_t)bh * g.nQ + qt1] : 0;
    L.l0 = a.kv_tile + ((size_t)bh * g.nQ + qt0) * g.nKmax;
    L.l1 = a.kv_tile + ((size_t)bh * g.nQ + min(qt1, g.nQ - 1)) * g.nKmax;
  } else {
    L.n0 = rf_cdiv(L.lkv, BN);
    L.n1 = qt1 < g.nQ ? L.n0 : 0;
    L.l0 = L.l1 = nullptr;
  }

  if (tid == 0) {
    mbar_init(bar(C::B_QF), 1);
    for (int s = 0; s < 2; ++s) mbar_init(bar(C::B_KF + s), 1);
    for (int s = 0; s < 4; ++s) {
      mbar_init(bar(C::B_SF + s), 1);
      mbar_init(bar(C::B_OD + s), 1);
      mbar_init(bar(C::B_SE + s), 9);   // 4 softmax warps of each CTA + the leader's expect_tx for the TMA bytes
      mbar_init(bar(C::B_PF + s), 9);
    }
    for (int s = 0; s < 8; ++s) { mbar_init(bar(C::B_DEC + s), 1); mbar_init(bar(C::B_INF + s), 1); }
    *abort_flag = 0;
    *n_sh = 0;
    mbar_init_fence();
  }
  if (tid < 128) m_sh[tid] = -INFINITY;
  if (warp == kTmaWarp) {
    if (lane == 0) { prefetch_tmap(map_q); prefetch_tmap(map_k); prefetch_tmap(map_v); }
    __syncwarp();
    tmem_alloc_pair(smem_u32(const_cast<uint32_t*>(tmem_slot)), C::TMEM_COLS);
  }
  tc_fence_before();
  cluster_sync();            // both CTAs' barriers initialised and TMEM allocated before anything crosses over
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const WaitCtx wc{abort_flag, a.dev_status};
  // Record of tile u, or kEnd.  A record slot is rewritten eight tiles later, when the TMA warp has long seen
  // O += P(u-5) V(u-5) land (its V-slot wait), that is, after every reader of record u - 8.
  auto record = [&](int u) -> uint32_t {
    mbar_wait(bar(C::B_INF + (u & 7)), (u >> 3) & 1, wc);
    return rec_sh[u & 7];
  };

  if (warp >= 8) {
    RF_SETMAXNREG_DEC();
    if (warp == kTmaWarp) {
      // ------------------------------------------------------------ TMA producer (each CTA: its own halves)
      if (lane == 0) {
        auto lbar = [&](int slot) -> uint32_t { return mapa(bar(slot), 0); };   // the leader's barrier
        if (rank == 0) mbar_expect_tx(bar(C::B_QF), 2 * C::QTILE);
#pragma unroll
        for (int kb = 0; kb < KB; ++kb)
          tma_load_3d_pair(base + C::Q + kb * C::QBLK, map_q, kb * 64, qt_own * BM, bh, lbar(C::B_QF));
        // the walk runs three tiles ahead of the records: a record says how many tiles follow it (up to 3)
        Walk wk;
        wk.start(L);
        uint32_t pend[4];
        int np = 0, u = 0;
        bool more = true;
        for (;;) {
          while (more && np < 4) {
            int tile, uses, part;
            if (wk.next(L, tile, uses, part)) { pend[(u + np) & 3] = make_record(tile, uses, part); ++np; } else more = false;
          }
          if (np == 0) break;
          const uint32_t rec = pend[u & 3] | ((uint32_t)(np - 1) << 24);
          const int tile = (int)(rec & kTileMask);
          const int s = u % C::NK;   // NK == NV
          rec_sh[u & 7] = rec;
          mbar_arrive(bar(C::B_INF + (u & 7)));
          // K slot: free once S(u - NK) has been computed.  K of tiles 0 and 1 lands on barriers of its own; K(u)
          // of later tiles is counted on the barrier that also collects the reads of S(u - 2), whose buffer S(u)
          // is computed into: one wait of the issuer covers both.
          if (u >= C::NK) mbar_wait(bar(C::B_SF + ((u - C::NK) & 3)), ((u - C::NK) >> 2) & 1, wc);
          const int kbar = u < 2 ? C::B_KF + u : C::B_SE + ((u - 2) & 3);
          if (rank == 0) mbar_expect_tx(bar(kbar), 2 * C::KTILE);
#pragma unroll
          for (int kb = 0; kb < KB; ++kb)
            tma_load_3d_pair(base + C::K0 + s * C::KTILE + kb * C::KBLK, map_k, kb * 64, tile * BN + 64 * (int)rank, bh,
                             lbar(kbar));
          // V slot: free once O += P(u - NV) V(u - NV) has landed; MMAs complete in issue order and S(u - 1) was
          // issued after it.  V(u) is counted on the barrier that collects the stores of P(u).
          if (u >= C::NV) mbar_wait(bar(C::B_SF + ((u - 1) & 3)), ((u - 1) >> 2) & 1, wc);
          if (rank == 0) mbar_expect_tx(bar(C::B_PF + (u & 3)), 2 * C::VTILE);
          tma_load_3d_pair(base + C::V0 + s * C::VTILE, map_v, 64 * (int)rank, tile * BN, bh, lbar(C::B_PF + (u & 3)));
          ++u;
          --np;
        }
        *n_sh = u;
        for (int e = u; e < u + 2; ++e) {
          rec_sh[e & 7] = kEnd;
          mbar_arrive(bar(C::B_INF + (e & 7)));
        }
      }
    } else if (warp == kMmaWarp && rank == 0) {
      // ------------------------------------------------------------ MMA issuer (leader CTA, for both SMs)
      // Everything this thread does between two MMAs is idle tensor time, so per tile it takes one record, two
      // waits (each covering a TMA landing and the softmax warps of both CTAs) and one commit to each CTA.
      if (lane == 0) {
        constexpr uint32_t DESC_HI = (1024u >> 4) | (1u << 14) | (2u << 29);      // SBO 1024 B, version 1, 128B swizzle
        constexpr uint32_t LO_KMAJOR = 1u << 16;
        constexpr uint32_t LO_VMAJOR = (C::VTILE >> 4) << 16;                      // one 64-column block per CTA: unused
        auto desc = [](uint32_t lo) -> uint64_t { return ((uint64_t)DESC_HI << 32) | lo; };
        const uint32_t q_lo = ((base + C::Q) >> 4) | LO_KMAJOR, k_lo = ((base + C::K0) >> 4) | LO_KMAJOR;
        const uint32_t v_lo = ((base + C::V0) >> 4) | LO_VMAJOR;
        const uint32_t peer_bar0 = mapa(bar(0), 1);
        auto commit_both = [&](int slot) {
          tc_commit_pair(bar(slot));
          tc_commit_pair(peer_bar0 + 8u * slot);
        };
        auto issue_s = [&](int sbuf, int kslot) {
          const uint32_t b0 = k_lo + kslot * (C::KTILE >> 4);
          const uint32_t t_d = tmem_base + C::S_COL + sbuf * 128;
          mma_ss_pair<false>(t_d, desc(q_lo), desc(b0), IDESC_S);
#pragma unroll
          for (int k = 1; k < D / 16; ++k)
            mma_ss_pair<true>(t_d, desc(q_lo + (C::koff_q(k) >> 4)), desc(b0 + (C::koff_k(k) >> 4)), IDESC_S);
        };
        auto issue_pv = [&](int pbuf, int vslot, bool first) {
          const uint32_t b0 = v_lo + vslot * (C::VTILE >> 4);
          const uint32_t t_p = tmem_base + C::P_COL + pbuf * 64, t_o = tmem_base + C::O_COL;
          mma_ts_pair(t_o, t_p, desc(b0), IDESC_PV, !first);
#pragma unroll
          for (int k = 1; k < BN / 16; ++k)
            mma_ts_pair_c<true>(t_o, t_p + k * 8, desc(b0 + k * (2048 >> 4)), IDESC_PV);
        };
        uint32_t rec = record(0);
        if (rec != kEnd) {
          mbar_wait_cluster(bar(C::B_QF), 0, wc);
          mbar_wait_cluster(bar(C::B_KF), 0, wc);
          tc_fence_after();
          issue_s(0, 0);
          commit_both(C::B_SF);
          if (rec_more(rec) >= 1) {
            mbar_wait_cluster(bar(C::B_KF + 1), 0, wc);
            issue_s(1, 1);
            commit_both(C::B_SF + 1);
          }
          for (int u = 0; u < g.nKmax; ++u) {      // a union holds at most nKmax tiles: the bound ends the loop after an abort
            if (u > 0) rec = record(u);
            const int more = rec_more(rec);
            if (more >= 2) {
              // S(u + 2) into the buffer S(u) was read from; normally long before P(u) arrives
              mbar_wait_cluster(bar(C::B_SE + (u & 3)), (u >> 2) & 1, wc);      // K(u + 2) landed, S(u) read
              tc_fence_after();
              issue_s(u & 1, (u + 2) % C::NK);
              commit_both(C::B_SF + ((u + 2) & 3));
            }
            mbar_wait_cluster(bar(C::B_PF + (u & 3)), (u >> 2) & 1, wc);        // V(u) landed, P(u) stored
            tc_fence_after();
            issue_pv(u & 1, u % C::NV, u == 0);
            // only the last three tiles' O updates are waited for by themselves (see the softmax warps)
            if (more <= 2) commit_both(C::B_OD + (u & 3));
            if (more == 0) break;
          }
        }
      }
    }
  } else {
    RF_SETMAXNREG_INC();
    // ------------------------------------------------------------ softmax + epilogue, one thread per query row
    const int wg = warp >> 2, w4 = warp & 3;       // warpgroup A (0): even tiles of the union, B (1): odd tiles
    const int row = tid & 127;
    const int r = qt_own * BM + row;               // query slot in the head's coordinate space
    const uint32_t lane_sel = (uint32_t)(w4 * 32) << 16;
    const uint32_t t_s = tmem_base + lane_sel + C::S_COL + wg * 128;
    const uint32_t t_p = tmem_base + lane_sel + C::P_COL + wg * 64;
    const uint32_t t_o = tmem_base + lane_sel + C::O_COL;
    const uint32_t lead_bar0 = mapa(bar(0), 0);    // the leader's barrier slot 0
    const RowMask rmask = make_row_mask(g, cls, min(r, g.N - 1));
    const float sc = a.scale_log2;
    float m_mine = -INFINITY;  // the running maximum this thread's sums refer to (log2 domain)
    float l_run = 0.f;         // sum of the weights as rounded to bf16: normalises O
    float l_exact = 0.f;       // sum of the unrounded weights: the log-sum-exp

    for (int u = wg; u < g.nKmax + 2; u += 2) {   // the end record comes at most at nKmax + 1
      const uint32_t rec = record(u);
      if (rec == kEnd) break;
      const bool mine = (rec >> (28 + rank)) & 1;      // this CTA's query tile lists the tile
      const bool partial = (rec >> (30 + rank)) & 1;
      const int u0 = (int)(rec & kTileMask) * BN;
      const int more = rec_more(rec);                  // tiles of the union after this one (3: three or more)
      mbar_wait(bar(C::B_SF + (u & 3)), (u >> 2) & 1, wc);
      tc_fence_after();
      uint32_t s[128];
      float m_tile = -INFINITY;
      if (mine) {
        uint32_t(&s0)[32] = *reinterpret_cast<uint32_t(*)[32]>(&s[0]);
        uint32_t(&s1)[32] = *reinterpret_cast<uint32_t(*)[32]>(&s[32]);
        uint32_t(&s2)[32] = *reinterpret_cast<uint32_t(*)[32]>(&s[64]);
        uint32_t(&s3)[32] = *reinterpret_cast<uint32_t(*)[32]>(&s[96]);
        // the exact row maximum of the tile, in eight independent chains; on FULL tiles the first half is
        // reduced while the second half is still on its way out of TMEM
        float mx[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) mx[i] = -INFINITY;
        tmem_ld32(t_s, s0);
        tmem_ld32(t_s + 32, s1);
        tc_wait_ld();
        tmem_ld32(t_s + 64, s2);
        tmem_ld32(t_s + 96, s3);
        if (!partial) {
#pragma unroll
          for (int c = 0; c < 64; c += 2) mx[(c >> 1) & 7] = max3(mx[(c >> 1) & 7], __uint_as_float(s[c]), __uint_as_float(s[c + 1]));
        }
        tc_wait_ld();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(lead_bar0 + 8u * (C::B_SE + (u & 3)));  // the score buffer may be refilled
        if (partial) {
          uint32_t wbits[4];
          rmask.tile_bits(u0, wbits);
#pragma unroll
          for (int c = 0; c < 128; ++c)
            if (!((wbits[c >> 5] >> (c & 31)) & 1u)) s[c] = 0xff800000u;  // -inf
#pragma unroll
          for (int c = 0; c < 64; c += 2) mx[(c >> 1) & 7] = max3(mx[(c >> 1) & 7], __uint_as_float(s[c]), __uint_as_float(s[c + 1]));
        }
#pragma unroll
        for (int c = 64; c < 128; c += 2) mx[(c >> 1) & 7] = max3(mx[(c >> 1) & 7], __uint_as_float(s[c]), __uint_as_float(s[c + 1]));
        m_tile = fmaxf(fmaxf(max3(mx[0], mx[1], mx[2]), max3(mx[3], mx[4], mx[5])), fmaxf(mx[6], mx[7])) * sc;
      } else {
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(lead_bar0 + 8u * (C::B_SE + (u & 3)));
      }
      // The decision on the running maximum passes from tile u - 1 (the other warpgroup's warp of the same rows)
      // to tile u: normally that decision was published most of a tile ago.
      if (u > 0) mbar_wait(bar(C::B_DEC + (wg ^ 1) * 4 + w4), ((u - 1) >> 1) & 1, wc);
      const float m_cur = m_sh[row];
      if (m_cur != m_mine) {                       // the other warpgroup raised it: bring this thread's sums along
        const float f = ex2(m_mine - m_cur);       // m_mine = -inf: 0, and the sums are 0 anyway
        l_run *= f;
        l_exact *= f;
        m_mine = m_cur;
      }
      const bool raise = mine && (m_tile > m_mine + kLazyRaise || (m_mine == -INFINITY && m_tile > -INFINITY));
      if (__any_sync(0xffffffffu, raise)) {
        float alpha = 1.f;
        if (raise) {
          alpha = ex2(m_mine - m_tile);            // 0 when m_mine = -inf
          m_mine = m_tile;
          l_run *= alpha;
          l_exact *= alpha;
          m_sh[row] = m_mine;
        }
        if (u > 0) {
          // O may only be rescaled once everything issued into it has landed: that includes O += P(u-1) V(u-1),
          // whose P the other warpgroup computed against the old maximum.  MMAs complete in issue order and
          // S(u+2) is issued after it (every warp has already handed S(u) back, so this cannot deadlock); the
          // last tiles have no S(u+2) and wait for the update itself.
          if (more >= 2) mbar_wait(bar(C::B_SF + ((u + 2) & 3)), ((u + 2) >> 2) & 1, wc);
          else mbar_wait(bar(C::B_OD + ((u - 1) & 3)), 0, wc);
          tc_fence_after();
#pragma unroll
          for (int c = 0; c < 4; ++c) {
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
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(C::B_DEC + wg * 4 + w4));   // tile u + 1 may decide

      uint32_t pk[64];
      if (mine) {
        const float m_use = m_mine == -INFINITY ? 0.f : m_mine;
        const float2 sc2 = make_float2(sc, sc), mneg = make_float2(-m_use, -m_use);
        float2 la[2], lb[4];
        la[0] = la[1] = lb[0] = lb[1] = lb[2] = lb[3] = make_float2(0.f, 0.f);
#if RF_PAIR_MIXED_ADD
        float lm[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#endif
#pragma unroll
        for (int c = 0; c < 128; c += 4) {
          float2 e0 = __ffma2_rn(make_float2(__uint_as_float(s[c]), __uint_as_float(s[c + 1])), sc2, mneg);
          float2 e1 = __ffma2_rn(make_float2(__uint_as_float(s[c + 2]), __uint_as_float(s[c + 3])), sc2, mneg);
          if (((c >> 1) & 7) < kPolyEighths) e0 = ex2_poly2(e0); else { e0.x = ex2(e0.x); e0.y = ex2(e0.y); }
          if ((((c >> 1) + 1) & 7) < kPolyEighths) e1 = ex2_poly2(e1); else { e1.x = ex2(e1.x); e1.y = ex2(e1.y); }
          pk[c / 2] = pack_bf16(e0.x, e0.y);
          pk[c / 2 + 1] = pack_bf16(e1.x, e1.y);
          la[(c >> 2) & 1] = __fadd2_rn(la[(c >> 2) & 1], __fadd2_rn(e0, e1));
#if RF_PAIR_MIXED_ADD
          add_bf16x2(lm[(c >> 1) & 7], lm[((c >> 1) + 1) & 7], pk[c / 2]);
          add_bf16x2(lm[((c >> 1) + 2) & 7], lm[((c >> 1) + 3) & 7], pk[c / 2 + 1]);
#else
          lb[(c >> 2) & 3] = __fadd2_rn(lb[(c >> 2) & 3], __fadd2_rn(unpack_bf16(pk[c / 2]), unpack_bf16(pk[c / 2 + 1])));
#endif
        }
        la[0] = __fadd2_rn(la[0], la[1]);
#if RF_PAIR_MIXED_ADD
        lb[0] = make_float2((lm[0] + lm[1]) + (lm[2] + lm[3]), (lm[4] + lm[5]) + (lm[6] + lm[7]));
#else
        lb[0] = __fadd2_rn(__fadd2_rn(lb[0], lb[1]), __fadd2_rn(lb[2], lb[3]));
#endif
        l_exact += la[0].x + la[0].y;
        l_run += lb[0].x + lb[0].y;
      } else {
#pragma unroll
        for (int c = 0; c < 64; ++c) pk[c] = 0u;   // the other CTA's tile: nothing of it reaches this O
      }
      // the P buffer was read by O += P(u-2) V(u-2): S(u+1) was issued after it (long ready); the last tile waits
      // for the update itself
      if (u >= 2) {
        if (more >= 1) mbar_wait(bar(C::B_SF + ((u + 1) & 3)), ((u + 1) >> 2) & 1, wc);
        else mbar_wait(bar(C::B_OD + ((u - 2) & 3)), 0, wc);
      }
      {
        uint32_t(&p0)[32] = *reinterpret_cast<uint32_t(*)[32]>(&pk[0]);
        uint32_t(&p1)[32] = *reinterpret_cast<uint32_t(*)[32]>(&pk[32]);
        tmem_st32(t_p, p0);
        tmem_st32(t_p + 32, p1);
        tc_wait_st();
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(lead_bar0 + 8u * (C::B_PF + (u & 3)));
    }

    const int n = *n_sh;       // written before the end records this warpgroup has just seen (0 after an abort)
    // The two warpgroups' sums, brought to the row's final maximum.
    fin[(wg * 3 + 0) * 128 + row] = m_mine;
    fin[(wg * 3 + 1) * 128 + row] = l_run;
    fin[(wg * 3 + 2) * 128 + row] = l_exact;
    asm volatile("bar.sync 1, 256;" ::: "memory");
    const float m_o = fin[((wg ^ 1) * 3 + 0) * 128 + row];
    const float m_fin = fmaxf(m_mine, m_o);
    const float f_mine = m_mine == m_fin ? 1.f : ex2(m_mine - m_fin);
    const float f_o = m_o == m_fin ? 1.f : ex2(m_o - m_fin);
    const float l_all = l_run * f_mine + fin[((wg ^ 1) * 3 + 1) * 128 + row] * f_o;
    const float lx_all = l_exact * f_mine + fin[((wg ^ 1) * 3 + 2) * 128 + row] * f_o;

    if (n > 0) {
      mbar_wait(bar(C::B_OD + ((n - 1) & 3)), 0, wc);
      tc_fence_after();
      int tok = r;
      if (perm && r < g.Nv) tok = (r % g.T) * g.S + r / g.T;
      const float inv = l_all > 0.f ? 1.f / l_all : 0.f;
      // warpgroup A stores columns [0, 64), B columns [64, D)
      constexpr int NCH = D / 32;                  // 32-column chunks of O that hold real columns
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        const int ch = wg * 2 + c;
        if (ch < NCH) {
          uint32_t v[32];
          tmem_ld32(t_o + ch * 32, v);             // warp-collective: rows past N take part, they just do not store
          tc_wait_ld();
          if (r < g.N) {
            uint4* dst = reinterpret_cast<uint4*>(a.o + ((size_t)bh * g.N + tok) * D + ch * 32);
#pragma unroll
            for (int i = 0; i < 32; i += 8) {
              uint4 o4;
              o4.x = pack_bf16(__uint_as_float(v[i]) * inv, __uint_as_float(v[i + 1]) * inv);
              o4.y = pack_bf16(__uint_as_float(v[i + 2]) * inv, __uint_as_float(v[i + 3]) * inv);
              o4.z = pack_bf16(__uint_as_float(v[i + 4]) * inv, __uint_as_float(v[i + 5]) * inv);
              o4.w = pack_bf16(__uint_as_float(v[i + 6]) * inv, __uint_as_float(v[i + 7]) * inv);
              dst[i / 8] = o4;
            }
          }
        }
      }
      if (wg == 0 && r < g.N && a.lse != nullptr)
        a.lse[(size_t)bh * g.N + tok] = (m_fin + log2f(lx_all)) * 0.6931471805599453f;
    }
  }

  __syncwarp();
  tc_fence_before();
  cluster_sync();            // neither CTA frees TMEM or leaves while the other may still reach into it
  if (warp == kTmaWarp) {
    if (*abort_flag) __nanosleep(20000);  // let abandoned copies land before shared memory is released
    __syncwarp();
    tmem_dealloc_pair(tmem_base, C::TMEM_COLS);
  }
}

template <int D>
rf_status launch(const RfAttnArgs& a, const CUtensorMap* maps, cudaStream_t st) {
  static bool configured[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return RF_ERR_CUDA;
  if (dev >= 0 && dev < 64 && !configured[dev]) {
    if (!rf_regs_ok(rf_attn_pair_kernel<D>)) return RF_ERR_UNSUPPORTED;   // setmaxnreg.inc could never be granted
    if (cudaFuncSetAttribute(rf_attn_pair_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)PCfg<D>::ALLOC) != cudaSuccess)
      return RF_ERR_CUDA;
    configured[dev] = true;
  }
  PairMaps m;
  for (int i = 0; i < 11; ++i) m.m[i] = maps[i];
  dim3 grid(2 * rf_cdiv(a.g.nQ, 2), a.g.B * a.g.H);   // clusters of two along x: one query tile per CTA
  rf_attn_pair_kernel<D><<<grid, kThreads, PCfg<D>::ALLOC, st>>>(m, a);
  return cudaGetLastError() == cudaSuccess ? RF_OK : RF_ERR_CUDA;
}

}  // namespace

rf_status rf_launch_attention_pair(const RfAttnArgs& a, const CUtensorMap* maps, cudaStream_t st) {
  switch (a.g.D) {
    case 64: return launch<64>(a, maps, st);
    case 96: return launch<96>(a, maps, st);
    case 128: return launch<128>(a, maps, st);
  }
  return RF_ERR_UNSUPPORTED;
}
