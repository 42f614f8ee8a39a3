// Pattern-masked FlashAttention forward on tcgen05 / TMEM / TMA (Eq. 1-2 with the masks of Sec. 3.2).
//
// One CTA owns one 128-row query tile of one head and walks that tile's list of KV tiles.
// Per KV tile: S = Q K^T (tcgen05.mma, operands staged by TMA in 128B-swizzled shared memory,
// accumulator in TMEM), online softmax in fp32 with one thread per query row (tcgen05.ld), P rounded
// to bf16 into swizzled shared memory, O_tile = P V on the tensor cores, running O in registers.
// K/V tiles are double-buffered: the TMA for tile i+1 is in flight while tile i is computed.
// PARTIAL tiles apply the exact element mask of the head's pattern; FULL tiles skip it.
#include "rf_sm100.cuh"

namespace {

using namespace sm100;

constexpr int BM = 128, BN = 128;
constexpr int kThreads = 128;

struct Maps { CUtensorMap m[8]; };

template <int D>
struct Smem {
  static constexpr int KB = D / 64;                 // 64-column (128-byte) blocks per row
  static constexpr uint32_t BLK = 128 * 128;        // bytes of one 128-row x 64-col bf16 block
  static constexpr uint32_t Q = 0;
  static constexpr uint32_t K0 = Q + KB * BLK;
  static constexpr uint32_t V0 = K0 + 2 * KB * BLK;
  static constexpr uint32_t P = V0 + 2 * KB * BLK;
  static constexpr uint32_t BAR = P + 2 * BLK;      // mbarriers: q, kv[2], mma
  static constexpr uint32_t MISC = BAR + 64;        // tmem base, abort flag
  static constexpr uint32_t TOTAL = MISC + 64;
  static constexpr uint32_t ALLOC = TOTAL + 1024;   // slack for manual 1024-byte alignment
};

// Element mask of one query row in the head's key-slot space.
struct RowMask {
  int lo, hi;        // kept video slots [lo, hi) when !periodic
  int text0;         // first always-kept (text) slot
  int lkv;           // number of key slots
  int p, ws, S;      // periodic form: |slot % S - p| <= ws
  bool periodic;
  __device__ __forceinline__ bool keep(int u) const {
    if (u >= lkv) return false;
    if (u >= text0) return true;
    if (periodic) {
      const int d = (u % S) - p;
      return (d < 0 ? -d : d) <= ws;
    }
    return u >= lo && u < hi;
  }
};

__device__ __forceinline__ RowMask make_row_mask(const RfGeom& g, int cls, int r) {
  RowMask m;
  m.lkv = rf_kv_len(g, cls);
  m.text0 = m.lkv;
  m.lo = 0;
  m.hi = m.lkv;
  m.p = 0; m.ws = g.ws; m.S = g.S;
  m.periodic = false;
  if ((cls == RF_SPATIAL || cls == RF_TEMPORAL) && r < g.Nv) {
    m.text0 = g.Nv;
    if (cls == RF_SPATIAL) {
      const int f = r / g.S;
      m.lo = max(0, f - g.wf) * g.S;
      m.hi = min(g.T, f + g.wf + 1) * g.S;
    } else if (g.permute) {
      const int p = r / g.T;
      m.lo = max(0, p - g.ws) * g.T;
      m.hi = min(g.S, p + g.ws + 1) * g.T;
    } else {
      m.periodic = true;
      m.p = r % g.S;
    }
  }
  return m;
}

template <int D>
__global__ void __launch_bounds__(kThreads, 1) rf_attn_kernel(const __grid_constant__ Maps maps, const RfAttnArgs a) {
  using L = Smem<D>;
  constexpr int KB = L::KB;
  constexpr uint32_t TILE_BYTES = KB * L::BLK;
  constexpr uint32_t TMEM_COLS = 256;          // S: columns [0,128), O tile: [128, 128+D)
  constexpr uint32_t S_COL = 0, O_COL = 128;
  constexpr uint32_t IDESC_S = idesc_bf16(BM, BN, 0);
  constexpr uint32_t IDESC_PV = idesc_bf16(BM, D, 1);

  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t bar_q = base + L::BAR, bar_kv0 = bar_q + 8, bar_mma = bar_q + 24;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + L::MISC);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + L::MISC + 8);

  const RfGeom& g = a.g;
  const int tid = threadIdx.x, warp = tid >> 5;
  const int qt = blockIdx.x, bh = blockIdx.y;

  int cls = RF_DENSE;
  if (a.head_class != nullptr) {
    cls = a.head_class[bh];
    if (cls < 0 || cls > 3) {
      if (tid == 0) rf_report(a.dev_status, RF_ERR_INVALID_ARG);
      cls = RF_DENSE;
    }
  }
  const bool perm = cls == RF_TEMPORAL && g.permute;
  const bool tex = cls == RF_TEXTURAL;
  const CUtensorMap* map_q = &maps.m[perm ? 3 : 0];
  const CUtensorMap* map_k = &maps.m[perm ? 4 : (tex ? 6 : 1)];
  const CUtensorMap* map_v = &maps.m[perm ? 5 : (tex ? 7 : 2)];
  const int lkv = rf_kv_len(g, cls);
  const bool listed = a.head_class != nullptr;
  const int n_tiles = listed ? a.count[(size_t)bh * g.nQ + qt] : rf_cdiv(lkv, BN);
  const int32_t* list = listed ? a.kv_tile + ((size_t)bh * g.nQ + qt) * g.nKmax : nullptr;

  if (tid == 0) {
    mbar_init(bar_q, 1);
    mbar_init(bar_kv0, 1);
    mbar_init(bar_kv0 + 8, 1);
    mbar_init(bar_mma, 1);
    *abort_flag = 0;
    mbar_init_fence();
    prefetch_tmap(map_q);
    prefetch_tmap(map_k);
    prefetch_tmap(map_v);
  }
  if (warp == 0) {
    __syncwarp();
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), TMEM_COLS);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t tmem_lane = tmem_base + ((uint32_t)(warp * 32) << 16);
  const WaitCtx wc{abort_flag, a.dev_status};

  auto tile_entry = [&](int i) -> uint32_t {
    if (listed) return (uint32_t)list[i];
    const bool tail = (i + 1) * BN > lkv;
    return (uint32_t)i | (tail ? RF_PARTIAL_BIT : 0u);
  };
  auto load_kv = [&](int i, int stage) {
    const int tile = (int)(tile_entry(i) & ~RF_PARTIAL_BIT);
    const uint32_t bar = bar_kv0 + 8 * stage;
    mbar_expect_tx(bar, 2 * TILE_BYTES);
#pragma unroll
    for (int kb = 0; kb < KB; ++kb) {
      tma_load_3d(base + L::K0 + stage * TILE_BYTES + kb * L::BLK, map_k, kb * 64, tile * BN, bh, bar);
      tma_load_3d(base + L::V0 + stage * TILE_BYTES + kb * L::BLK, map_v, kb * 64, tile * BN, bh, bar);
    }
  };

  if (tid == 0) {
    mbar_expect_tx(bar_q, TILE_BYTES);
#pragma unroll
    for (int kb = 0; kb < KB; ++kb) tma_load_3d(base + L::Q + kb * L::BLK, map_q, kb * 64, qt * BM, bh, bar_q);
    if (n_tiles > 0) load_kv(0, 0);
  }

  const int r = qt * BM + tid;                       // this thread's query slot
  const RowMask rmask = make_row_mask(g, cls, min(r, g.N - 1));
  float o_acc[D];
#pragma unroll
  for (int d = 0; d < D; ++d) o_acc[d] = 0.f;
  float m_run = -INFINITY, l_run = 0.f;
  const float sc = a.scale_log2;

  for (int it = 0; it < n_tiles; ++it) {
    const int st = it & 1;
    const uint32_t entry = tile_entry(it);
    const bool partial = (entry & RF_PARTIAL_BIT) != 0;
    const int u0 = (int)(entry & ~RF_PARTIAL_BIT) * BN;

    if (tid == 0) {
      if (it + 1 < n_tiles) load_kv(it + 1, st ^ 1);
      if (it == 0) mbar_wait(bar_q, 0, wc);
      mbar_wait(bar_kv0 + 8 * st, (it >> 1) & 1, wc);
      tc_fence_after();
#pragma unroll
      for (int ks = 0; ks < D / 16; ++ks) {
        const uint32_t off = (ks >> 2) * L::BLK + (ks & 3) * 32;
        mma_ss(tmem_base + S_COL, smem_desc_sw128(base + L::Q + off, 16, 1024),
               smem_desc_sw128(base + L::K0 + st * TILE_BYTES + off, 16, 1024), IDESC_S, ks > 0);
      }
      tc_commit(bar_mma);
    }
    __syncwarp();
    mbar_wait(bar_mma, 0, wc);
    tc_fence_after();

    // pass 1: row maximum of the scaled, masked scores
    float rmax = -INFINITY;
#pragma unroll
    for (int c = 0; c < BN / 32; ++c) {
      uint32_t v[32];
      tmem_ld32(tmem_lane + S_COL + c * 32, v);
      tc_wait_ld();
      if (partial) {
#pragma unroll
        for (int j = 0; j < 32; ++j)
          if (rmask.keep(u0 + c * 32 + j)) rmax = fmaxf(rmax, __uint_as_float(v[j]) * sc);
      } else {
#pragma unroll
        for (int j = 0; j < 32; ++j) rmax = fmaxf(rmax, __uint_as_float(v[j]) * sc);
      }
    }
    const float m_new = fmaxf(m_run, rmax);
    const float m_use = (m_new == -INFINITY) ? 0.f : m_new;
    const float alpha = exp2f(m_run - m_use);
    m_run = m_new;
    l_run *= alpha;
#pragma unroll
    for (int d = 0; d < D; ++d) o_acc[d] *= alpha;

    // pass 2: P = exp2(S*scale - m), row sum, bf16 P into swizzled shared memory (K-major A operand)
#pragma unroll
    for (int c = 0; c < BN / 32; ++c) {
      uint32_t v[32];
      tmem_ld32(tmem_lane + S_COL + c * 32, v);
      tc_wait_ld();
      float p[32];
#pragma unroll
      for (int j = 0; j < 32; ++j) {
        float e = exp2f(fmaf(__uint_as_float(v[j]), sc, -m_use));
        if (partial && !rmask.keep(u0 + c * 32 + j)) e = 0.f;
        p[j] = e;
        l_run += e;
      }
      const uint32_t prow = base + L::P + (c >> 1) * L::BLK + tid * 128;
#pragma unroll
      for (int jj = 0; jj < 4; ++jj) {
        const uint32_t chunk = (uint32_t)((c & 1) * 4 + jj) ^ (uint32_t)(tid & 7);
        const uint32_t w0 = pack_bf16(p[jj * 8 + 0], p[jj * 8 + 1]), w1 = pack_bf16(p[jj * 8 + 2], p[jj * 8 + 3]);
        const uint32_t w2 = pack_bf16(p[jj * 8 + 4], p[jj * 8 + 5]), w3 = pack_bf16(p[jj * 8 + 6], p[jj * 8 + 7]);
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(prow + (chunk << 4)), "r"(w0), "r"(w1), "r"(w2), "r"(w3) : "memory");
      }
    }
    fence_proxy_async_smem();
    tc_fence_before();
    __syncthreads();

    if (tid == 0) {
      tc_fence_after();
#pragma unroll
      for (int ks = 0; ks < BN / 16; ++ks) {
        const uint32_t poff = (ks >> 2) * L::BLK + (ks & 3) * 32;
        mma_ss(tmem_base + O_COL, smem_desc_sw128(base + L::P + poff, 16, 1024),
               smem_desc_sw128(base + L::V0 + st * TILE_BYTES + ks * 2048, L::BLK, 1024), IDESC_PV, ks > 0);
      }
      tc_commit(bar_mma);
    }
    __syncwarp();
    mbar_wait(bar_mma, 1, wc);
    tc_fence_after();
#pragma unroll
    for (int c = 0; c < D / 32; ++c) {
      uint32_t v[32];
      tmem_ld32(tmem_lane + O_COL + c * 32, v);
      tc_wait_ld();
#pragma unroll
      for (int j = 0; j < 32; ++j) o_acc[c * 32 + j] += __uint_as_float(v[j]);
    }
  }

  // epilogue: normalise, write O (original token order) and lse
  if (r < g.N) {
    int tok = r;
    if (perm && r < g.Nv) tok = (r % g.T) * g.S + r / g.T;
    const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
    uint4* dst = reinterpret_cast<uint4*>(a.o + ((size_t)bh * g.N + tok) * D);
#pragma unroll
    for (int d = 0; d < D; d += 8) {
      uint4 w;
      w.x = pack_bf16(o_acc[d] * inv, o_acc[d + 1] * inv);
      w.y = pack_bf16(o_acc[d + 2] * inv, o_acc[d + 3] * inv);
      w.z = pack_bf16(o_acc[d + 4] * inv, o_acc[d + 5] * inv);
      w.w = pack_bf16(o_acc[d + 6] * inv, o_acc[d + 7] * inv);
      dst[d / 8] = w;
    }
    if (a.lse != nullptr) a.lse[(size_t)bh * g.N + tok] = (m_run + log2f(l_run)) * 0.6931471805599453f;
  }

  // never leave with a TMA still in flight: the Q load (unused when the list is empty)
  if (tid == 0 && n_tiles == 0) mbar_wait(bar_q, 0, wc);
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    __syncwarp();
    tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

template <int D>
rf_status launch(const RfAttnArgs& a, const CUtensorMap* maps, cudaStream_t st) {
  static bool configured[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return RF_ERR_CUDA;
  if (dev >= 0 && dev < 64 && !configured[dev]) {
    if (cudaFuncSetAttribute(rf_attn_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Smem<D>::ALLOC) != cudaSuccess)
      return RF_ERR_CUDA;
    configured[dev] = true;
  }
  Maps m;
  for (int i = 0; i < 8; ++i) m.m[i] = maps[i];
  dim3 grid(a.g.nQ, a.g.B * a.g.H);
  rf_attn_kernel<D><<<grid, kThreads, Smem<D>::ALLOC, st>>>(m, a);
  return cudaGetLastError() == cudaSuccess ? RF_OK : RF_ERR_CUDA;
}

}  // namespace

rf_status rf_launch_attention(const RfAttnArgs& a, const CUtensorMap* maps, cudaStream_t st) {
  switch (a.g.D) {
    case 64: return launch<64>(a, maps, st);
    case 128: return launch<128>(a, maps, st);
  }
  return RF_ERR_UNSUPPORTED;
}
