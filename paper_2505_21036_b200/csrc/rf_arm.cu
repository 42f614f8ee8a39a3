// ARM: Adaptive Recognition Module (Sec. 3.3, Eq. 6, Algorithm 1).
//
// The sampled score matrix S' = Q' K'^T / sqrt(d) is a dense contraction, so it runs on tcgen05 like the
// attention kernel, minus everything that concerns V: one CTA takes two 128-row tiles of sampled queries
// ("streams") of one head and walks all 128-key tiles of the sample.  Sampled rows are fetched straight
// from Q and K by TMA through tensor maps whose row stride is omega tokens (no gather pass).  Warp roles:
//   warps 0-3 / 4-7  softmax statistics of stream 0 / 1 (one thread per sampled query row)
//   warp 8           TMA producer: both Q tiles once, then K tiles into a shared-memory ring
//   warp 9           MMA issuer; each stream's S accumulator is double-buffered in TMEM (4 x 128 columns),
//                    so the next tile's scores are computed while the current ones are being reduced
// Per tile a softmax thread reads its row of S (tcgen05.ld), hands the buffer back, and updates an
// online softmax (running maximum, total mass) plus the masked masses Algorithm 1 needs: the share of
// the row kept by the sampled Temporal / Spatial (/ Textural, when recalls are requested) mask.
// On the first-frame sample positions equal sample indices, and on the stride sample frames grow
// with the sample index, so a row's kept keys form one index interval: tiles wholly inside or outside
// it for all 32 rows of a warp cost nothing extra, tiles an edge crosses use a 128-bit keep word per
// row.  Only the Temporal mask on the stride sample (RF_SAMPLE_GLOBAL) and the Textural diagnostic
// need per-key attributes, computed cooperatively per tile.
// With the first frame as a key frame of Spatial heads (Sec. 3.2: adjacent or key frames) the Spatial masks keep,
// in addition, the sampled keys of frame 0, a prefix of the stride sample.
// Per-row recalls go to scratch; a second kernel averages them in a fixed order (deterministic) and
// takes Algorithm 1's decision.  The n x n score matrix is never written.
// A bounded wait that runs out is recorded in a flag word at the end of the scratch (cleared at the start of
// every call); the decision kernel then writes class -1 for every head instead of a class computed from
// unwritten rows, and passes the code on to the caller's status word.  The tile builder and the attention
// kernel report a class outside 0..3 through their own status, so the failure cannot go unnoticed even by a
// caller that gave ARM no status pointer.
#include "rf_sm100.cuh"

namespace {

using namespace sm100;

constexpr int ARM_TILE = 128;
constexpr int ARM_THREADS = kWsThreads;    // softmax 0, softmax 1, {TMA, MMA, 2 idle warps}
constexpr int ARM_TMA_WARP = 8, ARM_MMA_WARP = 9;

struct ArmMaps { CUtensorMap q[2], k[2]; };   // per sample: 0 = stride sample, 1 = first-frame sample

constexpr int ARM_MAX_NB = RF_MAX_BANDWIDTHS;   // candidate windows per pattern (1 for plain Algorithm 1)

struct ArmSample {
  int n;          // sampled tokens
  int stride;     // token index of sample m is m * stride
  int pairs;      // CTAs per head: ceil(ceil(n/128) / 2)
  int want_t;     // accumulate the Temporal masses on this sample
  int want_s;     // accumulate the Spatial masses on this sample
  float* out;     // [B*H][2*NB+1][n_pad]: Temporal per window, Spatial per window, Textural
};
struct ArmWindows { int ws[ARM_MAX_NB], wf[ARM_MAX_NB]; };   // candidate spatial (Temporal) / frame (Spatial) windows

template <int D>
struct ArmCfg {
  static constexpr int KB = (D + 63) / 64;
  static constexpr int COL1 = 64;   // D = 96: the second 64-column box reaches past the tensor and is zero-filled
  static constexpr uint32_t BLK = 128 * 128;
  static constexpr uint32_t TILE = KB * BLK;
  static constexpr int NK = D == 64 ? 6 : 4;
  static constexpr uint32_t Q = 0;
  static constexpr uint32_t K0 = Q + 2 * TILE;
  static constexpr uint32_t BAR = K0 + NK * TILE;
  static constexpr int B_Q = 0, B_KF = 1, B_KE = B_KF + NK, B_SF = B_KE + NK, B_SE = B_SF + 4, B_COUNT = B_SE + 4;
  static constexpr uint32_t MISC = BAR + 8 * ((B_COUNT + 7) / 8 * 8);
  static constexpr uint32_t ATTR = MISC + 64;                    // int [8 warps][2][128]: key position / checkerboard flag
  static constexpr uint32_t TOTAL = ATTR + 8 * 2 * 128 * 4;
  static constexpr uint32_t ALLOC = TOTAL + 1024;
  static_assert(ALLOC <= 227 * 1024, "exceeds the shared memory a CTA can opt in to");
  static __host__ __device__ constexpr uint32_t koff(int ks) {
    return ks < 4 ? (uint32_t)ks * 32u : BLK + (uint32_t)(ks - 4) * 32u;
  }
};

__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t bits_below(int n) { return n >= 32 ? 0xffffffffu : ((1u << n) - 1u); }
// Bits of the tile starting at key u0 that fall in the key interval [a, b).
__device__ __forceinline__ void interval_bits(uint32_t (&w)[4], int u0, int a, int b) {
  a = max(a - u0, 0);
  b = min(b - u0, ARM_TILE);
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const int lo = min(max(a - 32 * k, 0), 32), hi = min(max(b - 32 * k, 0), 32);
    w[k] = hi > lo ? (bits_below(hi) & ~bits_below(lo)) : 0u;
  }
}

template <int D, int NB, bool TEX>
__global__ void __launch_bounds__(ARM_THREADS, 1) rf_arm_kernel(const __grid_constant__ ArmMaps maps, const RfGeom g,
                                                                const ArmSample sm0, const ArmSample sm1,
                                                                const ArmWindows win, int n_pad, float scale_log2,
                                                                int32_t* arm_flag) {
  using C = ArmCfg<D>;
  constexpr uint32_t IDESC_S = idesc_bf16(128, 128, 0);
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
  auto bar = [&](int slot) -> uint32_t { return base + C::BAR + 8u * slot; };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + C::MISC);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + C::MISC + 8);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int bh = blockIdx.y;
  // blockIdx.x enumerates the CTAs of the stride sample first, then those of the first-frame sample
  const bool second = (int)blockIdx.x >= sm0.pairs;
  const ArmSample& sm = second ? sm1 : sm0;
  const int which = second ? 1 : 0;
  const int pair = second ? blockIdx.x - sm0.pairs : blockIdx.x;
  const int n = sm.n, stride = sm.stride;
  const int nt = rf_cdiv(n, ARM_TILE);
  const int qt0 = 2 * pair;
  const bool stream1 = qt0 + 1 < nt;
  const CUtensorMap* map_q = &maps.q[which];
  const CUtensorMap* map_k = &maps.k[which];
  // positions equal sample indices only while the sample is contiguous and stays inside the first frame
  // (the 2-D in-frame window is not an interval of the sample index, so it always takes the per-key table)
  const bool t_generic = sm.want_t && (stride != 1 || n > g.S || g.t2d);    // needs per-key positions

  if (tid == 0) {
    mbar_init(bar(C::B_Q), 1);
    for (int s = 0; s < C::NK; ++s) { mbar_init(bar(C::B_KF + s), 1); mbar_init(bar(C::B_KE + s), 1); }
    for (int s = 0; s < 4; ++s) { mbar_init(bar(C::B_SF + s), 1); mbar_init(bar(C::B_SE + s), 4); }
    *abort_flag = 0;
    mbar_init_fence();
  }
  if (warp == ARM_TMA_WARP) {
    if (lane == 0) { prefetch_tmap(map_q); prefetch_tmap(map_k); }
    __syncwarp();
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), 512);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const WaitCtx wc{abort_flag, arm_flag};

  if (warp >= 8) {
    RF_SETMAXNREG_DEC();
    if (warp == ARM_TMA_WARP) {
      if (lane == 0) {
        mbar_expect_tx(bar(C::B_Q), 2 * C::TILE);
#pragma unroll
        for (int j = 0; j < 2; ++j)
#pragma unroll
          for (int kb = 0; kb < C::KB; ++kb)
            tma_load_3d(base + C::Q + j * C::TILE + kb * C::BLK, map_q, kb * C::COL1, (qt0 + j) * ARM_TILE, bh, bar(C::B_Q));
        for (int u = 0; u < nt; ++u) {
          const int ks = u % C::NK;
          if (u >= C::NK) mbar_wait(bar(C::B_KE + ks), ((u / C::NK) - 1) & 1, wc);
          mbar_expect_tx(bar(C::B_KF + ks), C::TILE);
#pragma unroll
          for (int kb = 0; kb < C::KB; ++kb)
            tma_load_3d(base + C::K0 + ks * C::TILE + kb * C::BLK, map_k, kb * C::COL1, u * ARM_TILE, bh, bar(C::B_KF + ks));
        }
      }
    } else if (warp == ARM_MMA_WARP) {
      if (lane == 0) {
        constexpr uint32_t DESC_HI = (1024u >> 4) | (1u << 14) | (2u << 29);
        auto desc = [](uint32_t lo) -> uint64_t { return ((uint64_t)DESC_HI << 32) | lo; };
        const uint32_t q_lo = ((base + C::Q) >> 4) | (1u << 16), k_lo = ((base + C::K0) >> 4) | (1u << 16);
        mbar_wait(bar(C::B_Q), 0, wc);
        for (int u = 0; u < nt; ++u) {
          const int ks = u % C::NK, b = u & 1;
          mbar_wait(bar(C::B_KF + ks), (u / C::NK) & 1, wc);
#pragma unroll
          for (int j = 0; j < 2; ++j) {
            if (j == 1 && !stream1) continue;
            if (u >= 2) mbar_wait(bar(C::B_SE + j * 2 + b), ((u >> 1) - 1) & 1, wc);
            tc_fence_after();
            const uint32_t a0 = q_lo + j * (C::TILE >> 4), b0 = k_lo + ks * (C::TILE >> 4);
#pragma unroll
            for (int k = 0; k < D / 16; ++k)
              mma_ss(tmem_base + (j * 2 + b) * 128, desc(a0 + (C::koff(k) >> 4)), desc(b0 + (C::koff(k) >> 4)), IDESC_S, k > 0);
            tc_commit(bar(C::B_SF + j * 2 + b));
          }
          tc_commit(bar(C::B_KE + ks));
        }
      }
    }
  } else {
    RF_SETMAXNREG_INC();
    const int j = warp >> 2;
    if (j == 0 || stream1) {
      const int m = (qt0 + j) * ARM_TILE + (tid & 127);          // sampled row of this thread
      const int mc = min(m, n - 1);
      const int tok = mc * stride;
      const int rf = tok / g.S, rp = tok - rf * g.S;
      const int ry = rp / g.Wf, rx = rp - ry * g.Wf;
      // Masks k = 0..NB-1: Temporal with window win.ws[k]; k = NB..2NB-1: Spatial with win.wf[k-NB];
      // k = 2NB: Textural.  Band masks keep one key interval [lo, hi) per row in sample-index space.
      constexpr int NM = 2 * NB + 1;
      int lo[2 * NB], hi[2 * NB];
#pragma unroll
      for (int i = 0; i < NB; ++i) {
        lo[i] = rp - win.ws[i];                                     // first-frame sample: position = index
        hi[i] = rp + win.ws[i] + 1;
        lo[NB + i] = rf_cdiv(max(rf - win.wf[i], 0) * g.S, stride);  // stride sample: frames grow with the index
        hi[NB + i] = rf_cdiv((rf + win.wf[i] + 1) * g.S, stride);
      }
      const uint32_t t_s = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + j * 256;
      int* attr_p = reinterpret_cast<int*>(base_ptr + C::ATTR) + warp * 256;           // per-warp tables
      int* attr_c = attr_p + 128;
      float mx = -INFINITY, l_all = 0.f;
      float l_m[NM];
#pragma unroll
      for (int k = 0; k < NM; ++k) l_m[k] = 0.f;

      for (int u = 0; u < nt; ++u) {
        const int b = u & 1, u0 = u * ARM_TILE;
        mbar_wait(bar(C::B_SF + j * 2 + b), (u >> 1) & 1, wc);
        tc_fence_after();
        uint32_t s[128];
        {
          uint32_t(&s0)[32] = *reinterpret_cast<uint32_t(*)[32]>(&s[0]);
          uint32_t(&s1)[32] = *reinterpret_cast<uint32_t(*)[32]>(&s[32]);
          uint32_t(&s2)[32] = *reinterpret_cast<uint32_t(*)[32]>(&s[64]);
          uint32_t(&s3)[32] = *reinterpret_cast<uint32_t(*)[32]>(&s[96]);
          tmem_ld32(t_s + b * 128, s0);
          tmem_ld32(t_s + b * 128 + 32, s1);
          tmem_ld32(t_s + b * 128 + 64, s2);
          tmem_ld32(t_s + b * 128 + 96, s3);
          tc_wait_ld();
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(C::B_SE + j * 2 + b));   // the buffer may be refilled

        if (u0 + ARM_TILE > n) {                                 // keys past the sample
#pragma unroll
          for (int c = 0; c < 128; ++c)
            if (u0 + c >= n) s[c] = 0xff800000u;
        }
        float m0 = -INFINITY, m1 = -INFINITY;
#pragma unroll
        for (int c = 0; c < 128; c += 4) {
          m0 = fmaxf(m0, fmaxf(__uint_as_float(s[c]), __uint_as_float(s[c + 1])));
          m1 = fmaxf(m1, fmaxf(__uint_as_float(s[c + 2]), __uint_as_float(s[c + 3])));
        }
        const float m_new = fmaxf(mx, fmaxf(m0, m1) * scale_log2);   // finite: every tile holds a real key
        const float corr = ex2f(mx - m_new);
        l_all *= corr;
#pragma unroll
        for (int k = 0; k < NM; ++k) l_m[k] *= corr;
        mx = m_new;

        // exponentials once, in place; their sum serves every mask the tile lies wholly inside
        const float2 sc2 = make_float2(scale_log2, scale_log2), mneg = make_float2(-m_new, -m_new);
        float2 la = make_float2(0.f, 0.f), lb = make_float2(0.f, 0.f);
#pragma unroll
        for (int c = 0; c < 128; c += 4) {
          float2 e0 = __ffma2_rn(make_float2(__uint_as_float(s[c]), __uint_as_float(s[c + 1])), sc2, mneg);
          float2 e1 = __ffma2_rn(make_float2(__uint_as_float(s[c + 2]), __uint_as_float(s[c + 3])), sc2, mneg);
          e0.x = ex2f(e0.x); e0.y = ex2f(e0.y);
          e1.x = ex2f(e1.x); e1.y = ex2f(e1.y);
          la = __fadd2_rn(la, e0);
          lb = __fadd2_rn(lb, e1);
          s[c] = __float_as_uint(e0.x); s[c + 1] = __float_as_uint(e0.y);
          s[c + 2] = __float_as_uint(e1.x); s[c + 3] = __float_as_uint(e1.y);
        }
        const float bs = (la.x + la.y) + (lb.x + lb.y);
        l_all += bs;

        // per mask: the tile lies inside the row's kept interval for the whole warp (add the tile sum),
        // outside it (nothing), or an edge crosses it (masked sum with a 128-bit keep word)
        const int u1 = min(u0 + ARM_TILE, n);
        bool table_ready = false;
#pragma unroll 1
        for (int k = 0; k < NM; ++k) {
          const bool is_t = k < NB, is_x = k == 2 * NB;
          if (is_x ? !TEX : (is_t ? !sm.want_t : !sm.want_s)) continue;
          const bool by_table = is_x || (is_t && t_generic);
          int cls = 1;
          int klo = 0, khi = 0, pre = 0;
          if (!by_table) {
#pragma unroll
            for (int i = 0; i < 2 * NB; ++i)
              if (i == k) { klo = lo[i]; khi = hi[i]; }
            // Spatial masks with the first frame as key frame also keep the sampled keys of frame 0: a prefix
            // [0, pre) of the stride sample, the same for every row
            pre = (!is_t && g.key_first) ? rf_cdiv(g.S, stride) : 0;
            const bool in = (klo <= u0 && u1 <= khi) || u1 <= pre, out = (u1 <= klo || khi <= u0) && u0 >= pre;
            cls = __all_sync(0xffffffffu, in) ? 2 : (__all_sync(0xffffffffu, out) ? 0 : 1);
          }
          float add = 0.f;
          if (cls == 2) {
            add = bs;
          } else if (cls == 1) {
            uint32_t w[4] = {0, 0, 0, 0};
            if (!by_table) {
              interval_bits(w, u0, klo, khi);
              if (pre > u0) {
                uint32_t wp[4];
                interval_bits(wp, u0, 0, pre);
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4) w[q4] |= wp[q4];
              }
            } else {
              if (!table_ready) {
                // per-key attributes of the tile, four keys per lane, into this warp's table
                __syncwarp();
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                  const int c = lane * 4 + i;
                  const int ktok = min(u0 + c, n - 1) * stride;
                  const int kp = ktok % g.S;
                  const int y = kp / g.Wf, x = kp - y * g.Wf;
                  attr_p[c] = g.t2d ? ((y << 16) | x) : kp;    // frame dimensions stay below 2^15 with the 2-D window
                  attr_c[c] = (y % g.tau) == (x % g.tau);
                }
                __syncwarp();
                table_ready = true;
              }
              int wk = 0;
#pragma unroll
              for (int i = 0; i < NB; ++i)
                if (i == k) wk = win.ws[i];
#pragma unroll
              for (int q4 = 0; q4 < 4; ++q4) {
                uint32_t bits = 0;
#pragma unroll 8
                for (int c = 0; c < 32; ++c) {
                  bool keep;
                  if (is_x) {
                    keep = attr_c[q4 * 32 + c] != 0;
                  } else if (g.t2d) {
                    const int yx = attr_p[q4 * 32 + c];
                    keep = abs((yx >> 16) - ry) <= g.wy && abs((yx & 0xffff) - rx) <= g.wx;
                  } else {
                    const int dp = attr_p[q4 * 32 + c] - rp;
                    keep = (dp < 0 ? -dp : dp) <= wk;
                  }
                  bits |= (keep ? 1u : 0u) << c;
                }
                w[q4] = bits;
              }
            }
#pragma unroll
            for (int c = 0; c < 128; ++c)
              if ((w[c >> 5] >> (c & 31)) & 1u) add += __uint_as_float(s[c]);
          }
#pragma unroll
          for (int i = 0; i < NM; ++i)
            if (i == k) l_m[i] += add;
        }
      }
      if (m < n) {
        float* out = sm.out + (size_t)bh * NM * n_pad;
        const float inv = 1.f / l_all;
#pragma unroll
        for (int k = 0; k < NM; ++k) {
          const bool is_t = k < NB, is_x = k == 2 * NB;
          if ((is_x ? TEX : (is_t ? sm.want_t != 0 : sm.want_s != 0)) && rf_in_bounds(m, n_pad, arm_flag))
            out[(size_t)k * n_pad + m] = l_m[k] * inv;
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == ARM_TMA_WARP) {
    if (*abort_flag) __nanosleep(20000);
    __syncwarp();
    tmem_dealloc(tmem_base, 512);
  }
}

// One CTA per head: means of the per-row recalls in a fixed order, then the decision.
//   plain (head_window == nullptr, nb = 1): Algorithm 1.
//   dynamic bandwidth: a pattern qualifies if any candidate window reaches alpha, Temporal before Spatial;
//   the head takes the smallest qualifying window (candidates ascend); Textural heads get window -1.
__global__ void __launch_bounds__(256) rf_arm_decide_kernel(int nb, int nb_user, int n_loc, int n_glb, int n_pad, int sample_mode,
                                                             float alpha, int two_mask, ArmWindows win, int with_tex,
                                                             const float* __restrict__ rows_loc,
                                                             const float* __restrict__ rows_glb,
                                                             int32_t* __restrict__ head_class,
                                                             int32_t* __restrict__ head_window, float* __restrict__ recall,
                                                             float* __restrict__ recall_plus,
                                                             const int32_t* __restrict__ arm_flag, int32_t* dev_status) {
  __shared__ double red[2 * ARM_MAX_NB + 1][256];
  const int bh = blockIdx.x, tid = threadIdx.x;
  const int nm = 2 * nb + 1;
  const int failed = *arm_flag;
  if (failed != 0) {
    // the score kernel gave up a wait: its rows are incomplete, no class may come out of them
    if (tid == 0) {
      rf_report(dev_status, failed);
      head_class[bh] = -1;
      if (head_window != nullptr) head_window[bh] = -1;
    }
    return;
  }
  const float* gl = rows_glb + (size_t)bh * nm * n_pad;
  const float* lo = rows_loc + (size_t)bh * nm * n_pad;
  const bool local_t = sample_mode == RF_SAMPLE_ALG1;
  for (int k = 0; k < nm; ++k) {
    const bool is_t = k < nb, is_x = k == 2 * nb;
    const float* src = ((is_t && local_t) ? lo : gl) + (size_t)k * n_pad;
    const int cnt = (is_t && local_t) ? n_loc : n_glb;
    double acc = 0.0;
    if (!is_x || with_tex)
      for (int i = tid; i < cnt; i += 256) acc += (double)src[i];
    red[k][tid] = acc;
  }
  __syncthreads();
  for (int o = 128; o > 0; o >>= 1) {
    if (tid < o)
      for (int k = 0; k < nm; ++k) red[k][tid] += red[k][tid + o];
    __syncthreads();
  }
  if (tid == 0) {
    float R[2 * ARM_MAX_NB + 1];
    for (int k = 0; k < nm; ++k) R[k] = (float)(red[k][0] / ((k < nb && local_t) ? n_loc : n_glb));
    if (head_window == nullptr) {
      const float Rt = R[0], Rs = R[nb], Rc = R[2 * nb];
      if (recall) { recall[bh * 3] = Rt; recall[bh * 3 + 1] = Rs; recall[bh * 3 + 2] = Rc; }
      // Algorithm 1; with only two masks (ablation) a head that reaches alpha with neither takes the larger recall
      const int otherwise = two_mask ? (Rt >= Rs ? RF_TEMPORAL : RF_SPATIAL) : RF_TEXTURAL;
      head_class[bh] = Rt >= alpha ? RF_TEMPORAL : (Rs >= alpha ? RF_SPATIAL : otherwise);
    } else {
      int cls = RF_TEXTURAL, window = -1;
      if (two_mask) {   // nothing qualifies: the larger recall at the widest candidate, with that bandwidth
        const bool t = R[nb_user - 1] >= R[nb + nb_user - 1];
        cls = t ? RF_TEMPORAL : RF_SPATIAL;
        window = t ? win.ws[nb_user - 1] : win.wf[nb_user - 1];
      }
      // nb slots were evaluated (the caller's nb_user candidates, padded by repeating the last one)
      for (int i = nb_user - 1; i >= 0; --i)
        if (R[nb + i] >= alpha) { cls = RF_SPATIAL; window = win.wf[i]; }
      for (int i = nb_user - 1; i >= 0; --i)
        if (R[i] >= alpha) { cls = RF_TEMPORAL; window = win.ws[i]; }
      head_class[bh] = cls;
      head_window[bh] = window;
      if (recall_plus)
        for (int i = 0; i < nb_user; ++i) {
          recall_plus[(bh * 2) * nb_user + i] = R[i];
          recall_plus[(bh * 2 + 1) * nb_user + i] = R[nb + i];
        }
    }
  }
}

// Self-test only: stands in for a score kernel whose wait ran out.
__global__ void rf_arm_set_flag_kernel(int32_t* arm_flag, int code) { *arm_flag = code; }

template <int D, int NB, bool TEX>
cudaError_t launch_arm_t(const ArmMaps& maps, const RfGeom& g, const ArmSample& s0, const ArmSample& s1,
                         const ArmWindows& win, int n_pad, int32_t* arm_flag, cudaStream_t st) {
  static bool configured[64] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev >= 0 && dev < 64 && !configured[dev]) {
    if (!rf_regs_ok(rf_arm_kernel<D, NB, TEX>)) return cudaErrorLaunchOutOfResources;   // setmaxnreg.inc could never be granted
    e = cudaFuncSetAttribute(rf_arm_kernel<D, NB, TEX>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ArmCfg<D>::ALLOC);
    if (e != cudaSuccess) return e;
    configured[dev] = true;
  }
  dim3 grid(s0.pairs + s1.pairs, g.B * g.H);
  const float scale_log2 = 1.4426950408889634f / sqrtf((float)D);
  rf_arm_kernel<D, NB, TEX><<<grid, ARM_THREADS, ArmCfg<D>::ALLOC, st>>>(maps, g, s0, s1, win, n_pad, scale_log2, arm_flag);
  return cudaGetLastError();
}

template <int D>
cudaError_t launch_arm_n(bool plus, bool tex, const ArmMaps& maps, const RfGeom& g, const ArmSample& s0,
                         const ArmSample& s1, const ArmWindows& win, int n_pad, int32_t* arm_flag, cudaStream_t st) {
  if (plus) return launch_arm_t<D, ARM_MAX_NB, false>(maps, g, s0, s1, win, n_pad, arm_flag, st);
  return tex ? launch_arm_t<D, 1, true>(maps, g, s0, s1, win, n_pad, arm_flag, st)
             : launch_arm_t<D, 1, false>(maps, g, s0, s1, win, n_pad, arm_flag, st);
}

int arm_n_pad(const RfGeom& g, int omega) {
  const int n_glb = rf_cdiv(g.Nv, omega);
  const int n = n_glb > g.S ? n_glb : g.S;
  return (n + 63) / 64 * 64;
}

}  // namespace

// Per-row recalls of both samples, then RF_ARM_FLAG_FLOATS floats whose first word is the call's failure flag.
size_t rf_arm_scratch_floats(const RfGeom& g, int omega, int nb) {
  return (size_t)2 * g.B * g.H * (2 * nb + 1) * arm_n_pad(g, omega) + RF_ARM_FLAG_FLOATS;
}

cudaError_t rf_launch_arm(const RfGeom& g, int sample_mode, int omega, float alpha, int nb, const int* ws_list,
                          const int* wf_list, const __nv_bfloat16* q, const __nv_bfloat16* k, int32_t* head_class,
                          int32_t* head_window, float* recall, float* recall_plus, float* row_scratch, int32_t* dev_status,
                          cudaStream_t st, bool selftest_abandon) {
  const bool plus = head_window != nullptr;
  const int NB = plus ? ARM_MAX_NB : 1;           // windows the kernel evaluates (candidate list padded by repetition)
  if (nb < 1 || nb > NB) return cudaErrorInvalidValue;
  ArmWindows win;
  for (int i = 0; i < ARM_MAX_NB; ++i) {
    win.ws[i] = ws_list[i < nb ? i : nb - 1];
    win.wf[i] = wf_list[i < nb ? i : nb - 1];
  }
  const int n_pad = arm_n_pad(g, omega);
  const int n_glb = rf_cdiv(g.Nv, omega), n_loc = g.S;
  const int heads = g.B * g.H;
  float* rows_glb = row_scratch;
  float* rows_loc = row_scratch + (size_t)heads * (2 * NB + 1) * n_pad;
  int32_t* arm_flag = reinterpret_cast<int32_t*>(row_scratch + (size_t)2 * heads * (2 * NB + 1) * n_pad);
  const bool alg1 = sample_mode == RF_SAMPLE_ALG1;
  const bool tex = !plus && recall != nullptr;   // the Textural recall is a diagnostic: Algorithm 1 does not use it
  const size_t row_bytes = (size_t)g.D * 2, head_bytes = (size_t)g.N * g.D * 2;
  ArmMaps maps;
  bool ok = rf_encode_rows_map(&maps.q[0], q, g.D, n_glb, row_bytes * omega, head_bytes, heads) &&
            rf_encode_rows_map(&maps.k[0], k, g.D, n_glb, row_bytes * omega, head_bytes, heads) &&
            rf_encode_rows_map(&maps.q[1], q, g.D, n_loc, row_bytes, head_bytes, heads) &&
            rf_encode_rows_map(&maps.k[1], k, g.D, n_loc, row_bytes, head_bytes, heads);
  if (!ok) return cudaErrorUnknown;
  ArmSample s0, s1;
  s0.n = n_glb; s0.stride = omega; s0.pairs = rf_cdiv(rf_cdiv(n_glb, ARM_TILE), 2);
  s0.want_t = alg1 ? 0 : 1; s0.want_s = 1; s0.out = rows_glb;
  s1.n = n_loc; s1.stride = 1; s1.pairs = alg1 ? rf_cdiv(rf_cdiv(n_loc, ARM_TILE), 2) : 0;
  s1.want_t = 1; s1.want_s = 0; s1.out = rows_loc;
  cudaError_t e = cudaMemsetAsync(arm_flag, 0, sizeof(int32_t), st);
  if (e != cudaSuccess) return e;
  if (selftest_abandon) {
    rf_arm_set_flag_kernel<<<1, 1, 0, st>>>(arm_flag, RF_ERR_TIMEOUT);
    e = cudaGetLastError();
  } else
  switch (g.D) {
    case 64: e = launch_arm_n<64>(plus, tex, maps, g, s0, s1, win, n_pad, arm_flag, st); break;
    case 96: e = launch_arm_n<96>(plus, tex, maps, g, s0, s1, win, n_pad, arm_flag, st); break;
    case 128: e = launch_arm_n<128>(plus, tex, maps, g, s0, s1, win, n_pad, arm_flag, st); break;
    default: e = cudaErrorInvalidValue;
  }
  if (e != cudaSuccess) return e;
  rf_arm_decide_kernel<<<heads, 256, 0, st>>>(NB, nb, n_loc, n_glb, n_pad, sample_mode, alpha, g.two_mask, win, tex ? 1 : 0, rows_loc,
                                              rows_glb, head_class, head_window, recall, recall_plus, arm_flag, dev_status);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
// Entry point for callers that can neither pass a workspace nor allocate one: the per-row recall
// scratch is a fixed array in this library's device image.
// ------------------------------------------------------------------------------------------------
static __device__ __align__(256) float g_arm_static_scratch[RF_ARM_STATIC_SCRATCH_FLOATS];

namespace {
// Device address of g_arm_static_scratch per device.  In host code the array's name is only a
// handle for the runtime, not a pointer a kernel may use; the address comes from cudaGetSymbolAddress
// with the device in question current.
float* static_scratch_ptr(int dev, cudaError_t* err) {
  static float* ptrs[64] = {};
  *err = cudaSuccess;
  if (dev < 0 || dev >= 64) { *err = cudaErrorInvalidDevice; return nullptr; }
  if (ptrs[dev] == nullptr) {
    void* p = nullptr;
    *err = cudaGetSymbolAddress(&p, g_arm_static_scratch);
    if (*err != cudaSuccess) return nullptr;
    ptrs[dev] = static_cast<float*>(p);
  }
  return ptrs[dev];
}
}  // namespace

extern "C" rf_status rf_arm_classify_noalloc(const rf_shape* shape, const rf_params* params, const void* q,
                                             const void* k, int32_t* head_class, float* recall, int32_t* dev_status,
                                             void* cuda_stream) {
  RfGeom g;
  rf_status st = rf_checked_geom(shape, params, &g);
  if (st != RF_OK) return st;
  if (g.D != 64 && g.D != 96 && g.D != 128) return RF_ERR_UNSUPPORTED;
  if (q == nullptr || k == nullptr || head_class == nullptr) return RF_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(q) & 15u) != 0 || (reinterpret_cast<uintptr_t>(k) & 15u) != 0) return RF_ERR_INVALID_ARG;
  if (rf_arm_scratch_floats(g, params->sample_stride, 1) > (size_t)RF_ARM_STATIC_SCRATCH_FLOATS)
    return RF_ERR_STATIC_SCRATCH_TOO_SMALL;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return RF_ERR_CUDA;
  cudaError_t e;
  float* scratch = static_scratch_ptr(dev, &e);
  if (scratch == nullptr) return RF_ERR_CUDA;
  e = rf_launch_arm(g, params->sample_mode, params->sample_stride, params->alpha, 1, &g.ws, &g.wf,
                    static_cast<const __nv_bfloat16*>(q), static_cast<const __nv_bfloat16*>(k), head_class, nullptr, recall,
                    nullptr, scratch, dev_status, static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? RF_OK : RF_ERR_CUDA;
}
