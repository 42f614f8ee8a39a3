// Pieces shared by the attention kernels: the element mask of one query row per tile, the two query tiles'
// KV-tile lists and their merge, small arithmetic helpers.
#pragma once

#include "rf_sm100.cuh"

namespace rf_attn {

using namespace sm100;

constexpr int BM = 128, BN = 128;

// The two bf16 values of a packed word, widened exactly.  The row sum is taken over these rounded weights, the
// ones the tensor core multiplies with V: O / l is then an exact convex combination of V rows with slightly
// perturbed weights, and the rounding of a dominant weight cancels instead of scaling the whole output row.
__device__ __forceinline__ float2 unpack_bf16(uint32_t w) {
  return make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
}

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Element mask of one query row in the head's key-slot space, evaluated per tile as a 128-bit word
// (bit c = key slot u0 + c kept).  Every pattern's kept set is a union of a few slot intervals:
// one window [lo, hi) (Spatial, position-major Temporal), one band per frame (Temporal in original
// order) and the always-kept text slots [text0, lkv).  Kept compact on purpose: PARTIAL tiles are
// rare, and a large rarely-run code block costs more in instruction fetch than in arithmetic.
struct RowMask {
  int lo, hi;        // kRange: kept video slots [lo, hi)
  int first_end;     // slots [0, first_end) are kept as well (Spatial with the first frame as key frame), else 0
  int text0;         // first always-kept (text) slot
  int lkv;           // number of key slots
  int p, ws, S, T;   // kPeriodic: |slot % S - p| <= ws for slots of frames 0..T-1
  uint8_t mode;      // kRange: [lo, hi) and [0, first_end); kPeriodic: p +- ws in every frame; kWindow2d: see window2d_bits
  enum : uint8_t { kRange = 0, kPeriodic = 1, kWindow2d = 2 };

  static __device__ __forceinline__ uint32_t below(int n) {  // bits [0, n) set, n in [0, 32]
    return n >= 32 ? 0xffffffffu : ((1u << n) - 1u);
  }
  // OR the slots [a, b) (absolute) into the tile's words.
  static __device__ __forceinline__ void add(uint32_t (&w)[4], int u0, int a, int b) {
    a = max(a - u0, 0);
    b = min(b - u0, BN);
    if (a >= b) return;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int lo_k = min(max(a - 32 * k, 0), 32), hi_k = min(max(b - 32 * k, 0), 32);
      w[k] |= below(hi_k) & ~below(lo_k);
    }
  }
  // mode == kWindow2d, a Temporal head with the 2-D in-frame window: the kept positions of query position
  // p = y*W + x are, for each frame row y' within wy of y, the run [y'*W + x - wx, y'*W + x + wx] clipped to the row.
  // In position-major order a position is T consecutive slots; in original order it recurs in every frame.  Only the
  // rows the tile reaches are visited.  The fields the other modes use carry the frame's width and the window:
  // lo = W, hi = wy, first_end = wx.
  __device__ __forceinline__ void window2d_bits(int u0, uint32_t (&w)[4]) const {
    const int W = lo, H = S / W, wy = hi, wx = first_end;
    const int yq = p / W, xq = p - yq * W;
    const int xlo = max(xq - wx, 0), xhi = min(xq + wx, W - 1);
    const int ylo = max(yq - wy, 0), yhi = min(yq + wy, H - 1);
    if (ws) {  // position-major slots
      const int pa = u0 / T, pb = min((u0 + BN - 1) / T, S - 1);                   // positions the tile reaches
      for (int y = max(ylo, pa / W); y <= min(yhi, pb / W); ++y) add(w, u0, (y * W + xlo) * T, (y * W + xhi + 1) * T);
    } else {
      const int f1 = min((u0 + BN - 1) / S, T - 1);
      for (int f = u0 / S; f <= f1; ++f) {
        const int pa = max(u0 - f * S, 0), pb = min(u0 + BN - 1 - f * S, S - 1);   // positions of frame f the tile reaches
        for (int y = max(ylo, pa / W); y <= min(yhi, pb / W); ++y) add(w, u0, f * S + y * W + xlo, f * S + y * W + xhi + 1);
      }
    }
  }
  __device__ __noinline__ void tile_bits(int u0, uint32_t (&w)[4]) const {
    w[0] = w[1] = w[2] = w[3] = 0u;
    if (mode == kWindow2d) {
      window2d_bits(u0, w);
    } else if (mode == kPeriodic) {
      const int f1 = min((u0 + BN - 1) / S, T - 1);
      for (int f = u0 / S; f <= f1; ++f) add(w, u0, f * S + max(p - ws, 0), f * S + min(p + ws, S - 1) + 1);
    } else {
      add(w, u0, lo, min(hi, text0));
      add(w, u0, 0, first_end);
    }
    add(w, u0, text0, lkv);
  }
};

__device__ __forceinline__ RowMask make_row_mask(const RfGeom& g, int cls, int r) {
  RowMask m;
  m.lkv = rf_kv_len(g, cls);
  m.text0 = m.lkv;
  m.lo = 0;
  m.hi = m.lkv;
  m.first_end = 0;
  m.p = 0; m.ws = g.ws; m.S = g.S; m.T = g.T;
  m.mode = RowMask::kRange;
  if ((cls == RF_SPATIAL || cls == RF_TEMPORAL) && r < g.Nv) {
    m.text0 = g.Nv;
    if (cls == RF_SPATIAL) {
      const int f = r / g.S;
      m.lo = max(0, f - g.wf) * g.S;
      m.hi = min(g.T, f + g.wf + 1) * g.S;
      m.first_end = g.key_first ? g.S : 0;
    } else if (g.t2d) {
      m.mode = RowMask::kWindow2d;
      m.p = g.permute ? r / g.T : r % g.S;
      m.lo = g.Wf; m.hi = g.wy; m.first_end = g.wx;
      m.ws = g.permute;
    } else if (g.permute) {
      const int p = r / g.T;
      m.lo = max(0, p - g.ws) * g.T;
      m.hi = min(g.S, p + g.ws + 1) * g.T;
    } else {
      m.mode = RowMask::kPeriodic;
      m.p = r % g.S;
    }
  }
  return m;
}

// Exact maximum of this thread's row of the S tile at t_s (slow path of the softmax; warp-collective loads).
static __device__ __noinline__ float tile_row_max(uint32_t t_s, bool partial, const RowMask& rmask, int u0) {
  uint32_t w[4] = {0xffffffffu, 0xffffffffu, 0xffffffffu, 0xffffffffu};
  if (partial) rmask.tile_bits(u0, w);
  float mx = -INFINITY;
#pragma unroll 1
  for (int q = 0; q < 4; ++q) {
    uint32_t v[32];
    tmem_ld32(t_s + q * 32, v);
    tc_wait_ld();
#pragma unroll
    for (int c = 0; c < 32; ++c)
      if ((w[q] >> c) & 1u) mx = fmaxf(mx, __uint_as_float(v[c]));
  }
  return mx;
}

// The two streams' ascending tile lists and their merge (the order K/V tiles are fetched in).
struct Lists {
  const int32_t* l0;
  const int32_t* l1;
  int n0, n1;
  int lkv;
  bool listed;
  __device__ __forceinline__ uint32_t entry(int j, int i) const {
    if (listed) return (uint32_t)(j == 0 ? l0[i] : l1[i]);
    const bool tail = (i + 1) * BN > lkv;
    return (uint32_t)i | (tail ? RF_PARTIAL_BIT : 0u);
  }
};
struct Merge {
  int i0 = 0, i1 = 0;
  // Raw list entries at i0 / i1, loaded by the previous call and not touched until the next one, so
  // that the load latency never sits between two MMA bursts of the (in-order) issuing thread.
  uint32_t raw0 = 0, raw1 = 0;
  __device__ __forceinline__ void start(const Lists& L) {
    if (L.n0 > 0) raw0 = L.entry(0, 0);
    if (L.n1 > 0) raw1 = L.entry(1, 0);
  }
  // Next tile of the union; uses bit j set when stream j lists it.  Returns false when exhausted.
  __device__ __forceinline__ bool next(const Lists& L, int& tile, int& uses) {
    const int h0 = i0 < L.n0 ? (int)(raw0 & ~RF_PARTIAL_BIT) : 0x7fffffff;
    const int h1 = i1 < L.n1 ? (int)(raw1 & ~RF_PARTIAL_BIT) : 0x7fffffff;
    tile = min(h0, h1);
    if (tile == 0x7fffffff) return false;
    uses = (h0 == tile ? 1 : 0) | (h1 == tile ? 2 : 0);
    if ((uses & 1) && ++i0 < L.n0) raw0 = L.entry(0, i0);
    if ((uses & 2) && ++i1 < L.n1) raw1 = L.entry(1, i1);
    return true;
  }
};

}  // namespace rf_attn
