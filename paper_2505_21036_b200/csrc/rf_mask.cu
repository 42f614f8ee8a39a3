// Block-mask / tile-schedule builder and the token reordering gathers.
//
// The pattern masks of Sec. 3.2 (Spatial: Eq. 3, Temporal, Textural: Eq. 4-5) are evaluated in
// closed form per tile: a tile's query slots and key slots each cover a contiguous range of
// frames (Spatial), of in-frame positions (Temporal in position-major order) or a cyclic range
// of positions (Temporal in original order), so "some pair kept" and "all pairs kept" reduce to
// distances between at most two intervals per side.
#include "rf_common.cuh"

namespace {

struct Iv { int lo, hi; };  // closed interval

// Positions (index mod S) covered by slots [a0, a1) of the original order: one or two intervals.
__device__ __forceinline__ int cyclic_intervals(int a0, int a1, int S, Iv out[2]) {
  if (a1 - a0 >= S) { out[0] = {0, S - 1}; return 1; }
  int s = a0 % S, e = (a1 - 1) % S;
  if (s <= e) { out[0] = {s, e}; return 1; }
  out[0] = {s, S - 1};
  out[1] = {0, e};
  return 2;
}

// 2-D in-frame window between two runs of consecutive positions A = [a0, a1] and B = [b0, b1] (row-major positions
// of a frame of width W): `any` - some pair (p in A, p' in B) has |dy| <= wy and |dx| <= wx; `all` - every pair has.
// A run of positions is up to three rectangles (a partial first row, whole rows, a partial last row); between two
// rectangles the smallest and largest |dy| and |dx| follow from the interval ends.
struct Rect { int y0, y1, x0, x1; };
__device__ __forceinline__ int run_rects(int p0, int p1, int W, Rect out[3]) {
  const int ya = p0 / W, xa = p0 - ya * W, yb = p1 / W, xb = p1 - yb * W;
  if (ya == yb) { out[0] = {ya, ya, xa, xb}; return 1; }
  int n = 0;
  out[n++] = {ya, ya, xa, W - 1};
  if (yb - ya > 1) out[n++] = {ya + 1, yb - 1, 0, W - 1};
  out[n++] = {yb, yb, 0, xb};
  return n;
}
__device__ void window2d(const Iv& A, const Iv& B, int W, int wy, int wx, bool& any, bool& all) {
  Rect ra[3], rb[3];
  const int na = run_rects(A.lo, A.hi, W, ra), nb = run_rects(B.lo, B.hi, W, rb);
  for (int i = 0; i < na; ++i)
    for (int j = 0; j < nb; ++j) {
      const int gy = max(max(rb[j].y0 - ra[i].y1, ra[i].y0 - rb[j].y1), 0), gx = max(max(rb[j].x0 - ra[i].x1, ra[i].x0 - rb[j].x1), 0);
      const int sy = max(ra[i].y1 - rb[j].y0, rb[j].y1 - ra[i].y0), sx = max(ra[i].x1 - rb[j].x0, rb[j].x1 - ra[i].x0);
      any = any || (gy <= wy && gx <= wx);
      all = all && (sy <= wy && sx <= wx);
    }
}

// 0: empty, 1: PARTIAL, 2: FULL.  Tile (a, b) of a head of class cls.
__device__ int tile_flag(const RfGeom& g, int cls, int a, int b) {
  const int Lkv = rf_kv_len(g, cls);
  const int r0 = a * g.BM, r1 = min(r0 + g.BM, g.N);
  const int u0 = b * g.BN, u1 = min(u0 + g.BN, Lkv);
  if (r0 >= r1 || u0 >= u1) return 0;
  const bool full_width = (b + 1) * g.BN <= Lkv;
  bool any = true, all = true;
  if (cls == RF_SPATIAL || cls == RF_TEMPORAL) {
    const int Nv = g.Nv;
    const bool text_row = r1 > Nv, text_col = u1 > Nv;
    const bool video_part = r0 < Nv && u0 < Nv;
    bool vv_any = false, vv_all = true;
    if (video_part) {
      const int rv1 = min(r1, Nv), uv1 = min(u1, Nv);
      if (cls == RF_TEMPORAL && g.t2d) {
        // 2-D in-frame window: the tile's query and key slots each cover one run of positions (position-major
        // order) or a run that may wrap round the frame's end (original order)
        Iv R[2], C[2];
        int nr, nc;
        if (g.permute) {
          R[0] = {r0 / g.T, (rv1 - 1) / g.T};
          C[0] = {u0 / g.T, (uv1 - 1) / g.T};
          nr = nc = 1;
        } else {
          nr = cyclic_intervals(r0, rv1, g.S, R);
          nc = cyclic_intervals(u0, uv1, g.S, C);
        }
        for (int i = 0; i < nr; ++i)
          for (int j = 0; j < nc; ++j) window2d(R[i], C[j], g.Wf, g.wy, g.wx, vv_any, vv_all);
      } else if (cls == RF_SPATIAL || g.permute) {
        // contiguous ranges of frames (Spatial) or of positions (position-major Temporal)
        const int unit = cls == RF_SPATIAL ? g.S : g.T;
        const int w = cls == RF_SPATIAL ? g.wf : g.ws;
        const int ra = r0 / unit, rb = (rv1 - 1) / unit, ca = u0 / unit, cb = (uv1 - 1) / unit;
        vv_any = max(max(ca - rb, ra - cb), 0) <= w;
        vv_all = max(rb - ca, cb - ra) <= w;
        if (cls == RF_SPATIAL && g.key_first) {
          // keys of frame 0 are kept for every query: the tile is non-empty if it reaches into frame 0, and all of
          // it is kept if the window holds for its keys of the other frames (if it has any)
          vv_any = vv_any || ca == 0;
          vv_all = cb == 0 || max(rb - max(ca, 1), cb - ra) <= w;
        }
      } else {
        Iv R[2], C[2];
        const int nr = cyclic_intervals(r0, rv1, g.S, R), nc = cyclic_intervals(u0, uv1, g.S, C);
        for (int i = 0; i < nr; ++i)
          for (int j = 0; j < nc; ++j) {
            vv_any = vv_any || max(max(C[j].lo - R[i].hi, R[i].lo - C[j].hi), 0) <= g.ws;
            vv_all = vv_all && max(R[i].hi - C[j].lo, C[j].hi - R[i].lo) <= g.ws;
          }
      }
    }
    any = text_row || text_col || vv_any;
    all = vv_all;
  }
  if (!any) return 0;
  return (all && full_width) ? 2 : 1;
}

// One warp per (query tile, head): flags for 32 key tiles at a time, ordered compaction by ballot.
// No block-level synchronisation; eight rows per CTA.
__global__ void __launch_bounds__(256) rf_build_tiles_kernel(RfGeom g, const int32_t* __restrict__ head_class,
                                                              const int32_t* __restrict__ head_window,
                                                              int32_t* __restrict__ count, int32_t* __restrict__ kv_tile,
                                                              uint32_t* __restrict__ bitmap, int32_t* __restrict__ kv_len,
                                                              int32_t* dev_status) {
  const int lane = threadIdx.x & 31;
  const int a = blockIdx.x * 8 + (threadIdx.x >> 5), bh = blockIdx.y;
  if (a >= g.nQ) return;   // whole warp
  int cls = head_class[bh];
  if (cls < 0 || cls > 3) {
    if (lane == 0) rf_report(dev_status, RF_ERR_INVALID_ARG);
    cls = RF_DENSE;
  }
  if (head_window != nullptr) {   // dynamic bandwidth: this head's own window
    const int w = head_window[bh];
    if (cls == RF_SPATIAL && w >= 0) g.wf = min(w, g.T);     // past the extent: same mask, no overflow
    if (cls == RF_TEMPORAL && w >= 0) g.ws = min(w, g.S);
  }
  const int Lkv = rf_kv_len(g, cls);
  const int nK = rf_cdiv(Lkv, g.BN);
  if (a == 0 && lane == 0 && rf_in_bounds(bh, (size_t)g.B * g.H, dev_status)) kv_len[bh] = Lkv;
  int32_t* row = kv_tile + ((size_t)bh * g.nQ + a) * g.nKmax;
  const int words = rf_cdiv(g.nKmax, 32);
  uint32_t* brow = bitmap ? bitmap + ((size_t)bh * g.nQ + a) * words : nullptr;
  int base = 0;
  for (int b0 = 0; b0 < words * 32; b0 += 32) {
    const int b = b0 + lane;
    const int f = (b < nK) ? tile_flag(g, cls, a, b) : 0;
    const unsigned m = __ballot_sync(0xffffffffu, f != 0);
    if (brow && lane == 0 && rf_in_bounds(b0 >> 5, words, dev_status)) brow[b0 >> 5] = m;
    if (f != 0) {
      const int slot = base + __popc(m & ((1u << lane) - 1));
      if (rf_in_bounds(slot, g.nKmax, dev_status)) row[slot] = (int32_t)((uint32_t)b | (f == 1 ? RF_PARTIAL_BIT : 0u));
    }
    base += __popc(m);
  }
  if (lane == 0 && rf_in_bounds((size_t)bh * g.nQ + a, (size_t)g.B * g.H * g.nQ, dev_status)) count[(size_t)bh * g.nQ + a] = base;
}

// Reordered copies for heads whose coordinate space is not the original one.
//   Temporal + permute: Q, K, V  -> slot pos*T + frame (text rows keep their index)
//   Textural:           K, V     -> frame*nC + rank(pos) for kept positions, text after T*nC
// One 16-byte vector per thread; grid.x walks source rows, grid.y = head.
__global__ void __launch_bounds__(256) rf_gather_kernel(RfGeom g, const int32_t* __restrict__ head_class,
                                                         const uint4* __restrict__ q, const uint4* __restrict__ k,
                                                         const uint4* __restrict__ v, uint4* __restrict__ wq,
                                                         uint4* __restrict__ wk, uint4* __restrict__ wv, int32_t* dev_status) {
  extern __shared__ int row_start[];  // [Hf] rank of the first kept token of each frame row (Textural)
  const int bh = blockIdx.y;
  const int cls = head_class[bh];
  const bool perm = cls == RF_TEMPORAL && g.permute;
  const bool tex = cls == RF_TEXTURAL;
  if (!perm && !tex) return;
  if (tex) {
    if (threadIdx.x == 0) {
      int acc = 0;
      for (int y = 0; y < g.Hf; ++y) {
        row_start[y] = acc;
        const int r = y % g.tau;
        acc += r < g.Wf ? (g.Wf - r + g.tau - 1) / g.tau : 0;
      }
    }
    __syncthreads();
  }
  const int vec = g.D / 8;  // uint4 per row
  const int rows_per_cta = 256 / vec;
  const int lr = threadIdx.x / vec, c = threadIdx.x % vec;
  if (lr >= rows_per_cta) return;
  const size_t head_off = (size_t)bh * g.N * vec;
  for (int i = blockIdx.x * rows_per_cta + lr; i < g.N; i += gridDim.x * rows_per_cta) {
    int dst;
    if (i >= g.Nv) {
      dst = tex ? g.T * g.nC + (i - g.Nv) : i;
    } else {
      const int f = i / g.S, p = i - f * g.S;
      if (perm) {
        dst = p * g.T + f;
      } else {
        const int y = p / g.Wf, x = p - y * g.Wf;
        if ((y % g.tau) != (x % g.tau)) continue;
        dst = f * g.nC + row_start[y] + x / g.tau;
      }
    }
    if (!rf_in_bounds(dst, perm ? g.N : g.LkvTex, dev_status)) continue;
    const size_t s = head_off + (size_t)i * vec + c, d = head_off + (size_t)dst * vec + c;
    if (perm) wq[d] = q[s];
    wk[d] = k[s];
    wv[d] = v[s];
  }
}

}  // namespace

cudaError_t rf_launch_build_tiles(const RfGeom& g, const int32_t* head_class, const int32_t* head_window, int32_t* count,
                                  int32_t* kv_tile, uint32_t* bitmap, int32_t* kv_len, int32_t* dev_status, cudaStream_t st) {
  dim3 grid(rf_cdiv(g.nQ, 8), g.B * g.H);
  rf_build_tiles_kernel<<<grid, 256, 0, st>>>(g, head_class, head_window, count, kv_tile, bitmap, kv_len, dev_status);
  return cudaGetLastError();
}

cudaError_t rf_launch_gather(const RfGeom& g, const int32_t* head_class, const __nv_bfloat16* q,
                             const __nv_bfloat16* k, const __nv_bfloat16* v, __nv_bfloat16* wq, __nv_bfloat16* wk,
                             __nv_bfloat16* wv, int32_t* dev_status, cudaStream_t st) {
  const int vec = g.D / 8;
  const int rows_per_cta = 256 / vec;
  int gx = rf_cdiv(g.N, rows_per_cta);
  if (gx > 148 * 8) gx = 148 * 8;
  dim3 grid(gx, g.B * g.H);
  rf_gather_kernel<<<grid, 256, g.Hf * sizeof(int), st>>>(g, head_class, (const uint4*)q, (const uint4*)k,
                                                           (const uint4*)v, (uint4*)wq, (uint4*)wk, (uint4*)wv, dev_status);
  return cudaGetLastError();
}
