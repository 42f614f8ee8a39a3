// ARM: Adaptive Recognition Module (Sec. 3.3, Eq. 6, Algorithm 1).
//
// For a sample I of video tokens (the first frame, or every omega-th token) each CTA takes 128
// sampled query rows and streams all sampled keys through shared memory in blocks of 64 (cp.async,
// double-buffered): scores on the tensor cores (mma.sync m16n8k16 bf16, fp32 accumulate), online
// softmax in fp32 with warp shuffles for the row maximum, and next to the total mass the masked
// masses: the part of the row kept by the Temporal, the Spatial and (when recalls are wanted) the
// Textural mask restricted to I.  A key block that lies wholly inside or outside a mask's band for
// all 16 rows of a warp is settled per block (frames grow monotonically with the sample index, and
// on the first-frame sample so do positions); only blocks a band edge crosses test per element.
// The n x n score matrix is never written.  Per-row recalls go to scratch; a second kernel
// averages them in a fixed order (deterministic) and takes Algorithm 1's decision.
#include "rf_common.cuh"

namespace {

constexpr int ARM_ROWS = 128;  // query rows per CTA (16 per warp)
constexpr int ARM_KEYS = 64;   // keys per shared-memory block
constexpr int ARM_THREADS = 256;

// Which masked masses a launch accumulates.
constexpr int ARM_LOCAL_T = 0;    // first-frame sample: Temporal only (positions = sample index)
constexpr int ARM_GLOBAL_S = 1;   // stride sample: Spatial
constexpr int ARM_GLOBAL_ST = 2;  // stride sample: Spatial and Temporal

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// 16-byte asynchronous copy; zero-fills when !valid (src must still be a readable address).
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid) {
  const int sz = valid ? 16 : 0;
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(sz) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

struct KeyAttr { int f, p, c; };  // frame, in-frame position, 1 if in the checkerboard set C

__device__ __forceinline__ KeyAttr token_attr(const RfGeom& g, int tok) {
  KeyAttr a;
  a.f = tok / g.S;
  a.p = tok - a.f * g.S;
  const int y = a.p / g.Wf, x = a.p - y * g.Wf;
  a.c = (y % g.tau) == (x % g.tau);
  return a;
}

// 0: no pair of (rows, cols) within w, 2: every pair within w, 1: mixed.  Closed integer ranges.
__device__ __forceinline__ int band_class(int ra, int rb, int ca, int cb, int w) {
  const int dmin = max(max(ca - rb, ra - cb), 0), dmax = max(rb - ca, cb - ra);
  return dmax <= w ? 2 : (dmin > w ? 0 : 1);
}

// grid = (ceil(n/128), B*H).  stride: token index of sample m is m*stride.
// row_out: [B*H][3][n_pad] per-row recalls (temporal, spatial, textural) of this sample; only the
// masses this launch accumulates are written.
template <int D, int MODE, bool TEX>
__global__ void __launch_bounds__(ARM_THREADS) rf_arm_rows_kernel(RfGeom g, int n, int stride, int n_pad,
                                                                   const __nv_bfloat16* __restrict__ q,
                                                                   const __nv_bfloat16* __restrict__ k,
                                                                   float scale_log2, float* __restrict__ row_out) {
  constexpr int LD = D + 8;  // padded row, keeps ldmatrix conflict-free
  constexpr int VEC = D / 8;
  constexpr bool WANT_T = MODE != ARM_GLOBAL_S, WANT_S = MODE != ARM_LOCAL_T;
  constexpr bool T_BAND = MODE == ARM_LOCAL_T;  // Temporal mask is a band in sample-index space
  // the Q tile first; once its fragments are in registers the same memory holds two key blocks
  __shared__ __align__(16) __nv_bfloat16 buf[ARM_ROWS * LD];
  __shared__ int kf[2][ARM_KEYS], kp[2][ARM_KEYS], kc[2][ARM_KEYS];

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int bh = blockIdx.y;
  const int row0 = blockIdx.x * ARM_ROWS;
  const size_t head = (size_t)bh * g.N * D;

  for (int i = tid; i < ARM_ROWS * VEC; i += ARM_THREADS) {
    const int r = i / VEC, c = i % VEC;
    const int m = min(row0 + r, n - 1);
    cp_async16(smem_u32(&buf[r * LD + c * 8]), q + head + (size_t)m * stride * D + c * 8, true);
  }
  cp_async_commit();
  cp_async_wait<0>();
  __syncthreads();

  uint32_t qa[D / 16][4];
#pragma unroll
  for (int ks = 0; ks < D / 16; ++ks) {
    const uint32_t addr = smem_u32(&buf[(warp * 16 + (lane & 15)) * LD + ks * 16 + (lane >> 4) * 8]);
    ldmatrix_x4(addr, qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3]);
  }
  __syncthreads();  // every warp has its fragments: the buffer may be overwritten with keys

  auto load_keys = [&](int blk) {
    const int k0 = blk * ARM_KEYS, b = blk & 1;
    for (int i = tid; i < ARM_KEYS * VEC; i += ARM_THREADS) {
      const int r = i / VEC, c = i % VEC;
      const int m = k0 + r;
      cp_async16(smem_u32(&buf[(b * ARM_KEYS + r) * LD + c * 8]), k + head + (size_t)min(m, n - 1) * stride * D + c * 8, m < n);
    }
    if (tid < ARM_KEYS) {
      const KeyAttr a = token_attr(g, min(k0 + tid, n - 1) * stride);
      kf[b][tid] = a.f; kp[b][tid] = a.p; kc[b][tid] = a.c;
    }
    cp_async_commit();
  };

  // the two rows this thread sees: warp*16 + lane/4 and +8
  int rf[2], rp[2];
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const KeyAttr a = token_attr(g, min(row0 + warp * 16 + (lane >> 2) + h * 8, n - 1) * stride);
    rf[h] = a.f;
    rp[h] = a.p;
  }
  // row range of this warp, for the per-block band classification
  const int wra = min(row0 + warp * 16, n - 1), wrb = min(row0 + warp * 16 + 15, n - 1);
  const int wfa = (wra * stride) / g.S, wfb = (wrb * stride) / g.S;

  float mx[2] = {-INFINITY, -INFINITY};
  float l_all[2] = {0.f, 0.f}, l_t[2] = {0.f, 0.f}, l_s[2] = {0.f, 0.f}, l_c[2] = {0.f, 0.f};

  const int nblk = rf_cdiv(n, ARM_KEYS);
  load_keys(0);
  for (int blk = 0; blk < nblk; ++blk) {
    const int k0 = blk * ARM_KEYS, b = blk & 1;
    if (blk + 1 < nblk) {
      load_keys(blk + 1);
      cp_async_wait<1>();
    } else {
      cp_async_wait<0>();
    }
    __syncthreads();
    const __nv_bfloat16* Ks = buf + b * ARM_KEYS * LD;

    float acc[ARM_KEYS / 8][4];
#pragma unroll
    for (int nt = 0; nt < ARM_KEYS / 8; ++nt) { acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f; }
#pragma unroll
    for (int ks = 0; ks < D / 16; ++ks) {
#pragma unroll
      for (int np = 0; np < ARM_KEYS / 16; ++np) {
        const int mi = lane >> 3;
        const uint32_t addr = smem_u32(&Ks[(np * 16 + (mi >> 1) * 8 + (lane & 7)) * LD + ks * 16 + (mi & 1) * 8]);
        uint32_t b0, b1, b2, b3;
        ldmatrix_x4(addr, b0, b1, b2, b3);
        mma_bf16_16816(acc[np * 2], qa[ks], b0, b1);
        mma_bf16_16816(acc[np * 2 + 1], qa[ks], b2, b3);
      }
    }

    // key slots past the sample (last block only) carry -inf
    if (k0 + ARM_KEYS > n) {
#pragma unroll
      for (int nt = 0; nt < ARM_KEYS / 8; ++nt)
#pragma unroll
        for (int e = 0; e < 4; ++e)
          if (k0 + nt * 8 + (lane & 3) * 2 + (e & 1) >= n) acc[nt][e] = -INFINITY;
    }
    float bm[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int nt = 0; nt < ARM_KEYS / 8; ++nt) {
      bm[0] = fmaxf(bm[0], fmaxf(acc[nt][0], acc[nt][1]));
      bm[1] = fmaxf(bm[1], fmaxf(acc[nt][2], acc[nt][3]));
    }
    float neg_m[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      bm[h] = fmaxf(bm[h], __shfl_xor_sync(0xffffffffu, bm[h], 1));
      bm[h] = fmaxf(bm[h], __shfl_xor_sync(0xffffffffu, bm[h], 2));
      const float m_new = fmaxf(mx[h], bm[h] * scale_log2);   // finite: every block holds >= 1 real key
      const float corr = ex2f(mx[h] - m_new);                  // 0 on the first block
      l_all[h] *= corr; l_t[h] *= corr; l_s[h] *= corr; l_c[h] *= corr;
      mx[h] = m_new;
      neg_m[h] = -m_new;
    }

    // band classes of this block for the warp's 16 rows (warp-uniform)
    const int ca = k0, cb = min(k0 + ARM_KEYS - 1, n - 1);
    const int t_cls = !WANT_T ? 0 : (T_BAND ? band_class(wra, wrb, ca, cb, g.ws) : 1);
    const int s_cls = !WANT_S ? 0 : band_class(wfa, wfb, (ca * stride) / g.S, (cb * stride) / g.S, g.wf);

    float bs[2] = {0.f, 0.f}, bt[2] = {0.f, 0.f}, bsp[2] = {0.f, 0.f}, bc[2] = {0.f, 0.f};
#pragma unroll
    for (int nt = 0; nt < ARM_KEYS / 8; ++nt) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int h = e >> 1;
        const int col = nt * 8 + (lane & 3) * 2 + (e & 1);
        const float p = ex2f(fmaf(acc[nt][e], scale_log2, neg_m[h]));
        bs[h] += p;
        if (WANT_T && t_cls == 1) { if (abs(kp[b][col] - rp[h]) <= g.ws) bt[h] += p; }
        if (WANT_S && s_cls == 1) { if (abs(kf[b][col] - rf[h]) <= g.wf) bsp[h] += p; }
        if (TEX) { if (kc[b][col]) bc[h] += p; }
      }
    }
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      l_all[h] += bs[h];
      if (WANT_T) l_t[h] += t_cls == 2 ? bs[h] : bt[h];
      if (WANT_S) l_s[h] += s_cls == 2 ? bs[h] : bsp[h];
      if (TEX) l_c[h] += bc[h];
    }
    __syncthreads();  // block consumed: its buffer is the target of the next prefetch
  }

  // quad reduction of the partial masses, then one lane per row writes its recalls
#pragma unroll
  for (int h = 0; h < 2; ++h) {
#pragma unroll
    for (int o = 1; o <= 2; o <<= 1) {
      l_all[h] += __shfl_xor_sync(0xffffffffu, l_all[h], o);
      l_t[h] += __shfl_xor_sync(0xffffffffu, l_t[h], o);
      l_s[h] += __shfl_xor_sync(0xffffffffu, l_s[h], o);
      l_c[h] += __shfl_xor_sync(0xffffffffu, l_c[h], o);
    }
    const int m = row0 + warp * 16 + (lane >> 2) + h * 8;
    if ((lane & 3) == 0 && m < n) {
      float* out = row_out + (size_t)bh * 3 * n_pad;
      const float inv = 1.f / l_all[h];
      if (WANT_T) out[m] = l_t[h] * inv;
      if (WANT_S) out[n_pad + m] = l_s[h] * inv;
      if (TEX) out[2 * n_pad + m] = l_c[h] * inv;
    }
  }
}

// One CTA per head: mean of the per-row recalls in a fixed order, then Algorithm 1.
__global__ void __launch_bounds__(256) rf_arm_decide_kernel(int n_loc, int n_glb, int n_pad, int sample_mode, float alpha,
                                                             const float* __restrict__ rows_loc,
                                                             const float* __restrict__ rows_glb,
                                                             int32_t* __restrict__ head_class, float* __restrict__ recall) {
  __shared__ double red[3][256];
  const int bh = blockIdx.x, tid = threadIdx.x;
  const float* gl = rows_glb + (size_t)bh * 3 * n_pad;
  const float* lo = rows_loc + (size_t)bh * 3 * n_pad;
  const bool local_t = sample_mode == RF_SAMPLE_ALG1;
  const float* src[3] = {local_t ? lo : gl, gl + n_pad, gl + 2 * n_pad};
  const int cnt[3] = {local_t ? n_loc : n_glb, n_glb, n_glb};
  const int nw = recall != nullptr ? 3 : 2;   // the Textural recall is only accumulated when recalls are wanted
  for (int w = 0; w < 3; ++w) {
    double s = 0.0;
    if (w < nw)
      for (int i = tid; i < cnt[w]; i += 256) s += (double)src[w][i];
    red[w][tid] = s;
  }
  __syncthreads();
  for (int o = 128; o > 0; o >>= 1) {
    if (tid < o)
      for (int w = 0; w < 3; ++w) red[w][tid] += red[w][tid + o];
    __syncthreads();
  }
  if (tid == 0) {
    const float Rt = (float)(red[0][0] / cnt[0]), Rs = (float)(red[1][0] / cnt[1]), Rc = (float)(red[2][0] / cnt[2]);
    if (recall) { recall[bh * 3] = Rt; recall[bh * 3 + 1] = Rs; recall[bh * 3 + 2] = Rc; }
    head_class[bh] = Rt >= alpha ? RF_TEMPORAL : (Rs >= alpha ? RF_SPATIAL : RF_TEXTURAL);
  }
}

template <int D, int MODE, bool TEX>
cudaError_t launch_rows(const RfGeom& g, int n, int stride, int n_pad, const __nv_bfloat16* q, const __nv_bfloat16* k,
                        float* out, cudaStream_t st) {
  dim3 grid(rf_cdiv(n, ARM_ROWS), g.B * g.H);
  const float scale_log2 = 1.4426950408889634f / sqrtf((float)D);
  rf_arm_rows_kernel<D, MODE, TEX><<<grid, ARM_THREADS, 0, st>>>(g, n, stride, n_pad, q, k, scale_log2, out);
  return cudaGetLastError();
}

template <int D>
cudaError_t launch_rows_m(int mode, bool tex, const RfGeom& g, int n, int stride, int n_pad, const __nv_bfloat16* q,
                          const __nv_bfloat16* k, float* out, cudaStream_t st) {
  if (mode == ARM_LOCAL_T) return launch_rows<D, ARM_LOCAL_T, false>(g, n, stride, n_pad, q, k, out, st);
  if (mode == ARM_GLOBAL_S)
    return tex ? launch_rows<D, ARM_GLOBAL_S, true>(g, n, stride, n_pad, q, k, out, st)
               : launch_rows<D, ARM_GLOBAL_S, false>(g, n, stride, n_pad, q, k, out, st);
  return tex ? launch_rows<D, ARM_GLOBAL_ST, true>(g, n, stride, n_pad, q, k, out, st)
             : launch_rows<D, ARM_GLOBAL_ST, false>(g, n, stride, n_pad, q, k, out, st);
}

cudaError_t launch_rows_d(int mode, bool tex, const RfGeom& g, int n, int stride, int n_pad, const __nv_bfloat16* q,
                          const __nv_bfloat16* k, float* out, cudaStream_t st) {
  switch (g.D) {
    case 64: return launch_rows_m<64>(mode, tex, g, n, stride, n_pad, q, k, out, st);
    case 96: return launch_rows_m<96>(mode, tex, g, n, stride, n_pad, q, k, out, st);
    case 128: return launch_rows_m<128>(mode, tex, g, n, stride, n_pad, q, k, out, st);
  }
  return cudaErrorInvalidValue;
}

int arm_n_pad(const RfGeom& g, int omega) {
  const int n_glb = rf_cdiv(g.Nv, omega);
  const int n = n_glb > g.S ? n_glb : g.S;
  return (n + 63) / 64 * 64;
}

}  // namespace

size_t rf_arm_scratch_floats(const RfGeom& g, int omega) { return (size_t)2 * g.B * g.H * 3 * arm_n_pad(g, omega); }

cudaError_t rf_launch_arm(const RfGeom& g, int sample_mode, int omega, float alpha, const __nv_bfloat16* q,
                          const __nv_bfloat16* k, int32_t* head_class, float* recall, float* row_scratch,
                          cudaStream_t st) {
  const int n_pad = arm_n_pad(g, omega);
  const int n_glb = rf_cdiv(g.Nv, omega), n_loc = g.S;
  float* rows_glb = row_scratch;
  float* rows_loc = row_scratch + (size_t)g.B * g.H * 3 * n_pad;
  const bool alg1 = sample_mode == RF_SAMPLE_ALG1;
  const bool tex = recall != nullptr;   // the Textural recall is a diagnostic: Algorithm 1 does not use it
  cudaError_t e = launch_rows_d(alg1 ? ARM_GLOBAL_S : ARM_GLOBAL_ST, tex, g, n_glb, omega, n_pad, q, k, rows_glb, st);
  if (e != cudaSuccess) return e;
  if (alg1) {
    e = launch_rows_d(ARM_LOCAL_T, false, g, n_loc, 1, n_pad, q, k, rows_loc, st);
    if (e != cudaSuccess) return e;
  }
  rf_arm_decide_kernel<<<g.B * g.H, 256, 0, st>>>(n_loc, n_glb, n_pad, sample_mode, alpha, rows_loc, rows_glb,
                                                  head_class, recall);
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
                                             const void* k, int32_t* head_class, float* recall, void* cuda_stream) {
  RfGeom g;
  rf_status st = rf_checked_geom(shape, params, &g);
  if (st != RF_OK) return st;
  if (g.D != 64 && g.D != 96 && g.D != 128) return RF_ERR_UNSUPPORTED;
  if (q == nullptr || k == nullptr || head_class == nullptr) return RF_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(q) & 15u) != 0 || (reinterpret_cast<uintptr_t>(k) & 15u) != 0) return RF_ERR_INVALID_ARG;
  if (rf_arm_scratch_floats(g, params->sample_stride) > (size_t)RF_ARM_STATIC_SCRATCH_FLOATS)
    return RF_ERR_STATIC_SCRATCH_TOO_SMALL;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return RF_ERR_CUDA;
  cudaError_t e;
  float* scratch = static_scratch_ptr(dev, &e);
  if (scratch == nullptr) return RF_ERR_CUDA;
  e = rf_launch_arm(g, params->sample_mode, params->sample_stride, params->alpha, static_cast<const __nv_bfloat16*>(q),
                    static_cast<const __nv_bfloat16*>(k), head_class, recall, scratch, static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? RF_OK : RF_ERR_CUDA;
}
