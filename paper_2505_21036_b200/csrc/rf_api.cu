// C ABI of the RainFusion CUDA path: argument validation, workspace layout, tensor-map encoding.
#include <math.h>
#include <string.h>

#include "rf_common.cuh"

namespace {

constexpr size_t kAlign = 256;
inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline bool pow2(int x) { return x > 0 && (x & (x - 1)) == 0; }

// The kernels pack a frame row and column into one word for the 2-D Temporal window.
rf_status check_2d(const rf_shape* s, const rf_params* p) {
  if (p->temporal_window_2d == 1 && (s->frame_h >= 32768 || s->frame_w >= 32768)) return RF_ERR_UNSUPPORTED;
  return RF_OK;
}

rf_status check_shape(const rf_shape* s) {
  if (s == nullptr) return RF_ERR_INVALID_ARG;
  if (s->B < 1 || s->H < 1 || s->T < 1 || s->frame_h < 1 || s->frame_w < 1 || s->L_text < 0) return RF_ERR_INVALID_ARG;
  if (s->D < 8 || s->D % 8 != 0) return RF_ERR_INVALID_ARG;
  const long long n = (long long)s->T * s->frame_h * s->frame_w + s->L_text;
  if (n > (1ll << 30) || (long long)s->B * s->H > 65535) return RF_ERR_UNSUPPORTED;
  return RF_OK;
}

rf_status check_params(const rf_params* p) {
  if (p == nullptr) return RF_ERR_INVALID_ARG;
  if (p->frame_window < 0 || p->spatial_window < 0 || p->textural_stride < 1 || p->sample_stride < 1)
    return RF_ERR_INVALID_ARG;
  if (p->sample_mode != RF_SAMPLE_ALG1 && p->sample_mode != RF_SAMPLE_GLOBAL) return RF_ERR_INVALID_ARG;
  if (!(p->alpha > 0.f && p->alpha <= 1.f)) return RF_ERR_INVALID_ARG;
  if (!pow2(p->block_m) || !pow2(p->block_n) || p->block_m < 16 || p->block_n < 16) return RF_ERR_INVALID_ARG;
  if (p->temporal_permute != 0 && p->temporal_permute != 1) return RF_ERR_INVALID_ARG;
  if (p->two_mask != 0 && p->two_mask != 1) return RF_ERR_INVALID_ARG;
  if (p->spatial_key_first_frame != 0 && p->spatial_key_first_frame != 1) return RF_ERR_INVALID_ARG;
  if (p->temporal_window_2d != 0 && p->temporal_window_2d != 1) return RF_ERR_INVALID_ARG;
  if (p->temporal_window_2d == 1 && (p->temporal_window_y < 0 || p->temporal_window_x < 0)) return RF_ERR_INVALID_ARG;
  return RF_OK;
}

// Kept tokens per frame of the checkerboard set C (Eq. 4).
int checkerboard_count(int Hf, int Wf, int tau) {
  int n = 0;
  for (int r = 0; r < tau; ++r) {
    const int rows = r < Hf ? (Hf - r + tau - 1) / tau : 0;
    const int cols = r < Wf ? (Wf - r + tau - 1) / tau : 0;
    n += rows * cols;
  }
  return n;
}

RfGeom make_geom(const rf_shape* s, int wf, int ws, int tau, int bm, int bn, int permute) {
  RfGeom g;
  g.B = s->B; g.H = s->H; g.D = s->D;
  g.T = s->T; g.Hf = s->frame_h; g.Wf = s->frame_w; g.S = s->frame_h * s->frame_w;
  g.Nv = g.T * g.S; g.L = s->L_text; g.N = g.Nv + g.L;
  // Windows past the extent and strides past the frame's longer side give the same masks as the extent itself
  // (every frame / position within reach; y mod tau = y and x mod tau = x); clamping keeps the kernels' index
  // arithmetic ((f + w_f + 1) * S, p + w_s, loops over tau) inside int range for any caller value.
  g.wf = wf < g.T ? wf : g.T;
  g.ws = ws < g.S ? ws : g.S;
  g.tau = tau < (g.Hf > g.Wf ? g.Hf : g.Wf) ? tau : (g.Hf > g.Wf ? g.Hf : g.Wf);
  tau = g.tau;
  g.nC = checkerboard_count(g.Hf, g.Wf, tau);
  g.LkvTex = g.T * g.nC + g.L;
  g.BM = bm; g.BN = bn;
  g.nQ = rf_cdiv(g.N, bm);
  g.nKmax = rf_cdiv(g.N, bn);
  g.permute = permute;
  g.two_mask = 0;
  g.key_first = 0;
  g.t2d = g.wy = g.wx = 0;
  return g;
}
RfGeom make_geom(const rf_shape* s, const rf_params* p) {
  RfGeom g = make_geom(s, p->frame_window, p->spatial_window, p->textural_stride, p->block_m, p->block_n, p->temporal_permute);
  g.two_mask = p->two_mask;
  g.key_first = p->spatial_key_first_frame;
  g.t2d = p->temporal_window_2d;
  g.wy = g.t2d ? (p->temporal_window_y < g.Hf ? p->temporal_window_y : g.Hf) : 0;   // past the frame: same mask
  g.wx = g.t2d ? (p->temporal_window_x < g.Wf ? p->temporal_window_x : g.Wf) : 0;
  return g;
}

size_t tensor_bytes(const RfGeom& g) { return align_up((size_t)g.B * g.H * g.N * g.D * sizeof(__nv_bfloat16)); }

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn == nullptr) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess)
      return nullptr;
    fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// bf16 [heads][rows (stride head_rows)][D] viewed as a 3-D tensor, box = 64 columns x 128 rows, 128B swizzle.
bool encode_map(CUtensorMap* m, const void* ptr, int D, int rows, int head_rows, int heads) {
  return rf_encode_rows_map(m, ptr, D, rows, (size_t)D * 2, (size_t)head_rows * D * 2, heads);
}

rf_status check_attn_shape(const rf_shape* s) {
  rf_status st = check_shape(s);
  if (st != RF_OK) return st;
  if (s->D != 64 && s->D != 96 && s->D != 128) return RF_ERR_UNSUPPORTED;
  return RF_OK;
}

}  // namespace

bool rf_encode_rows_map(CUtensorMap* m, const void* ptr, int D, int rows, size_t row_stride_bytes,
                        size_t head_stride_bytes, int heads) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return false;
  cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)rows, (cuuint64_t)heads};
  cuuint64_t strides[2] = {(cuuint64_t)row_stride_bytes, (cuuint64_t)head_stride_bytes};
  cuuint32_t box[3] = {64, 128, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

rf_status rf_checked_geom(const rf_shape* shape, const rf_params* params, RfGeom* out) {
  rf_status st = check_shape(shape);
  if (st != RF_OK) return st;
  st = check_params(params);
  if (st != RF_OK) return st;
  st = check_2d(shape, params);
  if (st != RF_OK) return st;
  *out = make_geom(shape, params);
  return RF_OK;
}

namespace {
// Shared by rf_sparse_attn_fwd(_plus) and rf_sparse_attn_reordered: the second skips the gather pass and
// reads the reordered copies a preceding rf_reorder_tokens call left in the workspace.
rf_status sparse_attn_impl(const rf_shape* shape, const rf_params* params, const void* q, const void* k, const void* v,
                           const int32_t* head_class, const int32_t* head_window, const rf_schedule* sched, void* o,
                           float* lse, void* ws, size_t ws_bytes, int32_t* dev_status, void* cuda_stream, bool gather) {
  rf_status st = check_attn_shape(shape);
  if (st != RF_OK) return st;
  st = check_params(params);
  if (st != RF_OK) return st;
  st = check_2d(shape, params);
  if (st != RF_OK) return st;
  if (params->block_m != 128 || params->block_n != 128) return RF_ERR_UNSUPPORTED;
  if (q == nullptr || k == nullptr || v == nullptr || o == nullptr || head_class == nullptr || sched == nullptr ||
      sched->count == nullptr || sched->kv_tile == nullptr || ws == nullptr)
    return RF_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o) ||
      (reinterpret_cast<uintptr_t>(ws) & (kAlign - 1)) != 0)
    return RF_ERR_INVALID_ARG;
  if (head_window != nullptr && params->temporal_window_2d) return RF_ERR_UNSUPPORTED;
  if (ws_bytes < rf_workspace_bytes(shape, params)) return RF_ERR_WORKSPACE_TOO_SMALL;
  const RfGeom g = make_geom(shape, params);
  if (sched->nQ != g.nQ || sched->nKmax != g.nKmax) return RF_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);

  uint8_t* w = static_cast<uint8_t*>(ws);
  __nv_bfloat16* wq = reinterpret_cast<__nv_bfloat16*>(w);
  __nv_bfloat16* wk = reinterpret_cast<__nv_bfloat16*>(w + tensor_bytes(g));
  __nv_bfloat16* wv = reinterpret_cast<__nv_bfloat16*>(w + 2 * tensor_bytes(g));

  CUtensorMap maps[RF_ATTN_MAPS];
  const int heads = g.B * g.H;
  bool ok = encode_map(&maps[0], q, g.D, g.N, g.N, heads) && encode_map(&maps[1], k, g.D, g.N, g.N, heads) &&
            encode_map(&maps[2], v, g.D, g.N, g.N, heads) && encode_map(&maps[3], wq, g.D, g.N, g.N, heads) &&
            encode_map(&maps[4], wk, g.D, g.N, g.N, heads) && encode_map(&maps[5], wv, g.D, g.N, g.N, heads) &&
            encode_map(&maps[6], wk, g.D, g.LkvTex, g.N, heads) && encode_map(&maps[7], wv, g.D, g.LkvTex, g.N, heads);
  if (!ok) return RF_ERR_CUDA;

  if (gather) {
    cudaError_t e = rf_launch_gather(g, head_class, static_cast<const __nv_bfloat16*>(q),
                                     static_cast<const __nv_bfloat16*>(k), static_cast<const __nv_bfloat16*>(v), wq, wk, wv,
                                     dev_status, stream);
    if (e != cudaSuccess) return RF_ERR_CUDA;
  }

  RfAttnArgs a;
  a.g = g;
  a.head_class = head_class;
  a.head_window = head_window;
  a.count = sched->count;
  a.kv_tile = sched->kv_tile;
  a.o = static_cast<__nv_bfloat16*>(o);
  a.lse = lse;
  a.dev_status = dev_status;
  a.scale_log2 = 1.4426950408889634f / sqrtf((float)g.D);
  return rf_launch_attention(a, maps, stream);
}
}  // namespace

extern "C" {

int32_t rf_bounds_checked(void) {
#ifdef RF_BOUNDS_CHECK
  return 1;
#else
  return 0;
#endif
}

const char* rf_status_string(rf_status s) {
  switch (s) {
    case RF_OK: return "ok";
    case RF_ERR_INVALID_ARG: return "invalid argument";
    case RF_ERR_UNSUPPORTED: return "unsupported shape or parameter";
    case RF_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case RF_ERR_CUDA: return "CUDA error";
    case RF_ERR_TIMEOUT: return "device-side wait timed out";
    case RF_ERR_STATIC_SCRATCH_TOO_SMALL:
      return "problem needs more scratch than the library's built-in array holds (use the workspace entry point)";
    case RF_ERR_BOUNDS: return "a kernel of the bounds-checking build was about to index outside an array";
  }
  return "unknown status";
}

rf_status rf_schedule_dims(const rf_shape* shape, const rf_params* params, int32_t* nQ, int32_t* nKmax) {
  rf_status st = check_shape(shape);
  if (st != RF_OK) return st;
  st = check_params(params);
  if (st != RF_OK) return st;
  st = check_2d(shape, params);
  if (st != RF_OK) return st;
  const RfGeom g = make_geom(shape, params);
  if (nQ) *nQ = g.nQ;
  if (nKmax) *nKmax = g.nKmax;
  return RF_OK;
}

size_t rf_workspace_bytes(const rf_shape* shape, const rf_params* params) {
  if (check_shape(shape) != RF_OK || check_params(params) != RF_OK) return 0;
  const RfGeom g = make_geom(shape, params);
  return 3 * tensor_bytes(g) + align_up(rf_arm_scratch_floats(g, params->sample_stride, RF_MAX_BANDWIDTHS) * sizeof(float));
}

rf_status rf_arm_classify(const rf_shape* shape, const rf_params* params, const void* q, const void* k,
                          int32_t* head_class, float* recall, void* ws, size_t ws_bytes, int32_t* dev_status,
                          void* cuda_stream) {
  rf_status st = check_shape(shape);
  if (st != RF_OK) return st;
  st = check_params(params);
  if (st != RF_OK) return st;
  st = check_2d(shape, params);
  if (st != RF_OK) return st;
  if (shape->D != 64 && shape->D != 96 && shape->D != 128) return RF_ERR_UNSUPPORTED;
  if (q == nullptr || k == nullptr || head_class == nullptr || ws == nullptr) return RF_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || (reinterpret_cast<uintptr_t>(ws) & (kAlign - 1)) != 0) return RF_ERR_INVALID_ARG;
  if (ws_bytes < rf_workspace_bytes(shape, params)) return RF_ERR_WORKSPACE_TOO_SMALL;
  const RfGeom g = make_geom(shape, params);
  float* scratch = reinterpret_cast<float*>(static_cast<uint8_t*>(ws) + 3 * tensor_bytes(g));
  cudaError_t e = rf_launch_arm(g, params->sample_mode, params->sample_stride, params->alpha, 1, &g.ws, &g.wf,
                                static_cast<const __nv_bfloat16*>(q), static_cast<const __nv_bfloat16*>(k), head_class,
                                nullptr, recall, nullptr, scratch, dev_status, static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? RF_OK : RF_ERR_CUDA;
}

rf_status rf_selftest_arm_abandoned(const rf_shape* shape, const rf_params* params, const void* q, const void* k,
                                    int32_t* head_class, void* ws, size_t ws_bytes, int32_t* dev_status, void* cuda_stream) {
  rf_status st = check_shape(shape);
  if (st != RF_OK) return st;
  st = check_params(params);
  if (st != RF_OK) return st;
  st = check_2d(shape, params);
  if (st != RF_OK) return st;
  if (shape->D != 64 && shape->D != 96 && shape->D != 128) return RF_ERR_UNSUPPORTED;
  if (q == nullptr || k == nullptr || head_class == nullptr || ws == nullptr) return RF_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || (reinterpret_cast<uintptr_t>(ws) & (kAlign - 1)) != 0) return RF_ERR_INVALID_ARG;
  if (ws_bytes < rf_workspace_bytes(shape, params)) return RF_ERR_WORKSPACE_TOO_SMALL;
  const RfGeom g = make_geom(shape, params);
  float* scratch = reinterpret_cast<float*>(static_cast<uint8_t*>(ws) + 3 * tensor_bytes(g));
  cudaError_t e = rf_launch_arm(g, params->sample_mode, params->sample_stride, params->alpha, 1, &g.ws, &g.wf,
                                static_cast<const __nv_bfloat16*>(q), static_cast<const __nv_bfloat16*>(k), head_class,
                                nullptr, nullptr, nullptr, scratch, dev_status, static_cast<cudaStream_t>(cuda_stream), true);
  return e == cudaSuccess ? RF_OK : RF_ERR_CUDA;
}

rf_status rf_arm_classify_plus(const rf_shape* shape, const rf_params* params, const float* bandwidths,
                               int32_t n_bandwidths, const void* q, const void* k, int32_t* head_class,
                               int32_t* head_window, float* recall, void* ws, size_t ws_bytes, int32_t* dev_status,
                               void* cuda_stream) {
  rf_status st = check_shape(shape);
  if (st != RF_OK) return st;
  st = check_params(params);
  if (st != RF_OK) return st;
  st = check_2d(shape, params);
  if (st != RF_OK) return st;
  if (shape->D != 64 && shape->D != 96 && shape->D != 128) return RF_ERR_UNSUPPORTED;
  if (params->temporal_window_2d) return RF_ERR_UNSUPPORTED;   // a bandwidth has no 2-D meaning defined here
  if (bandwidths == nullptr || n_bandwidths < 1 || n_bandwidths > RF_MAX_BANDWIDTHS) return RF_ERR_INVALID_ARG;
  if (q == nullptr || k == nullptr || head_class == nullptr || head_window == nullptr || ws == nullptr) return RF_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || (reinterpret_cast<uintptr_t>(ws) & (kAlign - 1)) != 0) return RF_ERR_INVALID_ARG;
  if (ws_bytes < rf_workspace_bytes(shape, params)) return RF_ERR_WORKSPACE_TOO_SMALL;
  const RfGeom g = make_geom(shape, params);
  int ws_list[RF_MAX_BANDWIDTHS], wf_list[RF_MAX_BANDWIDTHS];
  for (int i = 0; i < n_bandwidths; ++i) {
    const float b = bandwidths[i];
    if (!(b > 0.f && b <= 1.f) || (i > 0 && b <= bandwidths[i - 1])) return RF_ERR_INVALID_ARG;
    wf_list[i] = (int)floor((double)b * g.T);
    ws_list[i] = (int)floor((double)b * g.S);
  }
  float* scratch = reinterpret_cast<float*>(static_cast<uint8_t*>(ws) + 3 * tensor_bytes(g));
  cudaError_t e = rf_launch_arm(g, params->sample_mode, params->sample_stride, params->alpha, n_bandwidths, ws_list,
                                wf_list, static_cast<const __nv_bfloat16*>(q), static_cast<const __nv_bfloat16*>(k),
                                head_class, head_window, nullptr, recall, scratch, dev_status,
                                static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? RF_OK : RF_ERR_CUDA;
}

rf_status rf_build_block_mask(const rf_shape* shape, const rf_params* params, const int32_t* head_class,
                              rf_schedule* out, int32_t* dev_status, void* cuda_stream) {
  return rf_build_block_mask_plus(shape, params, head_class, nullptr, out, dev_status, cuda_stream);
}

rf_status rf_build_block_mask_plus(const rf_shape* shape, const rf_params* params, const int32_t* head_class,
                                   const int32_t* head_window, rf_schedule* out, int32_t* dev_status, void* cuda_stream) {
  rf_status st = check_shape(shape);
  if (st != RF_OK) return st;
  st = check_params(params);
  if (st != RF_OK) return st;
  st = check_2d(shape, params);
  if (st != RF_OK) return st;
  if (head_window != nullptr && params->temporal_window_2d) return RF_ERR_UNSUPPORTED;
  if (head_class == nullptr || out == nullptr || out->count == nullptr || out->kv_tile == nullptr || out->kv_len == nullptr)
    return RF_ERR_INVALID_ARG;
  const RfGeom g = make_geom(shape, params);
  if (out->nQ != g.nQ || out->nKmax != g.nKmax) return RF_ERR_INVALID_ARG;
  cudaError_t e = rf_launch_build_tiles(g, head_class, head_window, out->count, out->kv_tile, out->bitmap, out->kv_len,
                                        dev_status, static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? RF_OK : RF_ERR_CUDA;
}

rf_status rf_sparse_attn_fwd(const rf_shape* shape, const rf_params* params, const void* q, const void* k,
                             const void* v, const int32_t* head_class, const rf_schedule* sched, void* o, float* lse,
                             void* ws, size_t ws_bytes, int32_t* dev_status, void* cuda_stream) {
  return rf_sparse_attn_fwd_plus(shape, params, q, k, v, head_class, nullptr, sched, o, lse, ws, ws_bytes, dev_status,
                                 cuda_stream);
}

rf_status rf_sparse_attn_fwd_plus(const rf_shape* shape, const rf_params* params, const void* q, const void* k,
                                  const void* v, const int32_t* head_class, const int32_t* head_window,
                                  const rf_schedule* sched, void* o, float* lse, void* ws, size_t ws_bytes,
                                  int32_t* dev_status, void* cuda_stream) {
  return sparse_attn_impl(shape, params, q, k, v, head_class, head_window, sched, o, lse, ws, ws_bytes, dev_status,
                          cuda_stream, true);
}

rf_status rf_sparse_attn_reordered(const rf_shape* shape, const rf_params* params, const void* q, const void* k,
                                   const void* v, const int32_t* head_class, const int32_t* head_window,
                                   const rf_schedule* sched, void* o, float* lse, void* ws, size_t ws_bytes,
                                   int32_t* dev_status, void* cuda_stream) {
  return sparse_attn_impl(shape, params, q, k, v, head_class, head_window, sched, o, lse, ws, ws_bytes, dev_status,
                          cuda_stream, false);
}

rf_status rf_selftest_wait_timeout(int32_t* dev_status, int32_t limit_ms, int32_t* waits_returned, void* cuda_stream) {
  if (dev_status == nullptr || waits_returned == nullptr || limit_ms < 1 || limit_ms > 1000) return RF_ERR_INVALID_ARG;
  return rf_launch_selftest_timeout(dev_status, (uint64_t)limit_ms * 1000000ull, waits_returned,
                                    static_cast<cudaStream_t>(cuda_stream));
}

rf_status rf_reorder_tokens(const rf_shape* shape, const rf_params* params, const void* q, const void* k,
                            const void* v, const int32_t* head_class, void* ws, size_t ws_bytes, void* cuda_stream) {
  rf_status st = check_shape(shape);
  if (st != RF_OK) return st;
  st = check_params(params);
  if (st != RF_OK) return st;
  st = check_2d(shape, params);
  if (st != RF_OK) return st;
  if (q == nullptr || k == nullptr || v == nullptr || head_class == nullptr || ws == nullptr) return RF_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || (reinterpret_cast<uintptr_t>(ws) & (kAlign - 1)) != 0)
    return RF_ERR_INVALID_ARG;
  if (ws_bytes < rf_workspace_bytes(shape, params)) return RF_ERR_WORKSPACE_TOO_SMALL;
  const RfGeom g = make_geom(shape, params);
  uint8_t* w = static_cast<uint8_t*>(ws);
  cudaError_t e = rf_launch_gather(g, head_class, static_cast<const __nv_bfloat16*>(q), static_cast<const __nv_bfloat16*>(k),
                                   static_cast<const __nv_bfloat16*>(v), reinterpret_cast<__nv_bfloat16*>(w),
                                   reinterpret_cast<__nv_bfloat16*>(w + tensor_bytes(g)),
                                   reinterpret_cast<__nv_bfloat16*>(w + 2 * tensor_bytes(g)), nullptr,
                                   static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? RF_OK : RF_ERR_CUDA;
}

rf_status rf_dense_attn_fwd(const rf_shape* shape, const void* q, const void* k, const void* v, void* o, float* lse,
                            void* ws, size_t ws_bytes, int32_t* dev_status, void* cuda_stream) {
  (void)ws;
  (void)ws_bytes;
  rf_status st = check_attn_shape(shape);
  if (st != RF_OK) return st;
  if (q == nullptr || k == nullptr || v == nullptr || o == nullptr) return RF_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o)) return RF_ERR_INVALID_ARG;
  const RfGeom g = make_geom(shape, 0, 0, 1, 128, 128, 0);
  CUtensorMap maps[RF_ATTN_MAPS];
  const int heads = g.B * g.H;
  bool ok = encode_map(&maps[0], q, g.D, g.N, g.N, heads) && encode_map(&maps[1], k, g.D, g.N, g.N, heads) &&
            encode_map(&maps[2], v, g.D, g.N, g.N, heads);
  if (!ok) return RF_ERR_CUDA;
  for (int i = 3; i < 8; ++i) maps[i] = maps[i % 3];
  RfAttnArgs a;
  a.g = g;
  a.head_class = nullptr;
  a.head_window = nullptr;
  a.count = nullptr;
  a.kv_tile = nullptr;
  a.o = static_cast<__nv_bfloat16*>(o);
  a.lse = lse;
  a.dev_status = dev_status;
  a.scale_log2 = 1.4426950408889634f / sqrtf((float)g.D);
  return rf_launch_attention(a, maps, static_cast<cudaStream_t>(cuda_stream));
}

}  // extern "C"
