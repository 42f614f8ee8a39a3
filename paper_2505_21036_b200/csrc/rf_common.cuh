// Shared host/device definitions of the RainFusion CUDA path (sm_100a only).
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/rainfusion.h"

#define RF_PARTIAL_BIT 0x80000000u

// Geometry and pattern parameters as the kernels see them (passed by value).
struct RfGeom {
  int B, H, D;
  int T, Hf, Wf, S;      // frames, frame height/width, tokens per frame
  int Nv, L, N;          // video tokens, text tokens, all tokens
  int wf, ws, tau;       // frame window, spatial window, checkerboard stride
  int nC;                // kept tokens per frame for the Textural pattern
  int LkvTex;            // key slots of a Textural head: T*nC + L
  int BM, BN, nQ, nKmax; // block mask tile and its extents
  int permute;           // Temporal heads in position-major order
  int two_mask;          // ARM decides between Spatial and Temporal only (ablation of Sec. 4.4)
  int key_first;         // Spatial heads also keep every key of frame 0 (a key frame, Sec. 3.2)
  int t2d, wy, wx;       // Temporal heads keep the 2-D in-frame window |dy| <= wy, |dx| <= wx instead of the band ws
};

// Device-side error reporting: first error wins, kernels never trap.
__device__ __forceinline__ void rf_report(int32_t* dev_status, int code) {
  if (dev_status != nullptr) atomicCAS(dev_status, 0, code);
}

// Index check of the bounds-checking build: true when idx < limit; otherwise RF_ERR_BOUNDS is reported and the
// caller skips the access.  Compiles to `true` in the normal build.
#ifdef RF_BOUNDS_CHECK
__device__ __forceinline__ bool rf_in_bounds(unsigned long long idx, unsigned long long limit, int32_t* dev_status) {
  if (idx < limit) return true;
  rf_report(dev_status, RF_ERR_BOUNDS);
  return false;
}
#else
__device__ __forceinline__ bool rf_in_bounds(unsigned long long, unsigned long long, int32_t*) { return true; }
#endif

__host__ __device__ __forceinline__ int rf_cdiv(int a, int b) { return (a + b - 1) / b; }

// Number of key slots of a head of class `cls`.
__host__ __device__ __forceinline__ int rf_kv_len(const RfGeom& g, int cls) {
  return cls == RF_TEXTURAL ? g.LkvTex : g.N;
}

// Launchers implemented in the .cu files (host).
// head_window (nullable): per-head window replacing g.wf (Spatial heads) / g.ws (Temporal heads)
cudaError_t rf_launch_build_tiles(const RfGeom& g, const int32_t* head_class, const int32_t* head_window, int32_t* count,
                                  int32_t* kv_tile, uint32_t* bitmap, int32_t* kv_len, int32_t* dev_status, cudaStream_t st);
cudaError_t rf_launch_gather(const RfGeom& g, const int32_t* head_class, const __nv_bfloat16* q,
                             const __nv_bfloat16* k, const __nv_bfloat16* v, __nv_bfloat16* wq, __nv_bfloat16* wk,
                             __nv_bfloat16* wv, int32_t* dev_status, cudaStream_t st);
// nb candidate windows per pattern (ws_list for Temporal, wf_list for Spatial, ascending).  head_window == nullptr:
// plain Algorithm 1 on the first candidate (recall: [B,H,3] or null).  Otherwise dynamic bandwidth: head_window
// receives each head's chosen window, recall_plus ([B,H,2,nb] or null) the candidates' recalls.
// dev_status (nullable) receives RF_ERR_TIMEOUT if a wait inside the score kernel ran out; head_class is then -1.
// selftest_abandon: the score kernel is not launched; its failure flag is set instead, as if a wait had run out.
cudaError_t rf_launch_arm(const RfGeom& g, int sample_mode, int omega, float alpha, int nb, const int* ws_list,
                          const int* wf_list, const __nv_bfloat16* q, const __nv_bfloat16* k, int32_t* head_class,
                          int32_t* head_window, float* recall, float* recall_plus, float* row_scratch, int32_t* dev_status,
                          cudaStream_t st, bool selftest_abandon = false);
// Floats of ARM scratch: the per-row recalls plus RF_ARM_FLAG_FLOATS at the end whose first word records a
// wait that ran out inside the score kernel (cleared by every call before its kernels run).
#define RF_ARM_FLAG_FLOATS 64
size_t rf_arm_scratch_floats(const RfGeom& g, int omega, int nb);
// Tensor map over bf16 rows: [heads][rows][D] with the given row and head strides in bytes (multiples of 16),
// box = 64 columns x 128 rows, 128-byte swizzle, zero fill past `rows`.
bool rf_encode_rows_map(CUtensorMap* m, const void* ptr, int D, int rows, size_t row_stride_bytes,
                        size_t head_stride_bytes, int heads);
// Validates shape and parameters as the entry points do and fills the kernel-side geometry.
rf_status rf_checked_geom(const rf_shape* shape, const rf_params* params, RfGeom* out);

struct RfAttnArgs {
  RfGeom g;
  const int32_t* head_class;  // nullptr: every head Dense, implicit full tile list
  const int32_t* head_window; // nullable: per-head window replacing g.wf (Spatial) / g.ws (Temporal)
  const int32_t* count;
  const int32_t* kv_tile;
  __nv_bfloat16* o;
  float* lse;
  int32_t* dev_status;
  float scale_log2;           // log2(e) / sqrt(D)
};
// Tensor maps: [0..2] Q/K/V in original order, [3..5] the workspace copies with N rows per head
// (position-major Q/K/V of Temporal heads), [6..7] workspace K/V with LkvTex rows per head (Textural).
constexpr int RF_ATTN_MAPS = 8;
rf_status rf_launch_attention(const RfAttnArgs& a, const CUtensorMap* maps, cudaStream_t st);
rf_status rf_launch_selftest_timeout(int32_t* dev_status, uint64_t limit_ns, int32_t* waits_returned, cudaStream_t st);
