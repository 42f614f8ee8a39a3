// The whole path for callers whose Q, K, V and O live in host memory, behind the C ABI.
//
// Heads are independent at every stage (Algorithm 1 classifies per head; the masks of Sec. 3.2 and the attention of
// Eq. 1-2 are per head), so a call is pipelined over groups of heads on three streams: while one group's
// ARM -> tile schedule -> masked attention runs, the next group's inputs arrive from the host and the previous
// group's output leaves.  Every byte of Q, K, V still crosses to the device and every byte of O comes back in every
// call; only the waiting overlaps.  Calls made back to back overlap as well: a group's staging buffers are refilled
// for the next call as soon as this call's kernels have read them.  Consecutive groups compute on two alternating
// streams, each with a workspace and schedule arrays of its own: the last CTAs of one group's attention kernel
// (a CTA runs for about a millisecond at the large shapes) then leave their SMs to the next group's kernels instead
// of to nobody.
// The pipeline object holds streams and events only; device memory comes from the caller in one block.
#include <new>
#include <vector>

#include "rf_common.cuh"

struct rf_host_pipeline {
  rf_shape shape, gshape;       // whole call / one group of heads
  rf_params params;
  int groups, heads_per_group;
  size_t head_elems;            // N * D
  __nv_bfloat16 *q, *k, *v, *o; // staging, [B*H, N, D]
  int lanes;                    // compute streams in use: 2, or 1 when there is a single group
  uint8_t* ws[2];               // workspace of one group, per compute stream
  size_t ws_bytes;
  rf_schedule sched[2];         // schedule arrays of one group, per compute stream
  int32_t* head_class;          // [groups, heads_per_group]
  int32_t* head_window;         // the same, written when candidate bandwidths are set (dynamic bandwidth, Sec. 4.3)
  int n_bw;                     // number of candidate bandwidths, 0: the fixed windows of params
  float bw[RF_MAX_BANDWIDTHS];
  int32_t* status;
  cudaStream_t s_in, s_run[2], s_out;
  std::vector<cudaEvent_t> landed, run_done, out_done;
  cudaEvent_t all_done;
  bool ran;
};

namespace {

constexpr size_t kAlign = 256;
inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

struct Layout {
  size_t tensor, ws, count, kv_tile, kv_len, head_class, status, total;
};

bool layout_of(const rf_shape* shape, const rf_params* params, int groups, rf_shape* gshape, Layout* L, int32_t* nQ, int32_t* nK) {
  if (shape == nullptr || params == nullptr || groups < 1) return false;
  const long long heads = (long long)shape->B * shape->H;
  if (heads < 1 || heads % groups != 0) return false;
  *gshape = *shape;
  gshape->B = 1;
  gshape->H = (int32_t)(heads / groups);
  if (rf_schedule_dims(gshape, params, nQ, nK) != RF_OK) return false;
  const size_t ws = rf_workspace_bytes(gshape, params);
  if (ws == 0) return false;
  const size_t N = (size_t)shape->T * shape->frame_h * shape->frame_w + shape->L_text;
  L->tensor = align_up((size_t)heads * N * shape->D * sizeof(__nv_bfloat16));
  L->ws = align_up(ws);
  L->count = align_up((size_t)gshape->H * *nQ * sizeof(int32_t));
  L->kv_tile = align_up((size_t)gshape->H * *nQ * *nK * sizeof(int32_t));
  L->kv_len = align_up((size_t)gshape->H * sizeof(int32_t));
  L->head_class = align_up((size_t)heads * sizeof(int32_t));
  L->status = kAlign;
  const size_t lanes = groups > 1 ? 2 : 1;
  L->total = 4 * L->tensor + lanes * (L->ws + L->count + L->kv_tile + L->kv_len) + 2 * L->head_class + L->status;
  return true;
}

void destroy(rf_host_pipeline* p) {
  if (p == nullptr) return;
  for (auto* vec : {&p->landed, &p->run_done, &p->out_done})
    for (cudaEvent_t e : *vec)
      if (e) cudaEventDestroy(e);
  if (p->all_done) cudaEventDestroy(p->all_done);
  if (p->s_in) cudaStreamDestroy(p->s_in);
  for (cudaStream_t st : p->s_run)
    if (st) cudaStreamDestroy(st);
  if (p->s_out) cudaStreamDestroy(p->s_out);
  delete p;
}

}  // namespace

extern "C" {

size_t rf_host_pipeline_staging_bytes(const rf_shape* shape, const rf_params* params, int32_t head_groups) {
  rf_shape gs;
  Layout L;
  int32_t nQ, nK;
  return layout_of(shape, params, head_groups, &gs, &L, &nQ, &nK) ? L.total : 0;
}

rf_status rf_host_pipeline_create(const rf_shape* shape, const rf_params* params, int32_t head_groups, void* staging,
                                  size_t staging_bytes, rf_host_pipeline** out) {
  if (out == nullptr) return RF_ERR_INVALID_ARG;
  *out = nullptr;
  rf_shape gs;
  Layout L;
  int32_t nQ, nK;
  if (!layout_of(shape, params, head_groups, &gs, &L, &nQ, &nK)) return RF_ERR_INVALID_ARG;
  if (shape->D != 64 && shape->D != 96 && shape->D != 128) return RF_ERR_UNSUPPORTED;
  if (params->block_m != 128 || params->block_n != 128) return RF_ERR_UNSUPPORTED;
  if (staging == nullptr || (reinterpret_cast<uintptr_t>(staging) & (kAlign - 1)) != 0) return RF_ERR_INVALID_ARG;
  if (staging_bytes < L.total) return RF_ERR_WORKSPACE_TOO_SMALL;
  rf_host_pipeline* p = new (std::nothrow) rf_host_pipeline();
  if (p == nullptr) return RF_ERR_CUDA;
  p->shape = *shape;
  p->gshape = gs;
  p->params = *params;
  p->groups = head_groups;
  p->heads_per_group = gs.H;
  p->head_elems = ((size_t)shape->T * shape->frame_h * shape->frame_w + shape->L_text) * shape->D;
  uint8_t* b = static_cast<uint8_t*>(staging);
  p->q = reinterpret_cast<__nv_bfloat16*>(b); b += L.tensor;
  p->k = reinterpret_cast<__nv_bfloat16*>(b); b += L.tensor;
  p->v = reinterpret_cast<__nv_bfloat16*>(b); b += L.tensor;
  p->o = reinterpret_cast<__nv_bfloat16*>(b); b += L.tensor;
  p->lanes = head_groups > 1 ? 2 : 1;
  p->ws_bytes = L.ws;
  for (int r = 0; r < p->lanes; ++r) {
    p->ws[r] = b; b += L.ws;
    p->sched[r].count = reinterpret_cast<int32_t*>(b); b += L.count;
    p->sched[r].kv_tile = reinterpret_cast<int32_t*>(b); b += L.kv_tile;
    p->sched[r].kv_len = reinterpret_cast<int32_t*>(b); b += L.kv_len;
    p->sched[r].bitmap = nullptr;
    p->sched[r].nQ = nQ;
    p->sched[r].nKmax = nK;
  }
  p->head_class = reinterpret_cast<int32_t*>(b); b += L.head_class;
  p->head_window = reinterpret_cast<int32_t*>(b); b += L.head_class;
  p->n_bw = 0;
  p->status = reinterpret_cast<int32_t*>(b);
  p->s_in = p->s_run[0] = p->s_run[1] = p->s_out = nullptr;
  p->all_done = nullptr;
  p->ran = false;
  bool ok = cudaStreamCreateWithFlags(&p->s_in, cudaStreamNonBlocking) == cudaSuccess &&
            cudaStreamCreateWithFlags(&p->s_run[0], cudaStreamNonBlocking) == cudaSuccess &&
            (p->lanes < 2 || cudaStreamCreateWithFlags(&p->s_run[1], cudaStreamNonBlocking) == cudaSuccess) &&
            cudaStreamCreateWithFlags(&p->s_out, cudaStreamNonBlocking) == cudaSuccess &&
            cudaEventCreateWithFlags(&p->all_done, cudaEventDisableTiming) == cudaSuccess;
  for (auto* vec : {&p->landed, &p->run_done, &p->out_done}) {
    vec->assign(head_groups, nullptr);
    for (int g = 0; ok && g < head_groups; ++g) ok = cudaEventCreateWithFlags(&(*vec)[g], cudaEventDisableTiming) == cudaSuccess;
  }
  ok = ok && cudaMemsetAsync(p->status, 0, sizeof(int32_t), p->s_run[0]) == cudaSuccess &&
       cudaStreamSynchronize(p->s_run[0]) == cudaSuccess;
  if (!ok) {
    destroy(p);
    return RF_ERR_CUDA;
  }
  *out = p;
  return RF_OK;
}

void rf_host_pipeline_destroy(rf_host_pipeline* p) {
  if (p == nullptr) return;
  cudaStreamSynchronize(p->s_in);
  for (int r = 0; r < p->lanes; ++r) cudaStreamSynchronize(p->s_run[r]);
  cudaStreamSynchronize(p->s_out);
  destroy(p);
}

int32_t* rf_host_pipeline_status(rf_host_pipeline* p) { return p ? p->status : nullptr; }
const int32_t* rf_host_pipeline_head_class(rf_host_pipeline* p) { return p ? p->head_class : nullptr; }
const int32_t* rf_host_pipeline_head_window(rf_host_pipeline* p) { return p ? p->head_window : nullptr; }

rf_status rf_host_pipeline_set_bandwidths(rf_host_pipeline* p, const float* bandwidths, int32_t n_bandwidths) {
  if (p == nullptr || n_bandwidths < 0 || n_bandwidths > RF_MAX_BANDWIDTHS) return RF_ERR_INVALID_ARG;
  if (n_bandwidths > 0) {
    if (bandwidths == nullptr) return RF_ERR_INVALID_ARG;
    if (p->params.temporal_window_2d) return RF_ERR_UNSUPPORTED;
    for (int i = 0; i < n_bandwidths; ++i) {
      const float b = bandwidths[i];
      if (!(b > 0.f && b <= 1.f) || (i > 0 && b <= bandwidths[i - 1])) return RF_ERR_INVALID_ARG;
    }
    for (int i = 0; i < n_bandwidths; ++i) p->bw[i] = bandwidths[i];
  }
  p->n_bw = n_bandwidths;
  return RF_OK;
}

rf_status rf_host_pipeline_run(rf_host_pipeline* p, const void* q_host, const void* k_host, const void* v_host, void* o_host,
                               void* wait_stream) {
  if (p == nullptr || q_host == nullptr || k_host == nullptr || v_host == nullptr || o_host == nullptr) return RF_ERR_INVALID_ARG;
  const size_t gelems = (size_t)p->heads_per_group * p->head_elems, gbytes = gelems * sizeof(__nv_bfloat16);
  auto at = [&](const void* base, int g) { return static_cast<const uint8_t*>(base) + (size_t)g * gbytes; };
#define RF_TRY(call) do { if ((call) != cudaSuccess) return RF_ERR_CUDA; } while (0)
  for (int g = 0; g < p->groups; ++g) {
    // the previous call's kernels have read this group's staged inputs
    if (p->ran) RF_TRY(cudaStreamWaitEvent(p->s_in, p->run_done[g], 0));
    RF_TRY(cudaMemcpyAsync(p->q + g * gelems, at(q_host, g), gbytes, cudaMemcpyHostToDevice, p->s_in));
    RF_TRY(cudaMemcpyAsync(p->k + g * gelems, at(k_host, g), gbytes, cudaMemcpyHostToDevice, p->s_in));
    RF_TRY(cudaMemcpyAsync(p->v + g * gelems, at(v_host, g), gbytes, cudaMemcpyHostToDevice, p->s_in));
    RF_TRY(cudaEventRecord(p->landed[g], p->s_in));
  }
  for (int g = 0; g < p->groups; ++g) {
    const int r = g % p->lanes;
    cudaStream_t run = p->s_run[r];
    RF_TRY(cudaStreamWaitEvent(run, p->landed[g], 0));
    // the previous call's output of this group has left the staging buffer
    if (p->ran) RF_TRY(cudaStreamWaitEvent(run, p->out_done[g], 0));
    int32_t* hc = p->head_class + (size_t)g * p->heads_per_group;
    const __nv_bfloat16 *q = p->q + g * gelems, *k = p->k + g * gelems, *v = p->v + g * gelems;
    rf_status st;
    if (p->n_bw > 0) {
      int32_t* hw = p->head_window + (size_t)g * p->heads_per_group;
      st = rf_arm_classify_plus(&p->gshape, &p->params, p->bw, p->n_bw, q, k, hc, hw, nullptr, p->ws[r], p->ws_bytes, p->status,
                                run);
      if (st == RF_OK) st = rf_build_block_mask_plus(&p->gshape, &p->params, hc, hw, &p->sched[r], p->status, run);
      if (st == RF_OK)
        st = rf_sparse_attn_fwd_plus(&p->gshape, &p->params, q, k, v, hc, hw, &p->sched[r], p->o + g * gelems, nullptr, p->ws[r],
                                     p->ws_bytes, p->status, run);
    } else {
      st = rf_arm_classify(&p->gshape, &p->params, q, k, hc, nullptr, p->ws[r], p->ws_bytes, p->status, run);
      if (st == RF_OK) st = rf_build_block_mask(&p->gshape, &p->params, hc, &p->sched[r], p->status, run);
      if (st == RF_OK)
        st = rf_sparse_attn_fwd(&p->gshape, &p->params, q, k, v, hc, &p->sched[r], p->o + g * gelems, nullptr, p->ws[r],
                                p->ws_bytes, p->status, run);
    }
    if (st != RF_OK) return st;
    RF_TRY(cudaEventRecord(p->run_done[g], run));
    RF_TRY(cudaStreamWaitEvent(p->s_out, p->run_done[g], 0));
    RF_TRY(cudaMemcpyAsync(static_cast<uint8_t*>(o_host) + (size_t)g * gbytes, p->o + g * gelems, gbytes, cudaMemcpyDeviceToHost,
                           p->s_out));
    RF_TRY(cudaEventRecord(p->out_done[g], p->s_out));
  }
  p->ran = true;
  RF_TRY(cudaEventRecord(p->all_done, p->s_out));
  RF_TRY(cudaStreamWaitEvent(static_cast<cudaStream_t>(wait_stream), p->all_done, 0));
#undef RF_TRY
  return RF_OK;
}

}  // extern "C"
