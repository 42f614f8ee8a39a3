/* A caller of the library in plain C with the CUDA runtime: no Python, no torch.
 *
 * One attention call of the path of Fig. 2a on a small latent (5 frames of 6 x 7 tokens, 3 text tokens, 3 heads of
 * dimension 64): ARM picks a pattern per head (Algorithm 1), the tile schedule is built from the masks of Sec. 3.2, the
 * masked attention of Eq. 1-2 runs, O comes back to the host.  Inputs are bf16 values drawn from a 32-bit linear
 * congruential generator, so that a test can rebuild them bit for bit.
 *
 *   gcc -std=c99 -I include -I /usr/local/cuda/include rf_c_caller.c -o rf_c_caller \
 *       -L <dir of librainfusion.so> -l:librainfusion.so -L /usr/local/cuda/lib64 -lcudart -Wl,-rpath,<dir>
 *   ./rf_c_caller out.bin      # prints classes, recalls, the device status; writes O (bf16, [H][N][D]) to out.bin
 */
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <cuda_runtime_api.h>

#include "rainfusion.h"

#define CHECK_CUDA(x) do { cudaError_t e_ = (x); if (e_ != cudaSuccess) { fprintf(stderr, "%s: %s\n", #x, cudaGetErrorString(e_)); return 2; } } while (0)
#define CHECK_RF(x) do { rf_status s_ = (x); if (s_ != RF_OK) { fprintf(stderr, "%s: %s\n", #x, rf_status_string(s_)); return 3; } } while (0)

static uint32_t lcg_state;
static uint32_t lcg(void) { lcg_state = lcg_state * 1664525u + 1013904223u; return lcg_state; }

/* fp32 -> bf16 bits, round to nearest even */
static uint16_t bf16_bits(float x) {
  uint32_t u;
  memcpy(&u, &x, 4);
  u += 0x7FFFu + ((u >> 16) & 1u);
  return (uint16_t)(u >> 16);
}

/* values in [-1, 1) on a grid of 2^-15, times `scale` */
static void fill(uint16_t *dst, size_t n, uint32_t seed, float scale) {
  lcg_state = seed;
  for (size_t i = 0; i < n; ++i) dst[i] = bf16_bits(((float)(int32_t)(lcg() >> 16) - 32768.0f) * (1.0f / 32768.0f) * scale);
}

int main(int argc, char **argv) {
  rf_shape s;
  rf_params p;
  memset(&s, 0, sizeof s);
  memset(&p, 0, sizeof p);
  s.B = 1; s.H = 3; s.D = 64; s.T = 5; s.frame_h = 6; s.frame_w = 7; s.L_text = 3;
  p.frame_window = 1; p.spatial_window = 10; p.textural_stride = 2; p.sample_mode = RF_SAMPLE_ALG1; p.sample_stride = 4;
  p.alpha = 0.9f; p.block_m = 128; p.block_n = 128; p.temporal_permute = 1;

  const size_t N = (size_t)s.T * s.frame_h * s.frame_w + s.L_text, heads = (size_t)s.B * s.H;
  const size_t elems = heads * N * s.D, bytes = elems * sizeof(uint16_t);
  uint16_t *hq = malloc(bytes), *hk = malloc(bytes), *hv = malloc(bytes), *ho = malloc(bytes);
  if (!hq || !hk || !hv || !ho) return 1;
  fill(hq, elems, 1u, 2.0f);
  fill(hk, elems, 2u, 2.0f);
  fill(hv, elems, 3u, 1.0f);

  int32_t nQ = 0, nK = 0;
  CHECK_RF(rf_schedule_dims(&s, &p, &nQ, &nK));
  const size_t ws_bytes = rf_workspace_bytes(&s, &p);
  if (ws_bytes == 0) return 1;

  void *q, *k, *v, *o, *ws;
  int32_t *head_class, *status;
  float *recall, *lse;
  rf_schedule sched;
  memset(&sched, 0, sizeof sched);
  sched.nQ = nQ; sched.nKmax = nK;
  CHECK_CUDA(cudaMalloc(&q, bytes)); CHECK_CUDA(cudaMalloc(&k, bytes)); CHECK_CUDA(cudaMalloc(&v, bytes)); CHECK_CUDA(cudaMalloc(&o, bytes));
  CHECK_CUDA(cudaMalloc(&ws, ws_bytes));                  /* cudaMalloc is 256-byte aligned */
  CHECK_CUDA(cudaMalloc((void **)&head_class, heads * sizeof(int32_t)));
  CHECK_CUDA(cudaMalloc((void **)&status, sizeof(int32_t)));
  CHECK_CUDA(cudaMalloc((void **)&recall, heads * 3 * sizeof(float)));
  CHECK_CUDA(cudaMalloc((void **)&lse, heads * N * sizeof(float)));
  CHECK_CUDA(cudaMalloc((void **)&sched.count, heads * nQ * sizeof(int32_t)));
  CHECK_CUDA(cudaMalloc((void **)&sched.kv_tile, heads * nQ * nK * sizeof(int32_t)));
  CHECK_CUDA(cudaMalloc((void **)&sched.kv_len, heads * sizeof(int32_t)));
  CHECK_CUDA(cudaMemset(status, 0, sizeof(int32_t)));
  CHECK_CUDA(cudaMemcpy(q, hq, bytes, cudaMemcpyHostToDevice));
  CHECK_CUDA(cudaMemcpy(k, hk, bytes, cudaMemcpyHostToDevice));
  CHECK_CUDA(cudaMemcpy(v, hv, bytes, cudaMemcpyHostToDevice));

  cudaStream_t stream;
  CHECK_CUDA(cudaStreamCreate(&stream));
  /* the three calls of one attention layer; head_class never leaves the device */
  CHECK_RF(rf_arm_classify(&s, &p, q, k, head_class, recall, ws, ws_bytes, status, stream));
  CHECK_RF(rf_build_block_mask(&s, &p, head_class, &sched, status, stream));
  CHECK_RF(rf_sparse_attn_fwd(&s, &p, q, k, v, head_class, &sched, o, lse, ws, ws_bytes, status, stream));
  CHECK_CUDA(cudaStreamSynchronize(stream));

  int32_t hstatus = -1, hclass[3];
  float hrecall[9];
  CHECK_CUDA(cudaMemcpy(&hstatus, status, sizeof hstatus, cudaMemcpyDeviceToHost));
  CHECK_CUDA(cudaMemcpy(hclass, head_class, sizeof hclass, cudaMemcpyDeviceToHost));
  CHECK_CUDA(cudaMemcpy(hrecall, recall, sizeof hrecall, cudaMemcpyDeviceToHost));
  CHECK_CUDA(cudaMemcpy(ho, o, bytes, cudaMemcpyDeviceToHost));
  printf("status %d\n", (int)hstatus);
  for (int h = 0; h < 3; ++h)
    printf("head %d class %d recall_temporal %.6f recall_spatial %.6f recall_textural %.6f\n", h, (int)hclass[h],
           hrecall[3 * h], hrecall[3 * h + 1], hrecall[3 * h + 2]);
  if (argc > 1) {
    FILE *f = fopen(argv[1], "wb");
    if (!f || fwrite(ho, 1, bytes, f) != bytes) return 4;
    fclose(f);
  }
  cudaFree(q); cudaFree(k); cudaFree(v); cudaFree(o); cudaFree(ws); cudaFree(head_class); cudaFree(status); cudaFree(recall);
  cudaFree(lse); cudaFree(sched.count); cudaFree(sched.kv_tile); cudaFree(sched.kv_len);
  cudaStreamDestroy(stream);
  free(hq); free(hk); free(hv); free(ho);
  return hstatus == 0 ? 0 : 5;
}
