/* A plain C99 caller of the library's header: prints the layout of the structures and the results of the entry
 * points that run on the host alone, one "key value" pair per line.  tests/test_abi_cpu.py compiles it with gcc,
 * links it against the built library and compares every line with what the ctypes binding holds and returns, so a
 * field added on one side only, or a changed type, fails a CPU test.  No GPU is touched. */
#include <stddef.h>
#include <stdio.h>
#include <string.h>

#include "rainfusion.h"

#define OFF(type, field) printf("offsetof." #type "." #field " %zu\n", offsetof(type, field))

int main(void) {
  printf("sizeof.rf_shape %zu\n", sizeof(rf_shape));
  printf("sizeof.rf_params %zu\n", sizeof(rf_params));
  printf("sizeof.rf_schedule %zu\n", sizeof(rf_schedule));
  OFF(rf_shape, B); OFF(rf_shape, H); OFF(rf_shape, D); OFF(rf_shape, T); OFF(rf_shape, frame_h); OFF(rf_shape, frame_w);
  OFF(rf_shape, L_text);
  OFF(rf_params, frame_window); OFF(rf_params, spatial_window); OFF(rf_params, textural_stride); OFF(rf_params, sample_mode);
  OFF(rf_params, sample_stride); OFF(rf_params, alpha); OFF(rf_params, block_m); OFF(rf_params, block_n);
  OFF(rf_params, temporal_permute); OFF(rf_params, two_mask); OFF(rf_params, spatial_key_first_frame);
  OFF(rf_params, temporal_window_2d); OFF(rf_params, temporal_window_y); OFF(rf_params, temporal_window_x);
  OFF(rf_schedule, count); OFF(rf_schedule, kv_tile); OFF(rf_schedule, bitmap); OFF(rf_schedule, kv_len);
  OFF(rf_schedule, nQ); OFF(rf_schedule, nKmax);

  /* a latent of 5 frames of 6 x 7 tokens with 3 text tokens, three heads of dimension 64 */
  rf_shape s;
  rf_params p;
  memset(&s, 0, sizeof s);
  memset(&p, 0, sizeof p);
  s.B = 1; s.H = 3; s.D = 64; s.T = 5; s.frame_h = 6; s.frame_w = 7; s.L_text = 3;
  p.frame_window = 1; p.spatial_window = 10; p.textural_stride = 2; p.sample_mode = RF_SAMPLE_ALG1; p.sample_stride = 4;
  p.alpha = 0.9f; p.block_m = 128; p.block_n = 128; p.temporal_permute = 1;

  int32_t nQ = -1, nK = -1;
  printf("dims.status %d\n", (int)rf_schedule_dims(&s, &p, &nQ, &nK));
  printf("dims.nQ %d\n", (int)nQ);
  printf("dims.nKmax %d\n", (int)nK);
  printf("workspace_bytes %zu\n", rf_workspace_bytes(&s, &p));
  printf("staging_bytes.3 %zu\n", rf_host_pipeline_staging_bytes(&s, &p, 3));
  printf("staging_bytes.2 %zu\n", rf_host_pipeline_staging_bytes(&s, &p, 2));   /* 2 does not divide 3 heads: 0 */
  p.block_m = 16; p.block_n = 32;
  printf("dims16x32.status %d\n", (int)rf_schedule_dims(&s, &p, &nQ, &nK));
  printf("dims16x32.nQ %d\n", (int)nQ);
  printf("dims16x32.nKmax %d\n", (int)nK);
  p.temporal_window_2d = 1; p.temporal_window_y = -1; p.temporal_window_x = 2;
  printf("bad2d.status %d\n", (int)rf_schedule_dims(&s, &p, &nQ, &nK));
  p.temporal_window_y = 1;
  printf("good2d.status %d\n", (int)rf_schedule_dims(&s, &p, &nQ, &nK));
  printf("null.status %d\n", (int)rf_schedule_dims(NULL, &p, &nQ, &nK));
  printf("bounds_checked %d\n", (int)rf_bounds_checked());
  for (int c = 0; c <= 7; ++c) printf("status_string.%d %s\n", c, rf_status_string((rf_status)c));
  return 0;
}
