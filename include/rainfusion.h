/*
 * rainfusion.h - C ABI of the B200 (sm_100a) RainFusion hot path:
 * per-head adaptive block-sparse 3D attention for video Diffusion Transformers
 * (arxiv 2505.21036).
 *
 * Pipeline of one attention call (Sec. 1, last paragraph; Fig. 2a):
 *   rf_arm_classify      ARM: one pattern per head from sampled scores   (Sec. 3.3, Eq. 6, Algorithm 1)
 *   rf_build_block_mask  pattern masks as per-head lists of KV tiles     (Sec. 3.2, Eq. 3-5)
 *   rf_sparse_attn_fwd   attention that skips what the pattern masks     (Eq. 1-2 with the pattern's mask)
 *   rf_dense_attn_fwd    full 3D attention, the dense baseline           (Eq. 1-2)
 *
 * Conventions for every entry point
 *   - Tensors Q, K, V, O are bf16, contiguous [B, H, N, D], N = T*frame_h*frame_w + L_text.
 *     Video tokens come first, frame-major and row-major inside a frame (Sec. 3.1); text tokens last.
 *   - Pointers marked "device" are CUDA device pointers owned by the caller; rf_shape / rf_params /
 *     rf_schedule structs themselves are host memory, read during the call.
 *   - All work is enqueued on `cuda_stream` (a cudaStream_t passed as void*; NULL = default
 *     stream).  No entry point synchronises the host or allocates device memory.  The library keeps
 *     no state between calls apart from per-device kernel attributes set on first use.
 *   - Host-detectable errors return a code before anything is launched.  Device-detected ones
 *     (a bounded wait that ran out, a head class outside 0..3) are written to *dev_status
 *     (device int32, may be NULL; never reset by the library; the first error stays) and the kernels
 *     still terminate.  Every entry point that launches a kernel with such a wait takes a dev_status.
 *     If a wait runs out inside ARM, head_class (and head_window) are written as -1 for every head, so
 *     that rf_build_block_mask and rf_sparse_attn_fwd, given those classes, report RF_ERR_INVALID_ARG
 *     through their own dev_status even when ARM itself was given none.
 *   - frame_window >= T, spatial_window >= frame_h*frame_w and textural_stride >= max(frame_h, frame_w)
 *     are accepted and mean what the extent itself means (all frames, all positions, the diagonal y == x).
 *   - Supported: D in {64, 96, 128}; block_m = block_n = 128 for the attention entry points;
 *     rf_build_block_mask alone accepts any power-of-two blocks >= 16.
 */
#ifndef RAINFUSION_H_
#define RAINFUSION_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  RF_OK = 0,
  RF_ERR_INVALID_ARG = 1,
  RF_ERR_UNSUPPORTED = 2,
  RF_ERR_WORKSPACE_TOO_SMALL = 3,
  RF_ERR_CUDA = 4,
  RF_ERR_TIMEOUT = 5,
  RF_ERR_STATIC_SCRATCH_TOO_SMALL = 6,
  RF_ERR_BOUNDS = 7   /* only from a library built with -DRF_BOUNDS_CHECK: a kernel was about to index outside an
                         array (reported through dev_status; the access is skipped, nothing traps) */
} rf_status;

/* Head categories (Sec. 3.2).  RF_DENSE is not an ARM outcome; a caller may force it. */
typedef enum { RF_SPATIAL = 0, RF_TEMPORAL = 1, RF_TEXTURAL = 2, RF_DENSE = 3 } rf_pattern;

/* Which sample feeds which recall (Sec. 3.3; ablation column "L" of Table 2). */
typedef enum {
  RF_SAMPLE_ALG1 = 0,   /* Temporal recall on the first frame's tokens, Spatial recall on the stride sample */
  RF_SAMPLE_GLOBAL = 1  /* both recalls on the stride sample */
} rf_sample_mode;

typedef struct {
  int32_t B, H, D;            /* batch, heads, head dimension */
  int32_t T;                  /* latent frames */
  int32_t frame_h, frame_w;   /* tokens per frame = frame_h * frame_w */
  int32_t L_text;             /* text tokens appended after the video tokens (>= 0) */
} rf_shape;

typedef struct {
  int32_t frame_window;     /* w_f >= 0: a Spatial head keeps keys with |frame(q) - frame(k)| <= w_f (Eq. 3) */
  int32_t spatial_window;   /* w_s >= 0: a Temporal head keeps keys with |pos(q) - pos(k)| <= w_s, pos = y*frame_w + x */
  int32_t textural_stride;  /* tau >= 1: a Textural head keeps key (y, x) iff y mod tau == x mod tau (Eq. 4) */
  int32_t sample_mode;      /* rf_sample_mode */
  int32_t sample_stride;    /* omega >= 1: the stride sample is video tokens 0, omega, 2*omega, ... */
  float   alpha;            /* recall threshold of Algorithm 1, in (0, 1] */
  int32_t block_m, block_n; /* tile of the block mask: query rows x key slots */
  int32_t temporal_permute; /* 1: Temporal heads run in position-major token order (slot = pos*T + frame) */
  int32_t two_mask;         /* 0: Algorithm 1 as printed (Spatial, Temporal, else Textural).  1: the ablation of
                               Sec. 4.4 / Table 2 with only the Spatial and Temporal masks: a head that reaches alpha
                               with neither takes the one of larger recall (Temporal on equality), never Textural */
  int32_t spatial_key_first_frame; /* 0: a Spatial head keeps the frames within w_f (Eq. 3).  1: it keeps, in addition,
                               every key of frame 0 for every query: Sec. 3.2 lets the attended set hold adjacent
                               or key frames; the first frame is the one key frame offered here */
  int32_t temporal_window_2d; /* 0: a Temporal head keeps the 1-D band |pos(q) - pos(k)| <= spatial_window.  1: it keeps
                               the 2-D window |y(q) - y(k)| <= temporal_window_y and |x(q) - x(k)| <= temporal_window_x on
                               the rows and columns of the frame instead (the other reading of Sec. 3.2's locality inside
                               a frame; spatial_window is then unused).  Needs frame_h, frame_w < 32768; not available
                               with the dynamic-bandwidth entry points (RF_ERR_UNSUPPORTED) */
  int32_t temporal_window_y, temporal_window_x;   /* >= 0; read only when temporal_window_2d = 1 */
} rf_params;

/*
 * Tile schedule: for every (b, h, query tile a) the ascending list of non-empty KV tiles in the
 * head's own coordinate space (Dense/Spatial/Temporal: original order, or position-major for
 * Temporal with temporal_permute; Textural: the kept set C in ascending order, then text).
 * Entry = tile index, with bit 31 set when the tile is PARTIAL (some pair in it is masked, or
 * it holds fewer than block_n real key slots); FULL tiles need no element mask.
 * All arrays are device memory allocated by the caller.
 */
typedef struct {
  int32_t  *count;    /* [B, H, nQ] */
  int32_t  *kv_tile;  /* [B, H, nQ, nKmax], first count[...] entries of a row are valid */
  uint32_t *bitmap;   /* optional [B, H, nQ, ceil(nKmax/32)] bit b = tile b listed; may be NULL */
  int32_t  *kv_len;   /* [B, H] number of key slots of the head (N, or |C|*T + L_text for Textural) */
  int32_t   nQ, nKmax;
} rf_schedule;

const char *rf_status_string(rf_status s);

/* 1 if this library was built with -DRF_BOUNDS_CHECK (every kernel checks the indices of its global-memory
 * writes and of the schedule entries it reads, reports RF_ERR_BOUNDS through dev_status and skips the access),
 * else 0.  The memory checker of the CUDA toolkit is not available everywhere; this build is its stand-in for tests. */
int32_t rf_bounds_checked(void);

/* Host, pure: nQ = ceil(N/block_m), nKmax = ceil(N/block_n). */
rf_status rf_schedule_dims(const rf_shape *shape, const rf_params *params, int32_t *nQ, int32_t *nKmax);

/* Host, pure: bytes of device workspace that rf_arm_classify / rf_sparse_attn_fwd need
 * (reordered Q/K/V copies for Temporal and Textural heads, ARM per-row recalls).  0 on bad arguments. */
size_t rf_workspace_bytes(const rf_shape *shape, const rf_params *params);

/*
 * ARM (Sec. 3.3, Eq. 6, Algorithm 1).  For every (b, h): approximate softmax scores on the sampled
 * queries/keys, the share of each row's mass kept by the sampled Temporal / Spatial / Textural mask,
 * averaged over rows, then Temporal if R_t >= alpha, else Spatial if R_s >= alpha, else Textural.
 *   q, k        device bf16 [B,H,N,D]
 *   head_class  device int32 [B,H], written
 *   recall      device float [B,H,3] = (R_temporal, R_spatial, R_textural), written; may be NULL
 *   ws          device workspace of at least rf_workspace_bytes(), 256-byte aligned
 *   dev_status  device int32 or NULL: RF_ERR_TIMEOUT if a wait inside the score kernel ran out (head_class
 *               is then -1 for every head and recall is left unwritten)
 */
rf_status rf_arm_classify(const rf_shape *shape, const rf_params *params, const void *q, const void *k,
                          int32_t *head_class, float *recall, void *ws, size_t ws_bytes, int32_t *dev_status,
                          void *cuda_stream);

/*
 * Block mask / tile schedule of the pattern masks of Sec. 3.2 (Eq. 3-5), per head, from device-resident
 * head classes.  Fills out->count, out->kv_tile, out->kv_len (and out->bitmap when not NULL);
 * out->nQ / out->nKmax must equal rf_schedule_dims().
 */
rf_status rf_build_block_mask(const rf_shape *shape, const rf_params *params, const int32_t *head_class,
                              rf_schedule *out, int32_t *dev_status, void *cuda_stream);

/*
 * Pattern-masked attention forward (Eq. 1-2 with M_spatial / M_temporal / the checkerboard K_C, V_C
 * of Eq. 5).  Visits only the listed tiles and applies the exact element mask inside PARTIAL tiles,
 * so the result does not depend on the tile size or on temporal_permute.
 *   q, k, v     device bf16 [B,H,N,D]
 *   head_class  device int32 [B,H] (the classes the schedule was built from)
 *   o           device bf16 [B,H,N,D], written in original token order
 *   lse         device float [B,H,N], natural-log sum of exp(score) over kept keys; may be NULL
 *   ws          as for rf_arm_classify; holds the reordered copies this call makes
 */
rf_status rf_sparse_attn_fwd(const rf_shape *shape, const rf_params *params, const void *q, const void *k,
                             const void *v, const int32_t *head_class, const rf_schedule *sched, void *o,
                             float *lse, void *ws, size_t ws_bytes, int32_t *dev_status, void *cuda_stream);

/*
 * The token reordering that rf_sparse_attn_fwd performs before its attention kernel, on its own
 * (Sec. 3.2, Textural Head: the K, V sequence is rearranged and the checkerboard tokens retained;
 * Temporal heads with temporal_permute: Q, K, V to position-major order).  Writes the copies into ws.
 * Exposed so that the reordering can be timed or reused separately; rf_sparse_attn_fwd does not need
 * it to be called first.
 */
rf_status rf_reorder_tokens(const rf_shape *shape, const rf_params *params, const void *q, const void *k,
                            const void *v, const int32_t *head_class, void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * The attention kernel of rf_sparse_attn_fwd on its own (Eq. 1-2 under the masks of Eq. 3 and Eq. 5): the same
 * arguments as rf_sparse_attn_fwd_plus (head_window may be NULL), but no reordering pass is launched.  ws must
 * hold what rf_reorder_tokens wrote for the same q, k, v and head_class, earlier on the same stream.
 * rf_reorder_tokens followed by this call is rf_sparse_attn_fwd, bit for bit; the split lets a caller reuse
 * one reordering for several calls and lets each of the two kernels be timed by itself.
 */
rf_status rf_sparse_attn_reordered(const rf_shape *shape, const rf_params *params, const void *q, const void *k,
                                   const void *v, const int32_t *head_class, const int32_t *head_window,
                                   const rf_schedule *sched, void *o, float *lse, void *ws, size_t ws_bytes,
                                   int32_t *dev_status, void *cuda_stream);

/*
 * Self-test of the device-side failure handling (no counterpart in the paper).  Every wait inside the kernels
 * (on TMA data, on the tensor cores, on another warp role) is bounded; when one runs out the CTA stops waiting,
 * reports RF_ERR_TIMEOUT through dev_status and still terminates normally.  This entry point launches one warp
 * that waits limit_ms (1..1000) on a barrier nobody arrives at, so that the mechanism can be exercised without
 * faulting or hanging the GPU.  On return (after the stream is synchronised) *dev_status is RF_ERR_TIMEOUT if it
 * was 0 before, and *waits_returned is 4: neither wait succeeded, the abort flag is set.
 */
rf_status rf_selftest_wait_timeout(int32_t *dev_status, int32_t limit_ms, int32_t *waits_returned, void *cuda_stream);

/*
 * Self-test of ARM's failure reporting (no counterpart in the paper).  Runs rf_arm_classify's launch sequence
 * with the score kernel left out and its failure flag set instead, exactly as a wait that ran out inside that
 * kernel leaves it.  Nothing waits and nothing stalls.  Afterwards head_class is -1 for every head and
 * *dev_status is RF_ERR_TIMEOUT if it was 0 before; rf_build_block_mask / rf_sparse_attn_fwd given those
 * classes report RF_ERR_INVALID_ARG through their dev_status.  Arguments as for rf_arm_classify.
 */
rf_status rf_selftest_arm_abandoned(const rf_shape *shape, const rf_params *params, const void *q, const void *k,
                                    int32_t *head_class, void *ws, size_t ws_bytes, int32_t *dev_status,
                                    void *cuda_stream);

/* Full 3D attention (Eq. 1-2, all-zero mask): the same kernel walking every tile.  ws may be NULL. */
rf_status rf_dense_attn_fwd(const rf_shape *shape, const void *q, const void *k, const void *v, void *o,
                            float *lse, void *ws, size_t ws_bytes, int32_t *dev_status, void *cuda_stream);

/*
 * RainFusion+ (Sec. 4.3, last paragraph): per-head dynamic bandwidth.  ARM evaluates every candidate bandwidth
 * of the list (ascending, e.g. 0.125, 0.25, 0.5; at most RF_MAX_BANDWIDTHS) on the same approximate scores.
 * A bandwidth b stands for the windows w_f = floor(b*T), w_s = floor(b*frame_h*frame_w).  A pattern qualifies
 * if any candidate reaches alpha, Temporal before Spatial as in Algorithm 1, and the head takes the smallest
 * qualifying bandwidth; otherwise it is Textural.
 *   bandwidths   host float [n_bandwidths], ascending, each in (0, 1]
 *   head_window  device int32 [B,H], written: w_s of a Temporal head, w_f of a Spatial head, -1 for Textural
 *   recall       device float [B,H,2,n_bandwidths] = (Temporal, Spatial) x candidate, written; may be NULL
 *   dev_status   as for rf_arm_classify (head_class and head_window are -1 after a wait that ran out)
 * rf_build_block_mask_plus / rf_sparse_attn_fwd_plus are rf_build_block_mask / rf_sparse_attn_fwd with those
 * per-head windows in place of params->frame_window / spatial_window (head_window == NULL: identical to them).
 */
#define RF_MAX_BANDWIDTHS 4
rf_status rf_arm_classify_plus(const rf_shape *shape, const rf_params *params, const float *bandwidths,
                               int32_t n_bandwidths, const void *q, const void *k, int32_t *head_class,
                               int32_t *head_window, float *recall, void *ws, size_t ws_bytes, int32_t *dev_status,
                               void *cuda_stream);
rf_status rf_build_block_mask_plus(const rf_shape *shape, const rf_params *params, const int32_t *head_class,
                                   const int32_t *head_window, rf_schedule *out, int32_t *dev_status, void *cuda_stream);
rf_status rf_sparse_attn_fwd_plus(const rf_shape *shape, const rf_params *params, const void *q, const void *k,
                                  const void *v, const int32_t *head_class, const int32_t *head_window,
                                  const rf_schedule *sched, void *o, float *lse, void *ws, size_t ws_bytes,
                                  int32_t *dev_status, void *cuda_stream);

/*
 * The whole path of Fig. 2a (ARM of Sec. 3.3 -> masks of Sec. 3.2 -> masked attention, Eq. 1-2) for callers whose
 * Q, K, V and O live in HOST memory.  Heads are independent at every stage (Algorithm 1 outputs one category per
 * head), so a run is pipelined over `head_groups` groups of heads (head_groups must divide B*H) on streams of the
 * pipeline's own: copy-in, copy-out, and two compute streams that consecutive groups alternate on (so that one
 * group's kernels fill the SMs the previous group's last CTAs leave).  Every byte of Q, K, V crosses to the device
 * and every byte of O comes back in every run; only the waiting overlaps, inside a run and between runs made back
 * to back.
 *   rf_host_pipeline_staging_bytes  host, pure: device bytes the pipeline needs (staged Q, K, V, O for all heads,
 *                                   workspace and schedule of one group per compute stream, classes, status).
 *                                   0 on bad arguments.
 *   rf_host_pipeline_create         staging: device memory of at least that size, 256-byte aligned, owned by the caller
 *                                   and handed to the pipeline until it is destroyed.  Creates streams and events only.
 *   rf_host_pipeline_run            q/k/v/o_host: host bf16 [B,H,N,D], pinned for the copies to overlap; the inputs
 *                                   must be complete in host memory when the call is made.  Returns when the work is
 *                                   enqueued; `wait_stream` (a cudaStream_t, NULL = default stream) is made to wait for
 *                                   the last output copy.  o_host may be read once that stream has been synchronised.
 *   rf_host_pipeline_set_bandwidths host: candidate bandwidths of the dynamic-bandwidth variant (as for
 *                                   rf_arm_classify_plus; copied); from the next run on every head takes its own
 *                                   window.  n_bandwidths = 0 returns to the fixed windows of `params`.
 *                                   RF_ERR_UNSUPPORTED with params->temporal_window_2d.
 *   rf_host_pipeline_head_class / _head_window   device int32 [B*H], what ARM decided in the last run (the windows
 *                                   are written only while bandwidths are set); valid once that run has finished
 *   rf_host_pipeline_status         device int32 the pipeline's kernels report to (dev_status of the calls above)
 *   rf_host_pipeline_destroy        waits for the pipeline's streams, then releases streams and events
 * Errors: RF_ERR_INVALID_ARG (null pointers, head_groups not dividing B*H, misaligned staging), RF_ERR_UNSUPPORTED
 * (head dimension, block size), RF_ERR_WORKSPACE_TOO_SMALL (staging), RF_ERR_CUDA.
 */
typedef struct rf_host_pipeline rf_host_pipeline;
size_t rf_host_pipeline_staging_bytes(const rf_shape *shape, const rf_params *params, int32_t head_groups);
rf_status rf_host_pipeline_create(const rf_shape *shape, const rf_params *params, int32_t head_groups, void *staging,
                                  size_t staging_bytes, rf_host_pipeline **out);
rf_status rf_host_pipeline_run(rf_host_pipeline *p, const void *q_host, const void *k_host, const void *v_host,
                               void *o_host, void *wait_stream);
rf_status rf_host_pipeline_set_bandwidths(rf_host_pipeline *p, const float *bandwidths, int32_t n_bandwidths);
const int32_t *rf_host_pipeline_head_class(rf_host_pipeline *p);
const int32_t *rf_host_pipeline_head_window(rf_host_pipeline *p);
int32_t *rf_host_pipeline_status(rf_host_pipeline *p);
void rf_host_pipeline_destroy(rf_host_pipeline *p);

/*
 * rf_arm_classify for callers that cannot provide a workspace.  (The paper has no counterpart: this is
 * a packaging variant of rf_arm_classify, same kernels, same results.)
 *
 * Some callers of this library run where device allocation is off limits: inside a serving loop
 * whose memory pool was sized and frozen at start-up, or under a framework allocator that must not be
 * re-entered from a plug-in, so they have no buffer to hand over as `ws` and may not call cudaMalloc
 * to make one.  This entry point takes only inputs and outputs.  Its per-row recall scratch lives in
 * a fixed array inside the library's device image: RF_ARM_STATIC_SCRATCH_FLOATS floats (4 MiB) that
 * every GPU which loads the library holds until the process exits.
 *
 *   - Limit: 2 * B * H * 3 * roundup64(max(frame_h*frame_w, ceil(T*frame_h*frame_w / sample_stride))) + 64
 *     floats must fit (the HunyuanVideo-720p layer needs 525 376).  Larger problems are rejected
 *     with RF_ERR_STATIC_SCRATCH_TOO_SMALL before anything is launched.
 *   - Allocates nothing: no cudaMalloc / cudaFree, no allocating library call.
 *   - The first call on each device looks up the array's device address (cudaGetSymbolAddress, with
 *     that device current).  Make that first call outside any stream capture.
 *   - All calls share the one array and it keeps the previous call's contents.  The one word of it that
 *     has to start at zero (the flag that records a wait that ran out) is cleared by every call on its
 *     stream before its kernels run; every other element that is read was written earlier in the same
 *     call.  But two calls that overlap on the GPU - different streams, or different host threads -
 *     race on the array.  Serialise them, or use rf_arm_classify with separate workspaces.
 *   - dev_status: as for rf_arm_classify.
 */
#define RF_ARM_STATIC_SCRATCH_FLOATS (1u << 20)
rf_status rf_arm_classify_noalloc(const rf_shape *shape, const rf_params *params, const void *q, const void *k,
                                  int32_t *head_class, float *recall, int32_t *dev_status, void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* RAINFUSION_H_ */
