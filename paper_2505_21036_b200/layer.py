"""One attention layer's call sequence, as the sampler of a video DiT would drive it.

Policy only: which entry points of the C ABI run at which denoising step, with which buffers.  Every
arithmetic step is a kernel of the library.

  * the first `dense_fraction` of the sampling steps run dense attention (Sec. 4.2 keeps the first tenth of
    the timesteps dense);
  * every later step runs ARM -> tile schedule -> pattern-masked attention (Fig. 2a: the head categories are
    determined online, per call);
  * with `graph=True` the three calls of a sparse step are captured once into a CUDA graph per set of
    tensor addresses and replayed: the kernels take no host decision between them (head_class stays on
    the device), so a replay is the same work with one launch from the host.
"""
from __future__ import annotations

import math

from . import api


class RainFusionAttention:
    def __init__(self, shape: api.rf_shape, params: api.rf_params, device, dense_fraction: float = 0.1,
                 graph: bool = False, bandwidths=None):
        import torch
        if not (0.0 <= dense_fraction <= 1.0):
            raise ValueError("dense_fraction must be in [0, 1]")
        self.shape, self.params, self.device = shape, params, device
        self.dense_fraction = dense_fraction
        self.use_graph = graph
        self.bandwidths = list(bandwidths) if bandwidths else None      # RainFusion+ (Sec. 4.3) when given
        self.ws = api.alloc_workspace(shape, params, device)
        self.sched = api.Schedule(shape, params, device)
        self.head_class = torch.zeros((shape.B, shape.H), dtype=torch.int32, device=device)
        self.head_window = (torch.zeros((shape.B, shape.H), dtype=torch.int32, device=device)
                            if self.bandwidths else None)
        self.status = torch.zeros(1, dtype=torch.int32, device=device)
        self._graphs = {}

    # ------------------------------------------------------------------ policy
    def dense_steps(self, num_steps: int) -> int:
        """Number of leading sampling steps that stay dense."""
        return int(math.ceil(self.dense_fraction * num_steps - 1e-9))

    def is_dense_step(self, step: int, num_steps: int) -> bool:
        return step < self.dense_steps(num_steps)

    # ------------------------------------------------------------------ calls
    def _sparse(self, q, k, v, o, lse):
        s, p = self.shape, self.params
        if self.bandwidths:
            api.rf_arm_classify_plus(s, p, self.bandwidths, q, k, self.head_class, self.head_window, None, self.ws,
                                     self.status)
            api.rf_build_block_mask_plus(s, p, self.head_class, self.head_window, self.sched, self.status)
            api.rf_sparse_attn_fwd_plus(s, p, q, k, v, self.head_class, self.head_window, self.sched, o, lse, self.ws,
                                        self.status)
        else:
            api.rf_arm_classify(s, p, q, k, self.head_class, None, self.ws, self.status)
            api.rf_build_block_mask(s, p, self.head_class, self.sched, self.status)
            api.rf_sparse_attn_fwd(s, p, q, k, v, self.head_class, self.sched, o, lse, self.ws, self.status)

    def _sparse_graphed(self, q, k, v, o, lse):
        import torch
        key = (q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), None if lse is None else lse.data_ptr())
        g = self._graphs.get(key)
        if g is None:
            # one eager call first: per-device kernel attributes are set on first use, outside any capture
            self._sparse(q, k, v, o, lse)
            torch.cuda.current_stream().synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                self._sparse(q, k, v, o, lse)
            self._graphs[key] = g
        g.replay()

    def __call__(self, q, k, v, o, lse=None, step: int = 0, num_steps: int = 1):
        """Attention of one layer at sampling step `step` of `num_steps`; writes o (and lse)."""
        if self.is_dense_step(step, num_steps):
            api.rf_dense_attn_fwd(self.shape, q, k, v, o, lse, self.status)
        elif self.use_graph:
            self._sparse_graphed(q, k, v, o, lse)
        else:
            self._sparse(q, k, v, o, lse)

    def check(self):
        """Raises if a kernel reported an error since the last check (reads the device status word)."""
        code = int(self.status.item())
        if code != 0:
            self.status.zero_()
            raise api.RainFusionError(f"device status {code}: {api.load().rf_status_string(code).decode()}")

    def expected_attention_speedup(self, num_steps: int, density: float) -> float:
        """Whole-run attention speed-up if a sparse step costs `density` of a dense one (Sec. 4.2's arithmetic)."""
        d = self.dense_steps(num_steps)
        return num_steps / (d + (num_steps - d) * density)


class HostStagedAttention:
    """The whole path for callers whose Q, K, V and O live in (pinned) host memory: a thin wrapper over the
    library's rf_host_pipeline_* calls, which pipeline groups of heads over a copy-in stream, two alternating compute
    streams and a copy-out stream (heads are independent at every stage: Algorithm 1 classifies per head; masks and attention are per
    head).  Per call every byte of Q, K, V still crosses to the device and every byte of O comes back; only the
    waiting is overlapped, inside a call and between calls made back to back."""

    def __init__(self, shape: api.rf_shape, params: api.rf_params, device, groups: int = 4):
        heads = shape.B * shape.H
        if groups < 1 or heads % groups != 0:
            raise ValueError("groups must divide B*H")
        self.shape, self.params, self.device, self.groups = shape, params, device, groups
        self.N = shape.T * shape.frame_h * shape.frame_w + shape.L_text
        self.pipe = api.HostPipeline(shape, params, device, groups)
        self.h2d_bytes = 3 * heads * self.N * shape.D * 2
        self.d2h_bytes = heads * self.N * shape.D * 2

    def __call__(self, qh, kh, vh, oh):
        """qh, kh, vh, oh: pinned host bf16 tensors of [B, H, N, D]; the inputs must be complete in host memory
        when the call is made.  Returns when the work is enqueued; the current stream waits for the output copy."""
        for t in (qh, kh, vh, oh):
            if t.is_cuda or not t.is_contiguous():
                raise ValueError("host-staged call takes contiguous host tensors")
        self.pipe.run(qh, kh, vh, oh)

    @property
    def status(self):
        """Object with .item(): the pipeline's device status word."""
        pipe = self.pipe

        class _S:
            def item(self_inner):
                return pipe.status()
        return _S()
