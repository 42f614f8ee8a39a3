"""Helpers shared by the GPU parity tests: upload seeded inputs, run the C-ABI path, call the oracle."""
from __future__ import annotations

import numpy as np
import torch

from oracle import rainfusion_oracle as orc
from paper_2505_21036_b200 import api, synth

# Tolerances for bf16 inputs against the fp64 oracle (bf16 rounding of P and of the stored O):
# max-abs 2e-2, mean-abs 2e-3 on O; relative L2 2e-2 per head; 2e-3 on lse.
O_MAX_ABS, O_MEAN_ABS, O_REL_L2, LSE_ABS = 2e-2, 2e-3, 2e-2, 2e-3
RECALL_ABS = 2e-4
TIE_MARGIN = 1e-3


def geom(wl):
    return orc.Geometry(wl.T, wl.frame_h, wl.frame_w, wl.L_text)


def pparams(wl, key_first=False, t2d=None):
    return orc.PatternParams(wl.frame_window, wl.spatial_window, wl.textural_stride, bool(key_first),
                             None if t2d is None else tuple(t2d))


def to_dev(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def bits_of(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().view(torch.int16).numpy().view(np.uint16)


GUARD_BYTES = 1024          # on each side of every buffer a kernel writes; a multiple of the 256-byte alignment
GUARD_BYTE = 0xA5


class Guarded:
    """Device buffers a kernel writes, each carved out of a larger allocation with GUARD_BYTES of a known
    pattern in front of it and behind it.  check() verifies that every guard still holds the pattern: with the
    memory checker unavailable this is the evidence that no kernel writes outside its outputs (a stray store
    that lands further away than a guard goes unseen, one that is off by a row or a tile does not)."""

    def __init__(self):
        self.guards = []

    def alloc(self, shape, dtype, fill=None, name=""):
        n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        padded = -(-n // 256) * 256
        raw = torch.full((GUARD_BYTES + padded + GUARD_BYTES,), GUARD_BYTE, dtype=torch.uint8, device="cuda")
        assert raw.data_ptr() % 256 == 0
        body = raw[GUARD_BYTES:GUARD_BYTES + n].view(dtype).view(*shape)
        if fill is not None:
            body.fill_(fill)
        # the slack between the buffer's end and the next 256-byte boundary is guard too
        self.guards.append((name, raw, n))
        return body

    def check(self, what=""):
        for name, raw, n in self.guards:
            front = raw[:GUARD_BYTES]
            back = raw[GUARD_BYTES + n:]
            ok = bool((front == GUARD_BYTE).all().item()) and bool((back == GUARD_BYTE).all().item())
            assert ok, f"{what}: bytes next to `{name}` were overwritten"


class Run:
    """One workload resident on the GPU with its schedule and workspace.  Every buffer the library writes
    (classes, recalls, schedule arrays, workspace, outputs) sits between guard words that are checked after
    every call."""

    def __init__(self, wl, qkv=None, block=128, temporal_permute=1, two_mask=0, key_first=0, t2d=None):
        self.wl = wl
        self.q_bits, self.k_bits, self.v_bits = qkv if qkv is not None else synth.make_qkv(wl)
        self.q, self.k, self.v = (to_dev(x) for x in (self.q_bits, self.k_bits, self.v_bits))
        self.shape = api.shape_of(wl)
        self.params = api.params_of(wl, block, block, temporal_permute, two_mask, key_first, t2d)
        self.mem = Guarded()
        self.ws = self.mem.alloc((api.rf_workspace_bytes(self.shape, self.params),), torch.uint8, name="ws")
        self.sched = api.Schedule(self.shape, self.params, "cuda", with_bitmap=True)
        s = self.sched
        s.count = self.mem.alloc(tuple(s.count.shape), torch.int32, 0, "count")
        s.kv_tile = self.mem.alloc(tuple(s.kv_tile.shape), torch.int32, 0, "kv_tile")
        s.kv_len = self.mem.alloc(tuple(s.kv_len.shape), torch.int32, 0, "kv_len")
        s.bitmap = self.mem.alloc(tuple(s.bitmap.shape), torch.int32, 0, "bitmap")
        s.c = api.rf_schedule(s.count.data_ptr(), s.kv_tile.data_ptr(), s.bitmap.data_ptr(), s.kv_len.data_ptr(), s.nQ, s.nKmax)
        self.status = self.mem.alloc((1,), torch.int32, 0, "status")
        self.head_class = self.mem.alloc((wl.B, wl.H), torch.int32, 0, "head_class")
        self.recall = self.mem.alloc((wl.B, wl.H, 3), torch.float32, 0, "recall")
        self._out = None

    def outputs(self):
        """NaN-filled o and lse between guards (allocated once per Run, refilled per call)."""
        wl = self.wl
        if self._out is None:
            self._out = (self.mem.alloc((wl.B, wl.H, wl.N, wl.D), torch.bfloat16, name="o"),
                         self.mem.alloc((wl.B, wl.H, wl.N), torch.float32, name="lse"))
        o, lse = self._out
        o.fill_(float("nan"))
        lse.fill_(float("nan"))
        return o, lse

    def arm(self):
        api.rf_arm_classify(self.shape, self.params, self.q, self.k, self.head_class, self.recall, self.ws, self.status)
        torch.cuda.synchronize()
        self.mem.check("rf_arm_classify")
        return self.head_class.cpu().numpy(), self.recall.cpu().numpy()

    # dynamic bandwidth (RainFusion+): the per-head window array lives between guards as well
    def arm_plus(self, bandwidths):
        wl = self.wl
        self.head_window = self.mem.alloc((wl.B, wl.H), torch.int32, -7, "head_window")
        self.recall_plus = self.mem.alloc((wl.B, wl.H, 2, len(bandwidths)), torch.float32, 0, "recall_plus")
        api.rf_arm_classify_plus(self.shape, self.params, list(bandwidths), self.q, self.k, self.head_class,
                                 self.head_window, self.recall_plus, self.ws, self.status)
        torch.cuda.synchronize()
        self.mem.check("rf_arm_classify_plus")
        return self.head_class.cpu().numpy(), self.head_window.cpu().numpy(), self.recall_plus.cpu().numpy()

    def build_plus(self):
        api.rf_build_block_mask_plus(self.shape, self.params, self.head_class, self.head_window, self.sched, self.status)
        torch.cuda.synchronize()
        self.mem.check("rf_build_block_mask_plus")

    def sparse_plus(self, to_numpy=True):
        o, lse = self.outputs()
        api.rf_sparse_attn_fwd_plus(self.shape, self.params, self.q, self.k, self.v, self.head_class, self.head_window,
                                    self.sched, o, lse, self.ws, self.status)
        torch.cuda.synchronize()
        assert int(self.status.item()) == 0, f"device status {int(self.status.item())}"
        self.mem.check("rf_sparse_attn_fwd_plus")
        if not to_numpy:
            return o, lse
        return o.float().cpu().numpy().astype(np.float64), lse.cpu().numpy().astype(np.float64)

    def force_classes(self, classes):
        self.head_class.copy_(torch.as_tensor(np.asarray(classes, dtype=np.int32).reshape(self.wl.B, self.wl.H)))

    def build(self):
        api.rf_build_block_mask(self.shape, self.params, self.head_class, self.sched, self.status)
        torch.cuda.synchronize()
        self.mem.check("rf_build_block_mask")

    def sparse(self):
        o, lse = self.outputs()
        api.rf_sparse_attn_fwd(self.shape, self.params, self.q, self.k, self.v, self.head_class, self.sched, o, lse,
                               self.ws, self.status)
        torch.cuda.synchronize()
        self.mem.check("rf_sparse_attn_fwd")
        assert int(self.status.item()) == 0, f"device status {int(self.status.item())}"
        return o.float().cpu().numpy().astype(np.float64), lse.cpu().numpy().astype(np.float64)

    def dense(self):
        o, lse = self.outputs()
        api.rf_dense_attn_fwd(self.shape, self.q, self.k, self.v, o, lse, self.status)
        torch.cuda.synchronize()
        self.mem.check("rf_dense_attn_fwd")
        assert int(self.status.item()) == 0, f"device status {int(self.status.item())}"
        return o.float().cpu().numpy().astype(np.float64), lse.cpu().numpy().astype(np.float64)

    def lists(self, b, h):
        cnt = self.sched.count[b, h].cpu().numpy()
        til = self.sched.kv_tile[b, h].cpu().numpy().view(np.uint32)
        return [til[a, :cnt[a]].tolist() for a in range(self.sched.nQ)]


def check_attention(O_gpu, lse_gpu, O_ref, lse_ref, what="", strict=True):
    """strict: the absolute bar as stated, on every element.  Otherwise the max-abs bar of a query ROW grows
    with that row's own largest reference output: a bf16 output in [4, 8) alone rounds by up to 2^-6 = 1.6e-2,
    and the bf16 rounding of P (2^-9 relative) scales with |O| as well.  Rows whose outputs stay within 2 in
    magnitude, which is most rows of every input, keep the stated bar whatever the rest of the tensor holds."""
    err = np.abs(O_gpu - O_ref)
    assert np.isfinite(O_gpu).all(), f"{what}: non-finite output"
    if strict:
        assert err.max() <= O_MAX_ABS, f"{what}: max-abs {err.max():.3e}"
    else:
        row_bar = O_MAX_ABS * np.maximum(1.0, np.abs(O_ref).max(axis=-1) / 2.0)
        excess = err.max(axis=-1) / row_bar
        assert excess.max() <= 1.0, (f"{what}: a row's max-abs error is {excess.max():.2f} x its bar "
                                     f"(error {err.max(axis=-1).flat[excess.argmax()]:.3e}, bar {row_bar.flat[excess.argmax()]:.3e})")
    assert err.mean() <= O_MEAN_ABS, f"{what}: mean-abs {err.mean():.3e}"
    rel = np.linalg.norm(O_gpu - O_ref) / max(np.linalg.norm(O_ref), 1e-30)
    assert rel <= O_REL_L2, f"{what}: rel-L2 {rel:.3e}"
    lerr = np.abs(lse_gpu - lse_ref).max()
    assert lerr <= LSE_ABS, f"{what}: lse {lerr:.3e}"
    return err.max(), err.mean(), rel, lerr


def oracle_lists(wl, cls, block, permute, tiles=None, key_first=False, t2d=None):
    g, pp = geom(wl), pparams(wl, key_first, t2d)
    nQ = -(-g.N // block)
    tiles = range(nQ) if tiles is None else tiles
    return {a: orc.tile_row(cls, g, pp, bool(permute), block, block, a) for a in tiles}
