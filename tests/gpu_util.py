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


def pparams(wl):
    return orc.PatternParams(wl.frame_window, wl.spatial_window, wl.textural_stride)


def to_dev(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def bits_of(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().view(torch.int16).numpy().view(np.uint16)


class Run:
    """One workload resident on the GPU with its schedule and workspace."""

    def __init__(self, wl, qkv=None, block=128, temporal_permute=1, two_mask=0):
        self.wl = wl
        self.q_bits, self.k_bits, self.v_bits = qkv if qkv is not None else synth.make_qkv(wl)
        self.q, self.k, self.v = (to_dev(x) for x in (self.q_bits, self.k_bits, self.v_bits))
        self.shape = api.shape_of(wl)
        self.params = api.params_of(wl, block, block, temporal_permute, two_mask)
        self.ws = api.alloc_workspace(self.shape, self.params, "cuda")
        self.sched = api.Schedule(self.shape, self.params, "cuda", with_bitmap=True)
        self.status = torch.zeros(1, dtype=torch.int32, device="cuda")
        self.head_class = torch.zeros((wl.B, wl.H), dtype=torch.int32, device="cuda")
        self.recall = torch.zeros((wl.B, wl.H, 3), dtype=torch.float32, device="cuda")

    def arm(self):
        api.rf_arm_classify(self.shape, self.params, self.q, self.k, self.head_class, self.recall, self.ws)
        torch.cuda.synchronize()
        return self.head_class.cpu().numpy(), self.recall.cpu().numpy()

    def force_classes(self, classes):
        self.head_class.copy_(torch.as_tensor(np.asarray(classes, dtype=np.int32).reshape(self.wl.B, self.wl.H)))

    def build(self):
        api.rf_build_block_mask(self.shape, self.params, self.head_class, self.sched, self.status)
        torch.cuda.synchronize()

    def sparse(self):
        o = torch.full((self.wl.B, self.wl.H, self.wl.N, self.wl.D), float("nan"), dtype=torch.bfloat16, device="cuda")
        lse = torch.full((self.wl.B, self.wl.H, self.wl.N), float("nan"), dtype=torch.float32, device="cuda")
        api.rf_sparse_attn_fwd(self.shape, self.params, self.q, self.k, self.v, self.head_class, self.sched, o, lse,
                               self.ws, self.status)
        torch.cuda.synchronize()
        assert int(self.status.item()) == 0, f"device status {int(self.status.item())}"
        return o.float().cpu().numpy().astype(np.float64), lse.cpu().numpy().astype(np.float64)

    def dense(self):
        o = torch.full((self.wl.B, self.wl.H, self.wl.N, self.wl.D), float("nan"), dtype=torch.bfloat16, device="cuda")
        lse = torch.full((self.wl.B, self.wl.H, self.wl.N), float("nan"), dtype=torch.float32, device="cuda")
        api.rf_dense_attn_fwd(self.shape, self.q, self.k, self.v, o, lse, self.status)
        torch.cuda.synchronize()
        assert int(self.status.item()) == 0, f"device status {int(self.status.item())}"
        return o.float().cpu().numpy().astype(np.float64), lse.cpu().numpy().astype(np.float64)

    def lists(self, b, h):
        cnt = self.sched.count[b, h].cpu().numpy()
        til = self.sched.kv_tile[b, h].cpu().numpy().view(np.uint32)
        return [til[a, :cnt[a]].tolist() for a in range(self.sched.nQ)]


def check_attention(O_gpu, lse_gpu, O_ref, lse_ref, what="", strict=True):
    """strict: the absolute bar as stated (outputs of magnitude <= ~2).  Otherwise the max-abs bar
    grows with the output magnitude: a bf16 output in [2, 4) alone rounds by up to 2^-7, and the bf16
    rounding of P (2^-9 relative) scales with |O| as well."""
    err = np.abs(O_gpu - O_ref)
    assert np.isfinite(O_gpu).all(), f"{what}: non-finite output"
    bar = O_MAX_ABS if strict else O_MAX_ABS * max(1.0, np.abs(O_ref).max() / 2.0)
    assert err.max() <= bar, f"{what}: max-abs {err.max():.3e}"
    assert err.mean() <= O_MEAN_ABS, f"{what}: mean-abs {err.mean():.3e}"
    rel = np.linalg.norm(O_gpu - O_ref) / max(np.linalg.norm(O_ref), 1e-30)
    assert rel <= O_REL_L2, f"{what}: rel-L2 {rel:.3e}"
    lerr = np.abs(lse_gpu - lse_ref).max()
    assert lerr <= LSE_ABS, f"{what}: lse {lerr:.3e}"
    return err.max(), err.mean(), rel, lerr


def oracle_lists(wl, cls, block, permute, tiles=None):
    g, pp = geom(wl), pparams(wl)
    nQ = -(-g.N // block)
    tiles = range(nQ) if tiles is None else tiles
    return {a: orc.tile_row(cls, g, pp, bool(permute), block, block, a) for a in tiles}
