"""Seeded synthetic Q/K/V for video-DiT-shaped 3D attention layers.

This module only draws random numbers and rounds them to bf16. It contains none
of the method's arithmetic (no masks, no softmax, no recall), so both the CPU
oracle's tests and the CUDA path's tests may take their inputs from it.

Tensors are returned as numpy uint16 arrays holding bf16 bit patterns, laid out
[B, H, N, D] with N = T*frame_h*frame_w + L_text (video tokens frame-major,
row-major inside a frame, text tokens last).

Each (tensor, b, h) slice has its own seed, so a single head of a large
configuration can be regenerated without drawing the others.

Planted structure (added to Q and K of video tokens only; V and text tokens
stay iid N(0,1)):
  "frame"    one vector per latent frame, shared by every token of the frame
  "position" one vector per in-frame position, shared across frames
  "lowrank"  a rank-4 component W g_i (queries) / W h_j (keys)
  "none"     nothing planted
Each planted component has per-coordinate standard deviation `amp`.
"""
from __future__ import annotations

import dataclasses
from typing import Dict, List, Sequence, Tuple

import numpy as np

BASE_SEED = 250521036
TENSOR_Q, TENSOR_K, TENSOR_V = 0, 1, 2


@dataclasses.dataclass(frozen=True)
class Workload:
    """Shapes and pattern parameters of one attention layer call."""
    name: str
    B: int
    H: int
    D: int
    T: int
    frame_h: int
    frame_w: int
    L_text: int
    frame_window: int
    spatial_window: int
    textural_stride: int
    sample_mode: int          # 0: first frame for temporal recall, stride sample for spatial; 1: stride sample for both
    sample_stride: int
    alpha: float
    amp: float
    config_id: int

    @property
    def S(self) -> int:
        return self.frame_h * self.frame_w

    @property
    def Nv(self) -> int:
        return self.T * self.S

    @property
    def N(self) -> int:
        return self.Nv + self.L_text

    def head_kinds(self) -> List[str]:
        """First third frame-local, second third position-local, last third low-rank."""
        third = self.H // 3
        kinds = []
        for h in range(self.H):
            if h < third:
                kinds.append("frame")
            elif h < 2 * third:
                kinds.append("position")
            else:
                kinds.append("lowrank")
        return kinds


def _wl(name, cid, B, H, D, T, fh, fw, L, wf=None, ws=None, tau=2, mode=0, omega=1, alpha=0.9, amp=1.5):
    S = fh * fw
    return Workload(name=name, B=B, H=H, D=D, T=T, frame_h=fh, frame_w=fw, L_text=L,
                    frame_window=(T // 4 if wf is None else wf),
                    spatial_window=(S // 4 if ws is None else ws),
                    textural_stride=tau, sample_mode=mode, sample_stride=omega,
                    alpha=alpha, amp=amp, config_id=cid)


WORKLOADS: Dict[str, Workload] = {
    # tiny case: frame window 1, spatial window 2, stride-4 global sample (64 rows)
    "tiny": _wl("tiny", 1, 1, 3, 64, 4, 8, 8, 16, wf=1, ws=2, tau=2, mode=1, omega=4, amp=1.5),
    # CogVideoX-5B-shaped layer; planted std 0.5 as stated for this configuration
    "cogvideox": _wl("cogvideox", 2, 1, 48, 64, 13, 30, 45, 226, mode=0, omega=15, amp=0.5),
    # same shape, planted amplitude strong enough that all three branches fire
    "cogvideox_cal": _wl("cogvideox_cal", 2, 1, 48, 64, 13, 30, 45, 226, mode=0, omega=15, amp=2.0),
    # parameter-sensitivity settings on the CogVideoX-shaped layer: bandwidth 0.18 / 0.13, stride 3 / 4
    "cogvideox_2p5x": _wl("cogvideox_2p5x", 2, 1, 48, 64, 13, 30, 45, 226, wf=int(0.18 * 13), ws=int(0.18 * 1350), tau=3,
                          mode=0, omega=15, amp=2.0),
    "cogvideox_3p0x": _wl("cogvideox_3p0x", 2, 1, 48, 64, 13, 30, 45, 226, wf=int(0.13 * 13), ws=int(0.13 * 1350), tau=4,
                          mode=0, omega=15, amp=2.0),
    # OpenSoraPlan-1.2-shaped layer; 1 % of tokens sampled at equal intervals
    "opensoraplan": _wl("opensoraplan", 3, 1, 24, 96, 24, 45, 80, 300, mode=1, omega=100, amp=1.5),
    # HunyuanVideo-720p-shaped layer
    "hunyuan720p": _wl("hunyuan720p", 4, 1, 24, 128, 33, 45, 80, 256, mode=0, omega=36, amp=1.5),
    # pattern-mix / shape sweep at D=128
    "sweep_8x1024": _wl("sweep_8x1024", 5, 1, 24, 128, 8, 32, 32, 256, mode=0, omega=8, amp=1.5),
    "sweep_16x2040": _wl("sweep_16x2040", 5, 1, 24, 128, 16, 34, 60, 256, mode=0, omega=17, amp=1.5),
    "sweep_33x3600": _wl("sweep_33x3600", 5, 1, 24, 128, 33, 45, 80, 256, mode=0, omega=36, amp=1.5),
}


def small_workload(name="small", H=3, D=64, T=5, fh=6, fw=7, L=3, **kw) -> Workload:
    """Free-form small workload for tests (config id 0)."""
    return _wl(name, 0, kw.pop("B", 1), H, D, T, fh, fw, L, **kw)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even fp32 -> bf16, returned as uint16 bit patterns."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    rounded = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to fp32."""
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def _rng(wl: Workload, tensor_id: int, b: int, h: int) -> np.random.Generator:
    ss = np.random.SeedSequence([BASE_SEED, 1000 * wl.config_id, tensor_id, b, h,
                                 wl.T, wl.frame_h, wl.frame_w, wl.L_text, wl.D])
    return np.random.Generator(np.random.PCG64(ss))


def _planted(wl: Workload, kind: str, b: int, h: int) -> Tuple[np.ndarray, np.ndarray]:
    """Planted additive components for the video tokens of Q and K: two [Nv, D] fp32 arrays."""
    T, S, D, a = wl.T, wl.S, wl.D, wl.amp
    r = _rng(wl, 7, b, h)
    if kind == "frame":
        u = r.standard_normal((T, 1, D), dtype=np.float32) * np.float32(a)
        comp = np.broadcast_to(u, (T, S, D)).reshape(T * S, D)
        return comp, comp
    if kind == "position":
        v = r.standard_normal((1, S, D), dtype=np.float32) * np.float32(a)
        comp = np.broadcast_to(v, (T, S, D)).reshape(T * S, D)
        return comp, comp
    if kind == "lowrank":
        rank = 4
        W = r.standard_normal((rank, D), dtype=np.float32) * np.float32(a / np.sqrt(rank))
        g = r.standard_normal((T * S, rank), dtype=np.float32)
        hh = r.standard_normal((T * S, rank), dtype=np.float32)
        return g @ W, hh @ W
    if kind == "none":
        z = np.zeros((1, D), dtype=np.float32)
        return z, z
    raise ValueError(kind)


def make_head(wl: Workload, b: int, h: int, kind: str | None = None):
    """bf16 bit patterns (q, k, v), each [N, D] uint16, for one (b, h)."""
    if kind is None:
        kind = wl.head_kinds()[h]
    out = []
    pq, pk = _planted(wl, kind, b, h)
    for tid, comp in ((TENSOR_Q, pq), (TENSOR_K, pk), (TENSOR_V, None)):
        x = _rng(wl, tid, b, h).standard_normal((wl.N, wl.D), dtype=np.float32)
        if comp is not None and kind != "none":
            x[: wl.Nv] += comp
        out.append(f32_to_bf16_bits(x))
    return tuple(out)


def make_qkv(wl: Workload, kinds: Sequence[str] | None = None):
    """bf16 bit patterns (q, k, v), each [B, H, N, D] uint16."""
    if kinds is None:
        kinds = wl.head_kinds()
    q = np.empty((wl.B, wl.H, wl.N, wl.D), dtype=np.uint16)
    k = np.empty_like(q)
    v = np.empty_like(q)

    def fill(bh):
        b, h = divmod(bh, wl.H)
        q[b, h], k[b, h], v[b, h] = make_head(wl, b, h, kinds[h])

    if wl.B * wl.H * wl.N * wl.D > (1 << 24):
        from concurrent.futures import ThreadPoolExecutor
        import os
        with ThreadPoolExecutor(max_workers=min(16, os.cpu_count() or 1)) as ex:
            list(ex.map(fill, range(wl.B * wl.H)))
    else:
        for bh in range(wl.B * wl.H):
            fill(bh)
    return q, k, v


def sample_rows(wl: Workload, count: int, seed: int = 0, block: int = 128) -> np.ndarray:
    """A sorted set of query rows for spot checks at large sizes: first/last rows of
    some frames, rows next to tile boundaries, the last video row, several text rows,
    and seeded random rows up to `count`."""
    N, Nv, S = wl.N, wl.Nv, wl.S
    rows = {0, N - 1, Nv - 1}
    if wl.L_text > 0:
        rows.update(range(Nv, min(N, Nv + 8)))
    for f in (0, 1, wl.T // 2, wl.T - 1):
        if 0 <= f < wl.T:
            rows.update((f * S, f * S + S - 1))
    for t in (1, (N // block) // 2, N // block):
        for r in (t * block - 1, t * block):
            if 0 <= r < N:
                rows.add(r)
    r = np.random.Generator(np.random.PCG64([BASE_SEED, 99, seed, wl.config_id]))
    while len(rows) < min(count, N):
        rows.add(int(r.integers(0, N)))
    rows = sorted(rows)[: max(count, 1)] if len(rows) > count else sorted(rows)
    return np.asarray(rows, dtype=np.int64)
