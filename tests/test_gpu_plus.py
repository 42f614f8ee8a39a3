"""GPU parity of the dynamic-bandwidth variant (RainFusion+): ARM picks a window per head, the tile
schedule and the attention kernel honour it; all against the oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import rainfusion_oracle as orc
from paper_2505_21036_b200 import api, synth

import gpu_util as gu

pytestmark = pytest.mark.gpu

BWS = [0.125, 0.25, 0.5]


def planted_groups(wl, h, frames_per_group=0, positions_per_group=0, amp=2.0):
    """iid head plus one shared vector per group of consecutive frames (or of in-frame positions)."""
    q, k, v = synth.make_head(wl, 0, h, kind="none")
    qf, kf = synth.bf16_bits_to_f32(q).copy(), synth.bf16_bits_to_f32(k).copy()
    rng = np.random.default_rng(100 + h)
    tok = np.arange(wl.Nv)
    if frames_per_group:
        grp = (tok // wl.S) // frames_per_group
    else:
        grp = (tok % wl.S) // positions_per_group
    vec = rng.standard_normal((grp.max() + 1, wl.D)).astype(np.float32) * amp
    qf[:wl.Nv] += vec[grp]
    kf[:wl.Nv] += vec[grp]
    return synth.f32_to_bf16_bits(qf), synth.f32_to_bf16_bits(kf), v


@pytest.mark.parametrize("mode", [0, 1])
def test_dynamic_bandwidth_pipeline(mode):
    wl = synth.small_workload("plus", H=6, D=64, T=8, fh=16, fw=16, L=32, tau=2, mode=mode, omega=4, amp=2.0)
    heads = [planted_groups(wl, 0, frames_per_group=1),      # needs only the frame itself: smallest window
             planted_groups(wl, 1, frames_per_group=3),      # needs |df| <= 2: the middle bandwidth
             planted_groups(wl, 2, positions_per_group=16),  # needs |dp| <= 15: smallest Temporal window
             planted_groups(wl, 3, positions_per_group=100), # needs |dp| <= 99: the widest Temporal window
             synth.make_head(wl, 0, 4, kind="lowrank"),      # nothing qualifies: Textural
             synth.make_head(wl, 0, 5, kind="none")]
    q = np.stack([h[0] for h in heads])[None]
    k = np.stack([h[1] for h in heads])[None]
    v = np.stack([h[2] for h in heads])[None]
    run = gu.Run(wl, qkv=(q, k, v))
    g = gu.geom(wl)
    cls_gpu, win_gpu, rec_gpu = (x[0] for x in run.arm_plus(BWS))

    seen = set()
    for h in range(wl.H):
        cls, idx, window, Rt, Rs = orc.arm_head_plus(q[0, h], k[0, h], g, BWS, wl.textural_stride, mode, wl.sample_stride,
                                                     wl.alpha)
        assert np.abs(rec_gpu[h, 0] - np.asarray(Rt)).max() <= gu.RECALL_ABS
        assert np.abs(rec_gpu[h, 1] - np.asarray(Rs)).max() <= gu.RECALL_ABS
        margin = min(abs(r - wl.alpha) for r in list(Rt) + list(Rs))
        if margin > gu.TIE_MARGIN:
            assert (int(cls_gpu[h]), int(win_gpu[h])) == (cls, window), h
        seen.add((cls, idx))
    assert len(seen) >= 4          # the planted heads really exercise several (pattern, bandwidth) outcomes

    # schedule and attention with the per-head windows the GPU chose
    run.build_plus()
    O, LSE = (x[0] for x in run.sparse_plus())
    for h in range(wl.H):
        cls, w = int(cls_gpu[h]), int(win_gpu[h])
        pp = orc.PatternParams(w if cls == orc.SPATIAL else wl.frame_window, w if cls == orc.TEMPORAL else wl.spatial_window,
                               wl.textural_stride)
        got = run.lists(0, h)
        for a in range(run.sched.nQ):
            assert got[a] == orc.tile_row(cls, g, pp, True, 128, 128, a), (h, a)
        Or, lr = orc.masked_attention(q[0, h], k[0, h], v[0, h], cls, g, pp)
        gu.check_attention(O[h], LSE[h], Or, lr, f"plus head {h} class {cls} window {w}", strict=False)


def test_dynamic_bandwidth_with_two_masks():
    """Dynamic bandwidth without the Textural mask: a head no candidate qualifies for takes the mask of larger
    recall at the widest candidate."""
    wl = synth.small_workload("plus2", H=4, D=64, T=8, fh=16, fw=16, L=32, tau=2, mode=0, omega=4, amp=2.0)
    heads = [planted_groups(wl, 0, frames_per_group=1), planted_groups(wl, 2, positions_per_group=16),
             synth.make_head(wl, 0, 4, kind="lowrank"), synth.make_head(wl, 0, 5, kind="none")]
    q, k, v = (np.stack([h[i] for h in heads])[None] for i in range(3))
    run = gu.Run(wl, qkv=(q, k, v), two_mask=1)
    cls_gpu, win_gpu, _ = (x[0] for x in run.arm_plus(BWS))
    g = gu.geom(wl)
    fell_back = 0
    for h in range(wl.H):
        cls, idx, window, Rt, Rs = orc.arm_head_plus(q[0, h], k[0, h], g, BWS, wl.textural_stride, 0, wl.sample_stride,
                                                     wl.alpha, two_mask=True)
        assert cls in (orc.SPATIAL, orc.TEMPORAL) and window >= 0
        margin = min([abs(r - wl.alpha) for r in list(Rt) + list(Rs)] + [abs(Rt[-1] - Rs[-1])])
        if margin > gu.TIE_MARGIN:
            assert (int(cls_gpu[h]), int(win_gpu[h])) == (cls, window), h
        fell_back += max(max(Rt), max(Rs)) < wl.alpha
    assert fell_back >= 1


def test_plus_entry_points_with_null_windows_equal_the_plain_ones():
    wl = synth.WORKLOADS["tiny"]
    run = gu.Run(wl)
    run.force_classes([0, 1, 2])
    run.build()
    ref = [run.lists(0, h) for h in range(wl.H)]
    api.rf_build_block_mask_plus(run.shape, run.params, run.head_class, None, run.sched, run.status)
    torch.cuda.synchronize()
    assert [run.lists(0, h) for h in range(wl.H)] == ref


def test_plus_rejects_bad_bandwidth_lists():
    wl = synth.WORKLOADS["tiny"]
    run = gu.Run(wl)
    hw = torch.zeros((1, 3), dtype=torch.int32, device="cuda")
    for bad in ([0.5, 0.25], [0.0, 0.5], [0.1, 0.2, 0.3, 0.4, 0.5], [1.5]):
        with pytest.raises(api.RainFusionError):
            api.rf_arm_classify_plus(run.shape, run.params, bad, run.q, run.k, run.head_class, hw, None, run.ws)
