"""Seeded random shapes and parameters: the whole path against the oracle on small problems.

Every case draws the head dimension, the latent shape, the text length, the windows, the checkerboard
stride, the sampling mode and stride, the Temporal permutation and the per-head classes from a fixed seed,
then checks ARM (recalls, classes away from ties), the tile lists (bit-exact) and the attention output and
log-sum-exp of every head against the oracle, through the C ABI."""
import numpy as np
import pytest

from oracle import rainfusion_oracle as orc
from paper_2505_21036_b200 import synth

import gpu_util as gu

pytestmark = pytest.mark.gpu


def draw_case(seed, large=False):
    rng = np.random.default_rng((77000 if large else 9000) + seed)
    D = int(rng.choice([64, 96, 128]))
    T = int(rng.integers(1, 14 if large else 8))
    hi = 21 if large else 13
    fh, fw = int(rng.integers(1, hi)), int(rng.integers(1, hi))
    S = fh * fw
    L = int(rng.choice([0, 1, 17, 130]))
    if T * S + L < 2:
        L = 17
    kw = dict(B=1 if large else int(rng.choice([1, 2])), H=4, D=D, T=T, fh=fh, fw=fw, L=L,
              wf=int(rng.integers(0, T + 1)), ws=int(rng.integers(0, S + 1)), tau=int(rng.integers(1, 5)),
              mode=int(rng.integers(0, 2)), omega=int(rng.integers(1, max(2, S // 2 + 1))),
              amp=float(rng.choice([0.0, 0.8, 1.5, 2.5])))
    wl = synth.small_workload(f"fuzz{seed}", **kw)
    permute = int(rng.integers(0, 2))
    two_mask = int(rng.integers(0, 2))
    classes = rng.integers(0, 4, size=(wl.B, wl.H)).astype(np.int32)
    return wl, permute, two_mask, classes


@pytest.mark.parametrize("seed", range(int(__import__("os").environ.get("RF_FUZZ_FROM", "0")), int(__import__("os").environ.get("RF_FUZZ_TO", "32"))))
def test_random_case(seed):
    check_case(seed, *draw_case(seed))


@pytest.mark.parametrize("seed", range(int(__import__("os").environ.get("RF_FUZZ_LARGE_FROM", "0")),
                                       int(__import__("os").environ.get("RF_FUZZ_LARGE_TO", "8"))))
def test_random_case_up_to_forty_tiles(seed):
    check_case(seed, *draw_case(seed, large=True))


@pytest.mark.parametrize("seed", range(int(__import__("os").environ.get("RF_FUZZ_OPT_FROM", "0")),
                                       int(__import__("os").environ.get("RF_FUZZ_OPT_TO", "16"))))
def test_random_case_pattern_options(seed):
    """The optional readings of Sec. 3.2 on drawn shapes: the first frame as a key frame of Spatial heads, a 2-D
    in-frame window for Temporal heads, or both."""
    wl, permute, two_mask, classes = draw_case(5000 + seed, large=seed % 4 == 3)
    rng = np.random.default_rng(31000 + seed)
    which = int(rng.integers(1, 4))
    t2d = (int(rng.integers(0, wl.frame_h + 2)), int(rng.integers(0, wl.frame_w + 2))) if which & 2 else None
    check_case(seed, wl, permute, two_mask, classes, key_first=which & 1, t2d=t2d)


def check_case(seed, wl, permute, two_mask, classes, key_first=0, t2d=None):
    g, pp = gu.geom(wl), gu.pparams(wl, key_first, t2d)
    run = gu.Run(wl, temporal_permute=permute, two_mask=two_mask, key_first=key_first, t2d=t2d)
    # ARM
    cls_gpu, rec_gpu = run.arm()
    cls_ref, rec_ref, margin = orc.arm_classify(run.q_bits, run.k_bits, g, pp, wl.sample_mode, wl.sample_stride, wl.alpha,
                                                two_mask=bool(two_mask))
    assert np.abs(rec_gpu - rec_ref).max() <= gu.RECALL_ABS, (seed, np.abs(rec_gpu - rec_ref).max())
    decided = margin > gu.TIE_MARGIN
    assert np.array_equal(cls_gpu[decided], cls_ref[decided]), seed
    # schedule and attention on drawn classes (all four values, whatever ARM said)
    run.force_classes(classes)
    run.build()
    O, lse = run.sparse()
    for b in range(wl.B):
        for h in range(wl.H):
            cls = int(classes[b, h])
            ref = gu.oracle_lists(wl, cls, 128, permute, key_first=key_first, t2d=t2d)
            assert run.lists(b, h) == [ref[a] for a in range(run.sched.nQ)], (seed, b, h, cls)
            assert int(run.sched.kv_len[b, h]) == orc.kv_len(cls, g, pp)
            Or, lr = orc.masked_attention(run.q_bits[b, h], run.k_bits[b, h], run.v_bits[b, h], cls, g, pp)
            gu.check_attention(O[b, h], lse[b, h], Or, lr, f"fuzz {seed} b{b} h{h} class {cls}", strict=False)
    # the schedule builder alone at a smaller tile (the attention kernel itself only takes 128 x 128)
    block = (16, 32, 64)[seed % 3]
    small = gu.Run(wl, block=block, temporal_permute=permute, key_first=key_first, t2d=t2d)
    small.force_classes(classes)
    small.build()
    for b in range(wl.B):
        for h in range(wl.H):
            ref = gu.oracle_lists(wl, int(classes[b, h]), block, permute, key_first=key_first, t2d=t2d)
            assert small.lists(b, h) == [ref[a] for a in range(small.sched.nQ)], (seed, b, h, block)
    if seed % 4 == 0:
        Od, lsed = run.dense()
        Or, lr = orc.masked_attention(run.q_bits[0, 1], run.k_bits[0, 1], run.v_bits[0, 1], orc.DENSE, g, pp)
        gu.check_attention(Od[0, 1], lsed[0, 1], Or, lr, f"fuzz {seed} dense", strict=False)


@pytest.mark.parametrize("seed", range(int(__import__("os").environ.get("RF_FUZZ_PLUS_FROM", "0")),
                                       int(__import__("os").environ.get("RF_FUZZ_PLUS_TO", "12"))))
def test_random_case_dynamic_bandwidth(seed):
    """The dynamic-bandwidth variant on drawn shapes: candidate lists of one to four bandwidths, the per-head
    window ARM picks, the schedule and the attention that honour it."""
    import torch
    from paper_2505_21036_b200 import api
    wl, permute, two_mask, _ = draw_case(seed)
    rng = np.random.default_rng(555 + seed)
    bws = sorted(set(float(x) for x in rng.choice([0.05, 0.125, 0.2, 0.25, 0.4, 0.5, 0.75, 1.0], size=int(rng.integers(1, 5)))))
    g = gu.geom(wl)
    run = gu.Run(wl, temporal_permute=permute, two_mask=two_mask)
    head_window = run.mem.alloc((wl.B, wl.H), torch.int32, -7, "head_window")
    rec = run.mem.alloc((wl.B, wl.H, 2, len(bws)), torch.float32, 0, "recall_plus")
    api.rf_arm_classify_plus(run.shape, run.params, bws, run.q, run.k, run.head_class, head_window, rec, run.ws, run.status)
    torch.cuda.synchronize()
    run.mem.check("rf_arm_classify_plus")
    cls_gpu, win_gpu, rec_gpu = run.head_class.cpu().numpy(), head_window.cpu().numpy(), rec.cpu().numpy()
    for b in range(wl.B):
        for h in range(wl.H):
            cls, idx, window, Rt, Rs = orc.arm_head_plus(run.q_bits[b, h], run.k_bits[b, h], g, bws, wl.textural_stride,
                                                         wl.sample_mode, wl.sample_stride, wl.alpha, two_mask=bool(two_mask))
            assert np.abs(rec_gpu[b, h, 0] - np.asarray(Rt)).max() <= gu.RECALL_ABS, (seed, b, h)
            assert np.abs(rec_gpu[b, h, 1] - np.asarray(Rs)).max() <= gu.RECALL_ABS, (seed, b, h)
            margin = min([abs(r - wl.alpha) for r in list(Rt) + list(Rs)] + ([abs(Rt[-1] - Rs[-1])] if two_mask else []))
            if margin > gu.TIE_MARGIN:
                assert (int(cls_gpu[b, h]), int(win_gpu[b, h])) == (cls, window), (seed, b, h)
    api.rf_build_block_mask_plus(run.shape, run.params, run.head_class, head_window, run.sched, run.status)
    o, lse = run.outputs()
    api.rf_sparse_attn_fwd_plus(run.shape, run.params, run.q, run.k, run.v, run.head_class, head_window, run.sched, o, lse,
                                run.ws, run.status)
    torch.cuda.synchronize()
    assert int(run.status.item()) == 0
    run.mem.check("rf_build_block_mask_plus / rf_sparse_attn_fwd_plus")
    O, LSE = o.float().cpu().numpy().astype(np.float64), lse.cpu().numpy().astype(np.float64)
    for b in range(wl.B):
        for h in range(wl.H):
            cls, w = int(cls_gpu[b, h]), int(win_gpu[b, h])
            pp = orc.PatternParams(w if cls == orc.SPATIAL else wl.frame_window,
                                   w if cls == orc.TEMPORAL else wl.spatial_window, wl.textural_stride)
            got = run.lists(b, h)
            for a in range(run.sched.nQ):
                assert got[a] == orc.tile_row(cls, g, pp, bool(permute), 128, 128, a), (seed, b, h, a)
            Or, lr = orc.masked_attention(run.q_bits[b, h], run.k_bits[b, h], run.v_bits[b, h], cls, g, pp)
            gu.check_attention(O[b, h], LSE[b, h], Or, lr, f"fuzz+ {seed} b{b} h{h} class {cls} window {w}", strict=False)
