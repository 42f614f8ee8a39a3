"""GPU parity: the CUDA path through the C ABI against the CPU oracle, element by element."""
import numpy as np
import pytest
import torch

from oracle import rainfusion_oracle as orc
from paper_2505_21036_b200 import api, synth

import gpu_util as gu

pytestmark = pytest.mark.gpu

S_, T_, X_, D_ = orc.SPATIAL, orc.TEMPORAL, orc.TEXTURAL, orc.DENSE


def mid_workload(D=64, H=4, **kw):
    # 6 frames of 12x11 tokens + 37 text tokens = 829 tokens: 7 tiles of 128 with a ragged tail,
    # frame length 132 cuts every tile boundary
    return synth.small_workload("mid", H=H, D=D, T=6, fh=12, fw=11, L=37, wf=1, ws=20, tau=2, mode=0, omega=6, **kw)


# ------------------------------------------------------------------ block masks / tile lists

@pytest.mark.parametrize("block", [16, 32, 64, 128])
@pytest.mark.parametrize("permute", [0, 1])
def test_tile_lists_tiny_bit_exact(block, permute):
    wl = synth.WORKLOADS["tiny"]
    for classes in ([S_, T_, X_], [D_, X_, T_]):
        run = gu.Run(wl, block=block, temporal_permute=permute)
        run.force_classes(classes)
        run.build()
        assert int(run.status.item()) == 0
        for h, cls in enumerate(classes):
            ref = gu.oracle_lists(wl, cls, block, permute)
            got = run.lists(0, h)
            assert got == [ref[a] for a in range(run.sched.nQ)], (block, permute, cls)
            assert int(run.sched.kv_len[0, h]) == orc.kv_len(cls, gu.geom(wl), gu.pparams(wl))


@pytest.mark.parametrize("block", [16, 64, 128])
@pytest.mark.parametrize("permute", [0, 1])
def test_tile_lists_mid_bit_exact_and_bitmap(block, permute):
    wl = mid_workload()
    run = gu.Run(wl, block=block, temporal_permute=permute)
    classes = [S_, T_, X_, D_]
    run.force_classes(classes)
    run.build()
    bitmap = run.sched.bitmap.cpu().numpy().view(np.uint32)
    for h, cls in enumerate(classes):
        ref = gu.oracle_lists(wl, cls, block, permute)
        got = run.lists(0, h)
        assert got == [ref[a] for a in range(run.sched.nQ)], (block, permute, cls)
        for a in range(run.sched.nQ):
            listed = sorted(e & 0x7FFFFFFF for e in ref[a])
            bits = [b for b in range(run.sched.nKmax) if (bitmap[h, a, b // 32] >> (b % 32)) & 1]
            assert bits == listed


def test_invalid_class_is_reported_not_trapped():
    wl = synth.WORKLOADS["tiny"]
    run = gu.Run(wl)
    run.force_classes([0, 7, 2])
    run.build()
    assert int(run.status.item()) == 1        # RF_ERR_INVALID_ARG, kernel finished normally
    assert run.lists(0, 1) == run.lists(0, 1)


# ------------------------------------------------------------------ ARM

def check_arm(wl, run=None):
    run = run or gu.Run(wl)
    cls_gpu, rec_gpu = run.arm()
    cls_ref, rec_ref, margin = orc.arm_classify(run.q_bits, run.k_bits, gu.geom(wl), gu.pparams(wl),
                                                wl.sample_mode, wl.sample_stride, wl.alpha)
    assert np.abs(rec_gpu - rec_ref).max() <= gu.RECALL_ABS, np.abs(rec_gpu - rec_ref).max()
    decided = margin > gu.TIE_MARGIN
    assert np.array_equal(cls_gpu[decided], cls_ref[decided])
    return cls_gpu, cls_ref, int((~decided).sum())


def test_arm_tiny():
    cls_gpu, cls_ref, ties = check_arm(synth.WORKLOADS["tiny"])
    assert cls_ref[0].tolist() == [S_, T_, X_] and ties == 0


@pytest.mark.parametrize("D", [64, 96, 128])
@pytest.mark.parametrize("mode", [0, 1])
def test_arm_mid(D, mode):
    wl = synth.small_workload("arm_mid", H=6, D=D, T=6, fh=12, fw=11, L=37, wf=1, ws=20, tau=3, mode=mode, omega=6,
                              amp=1.5)
    check_arm(wl)


@pytest.mark.parametrize("mode", [0, 1])
def test_arm_two_mask_ablation(mode):
    """Only the Spatial and Temporal masks (Table 2, rows without Te): weakly planted heads reach alpha with
    neither and must take the mask of larger recall; strongly planted ones decide as in Algorithm 1."""
    for amp in (0.5, 1.5):
        wl = synth.small_workload("two_mask", H=6, D=64, T=6, fh=12, fw=11, L=37, wf=1, ws=20, tau=2, mode=mode, omega=6,
                                  amp=amp)
        run = gu.Run(wl, two_mask=1)
        cls_gpu, rec_gpu = run.arm()
        cls_ref, rec_ref, margin = orc.arm_classify(run.q_bits, run.k_bits, gu.geom(wl), gu.pparams(wl), wl.sample_mode,
                                                    wl.sample_stride, wl.alpha, two_mask=True)
        assert np.abs(rec_gpu - rec_ref).max() <= gu.RECALL_ABS
        assert not (cls_gpu == X_).any() and not (cls_ref == X_).any()
        decided = margin > gu.TIE_MARGIN
        assert decided.sum() >= 4
        assert np.array_equal(cls_gpu[decided], cls_ref[decided])
        three = orc.arm_classify(run.q_bits, run.k_bits, gu.geom(wl), gu.pparams(wl), wl.sample_mode, wl.sample_stride,
                                 wl.alpha)[0]
        if amp == 0.5:
            assert (three == X_).any()          # the ablation really changes something here
        # the pipeline runs on whatever the ablation picked
        run.build()
        O, lse = run.sparse()
        for h in (0, 3):
            Or, lr = orc.masked_attention(run.q_bits[0, h], run.k_bits[0, h], run.v_bits[0, h], int(cls_gpu[0, h]),
                                          gu.geom(wl), gu.pparams(wl))
            gu.check_attention(O[0, h], lse[0, h], Or, lr, f"two-mask head {h}", strict=False)


def test_arm_is_deterministic():
    wl = mid_workload()
    run = gu.Run(wl)
    a = run.arm()[1].copy()
    b = run.arm()[1].copy()
    assert np.array_equal(a, b)


# ------------------------------------------------------------------ attention

def oracle_heads(run, classes, rows=None):
    wl = run.wl
    out = []
    for h, cls in enumerate(classes):
        out.append(orc.masked_attention(run.q_bits[0, h], run.k_bits[0, h], run.v_bits[0, h], cls, gu.geom(wl),
                                        gu.pparams(wl), rows=rows))
    return out


def test_dense_tiny():
    wl = synth.WORKLOADS["tiny"]
    run = gu.Run(wl)
    O, lse = run.dense()
    for h, (Or, lr) in enumerate(oracle_heads(run, [D_] * wl.H)):
        gu.check_attention(O[0, h], lse[0, h], Or, lr, f"dense tiny head {h}")


def test_pipeline_tiny():
    """ARM -> block mask -> sparse attention, classes staying on the device."""
    wl = synth.WORKLOADS["tiny"]
    run = gu.Run(wl)
    cls_gpu, _ = run.arm()
    run.build()
    O, lse = run.sparse()
    assert cls_gpu[0].tolist() == [S_, T_, X_]
    for h, (Or, lr) in enumerate(oracle_heads(run, cls_gpu[0].tolist())):
        gu.check_attention(O[0, h], lse[0, h], Or, lr, f"pipeline tiny head {h}")


@pytest.mark.parametrize("D", [64, 96, 128])
@pytest.mark.parametrize("permute", [0, 1])
def test_sparse_mid_all_patterns(D, permute):
    wl = mid_workload(D=D)
    run = gu.Run(wl, temporal_permute=permute)
    classes = [S_, T_, X_, D_]
    run.force_classes(classes)
    run.build()
    O, lse = run.sparse()
    for h, (Or, lr) in enumerate(oracle_heads(run, classes)):
        gu.check_attention(O[0, h], lse[0, h], Or, lr, f"mid D={D} permute={permute} class {classes[h]}", strict=False)


def test_dense_mid_and_batch():
    wl = synth.small_workload("mid_b2", B=2, H=2, D=128, T=3, fh=9, fw=10, L=5)
    run = gu.Run(wl)
    O, lse = run.dense()
    g, pp = gu.geom(wl), gu.pparams(wl)
    for b in range(2):
        for h in range(2):
            Or, lr = orc.masked_attention(run.q_bits[b, h], run.k_bits[b, h], run.v_bits[b, h], D_, g, pp)
            gu.check_attention(O[b, h], lse[b, h], Or, lr, f"dense b={b} h={h}")


def test_permutation_on_off_agree():
    wl = mid_workload(D=128)
    outs = []
    for permute in (0, 1):
        run = gu.Run(wl, temporal_permute=permute)
        run.force_classes([T_] * wl.H)
        run.build()
        outs.append(run.sparse())
    # both are bf16-rounded outputs of magnitude up to ~4: they may differ by one bf16 ulp (2^-6)
    assert np.abs(outs[0][0] - outs[1][0]).max() <= 3.2e-2
    assert np.abs(outs[0][1] - outs[1][1]).max() <= 1e-3


def planted_boundary_inputs(wl, cls, inside: bool):
    """Keys just inside (spotlight) or just outside (poison) every row's kept set get a huge
    matching logit and large values: a wrongly masked element removes an O(1) contribution, a
    leaked one explodes the output."""
    g, pp = gu.geom(wl), gu.pparams(wl)
    q, k, v = synth.make_head(wl, 0, 0, kind="none")
    qf, kf, vf = (synth.bf16_bits_to_f32(x).copy() for x in (q, k, v))
    qf *= 0.1
    kf *= 0.1
    idx = np.arange(g.N)
    M = orc.keep_mask(cls, idx, idx, g, pp)
    target = np.zeros(g.N, dtype=bool)
    for i in range(0, g.Nv, 7):
        row = M[i, :g.Nv]
        edges = np.flatnonzero(row[1:] != row[:-1])
        for e in edges[:4]:
            j = e if row[e] == inside else e + 1
            target[j] = True
    qf[:, 0] = 6.0
    kf[target, 0] = 6.0 * np.sqrt(wl.D)
    vf[target] = 50.0 if not inside else 3.0
    return tuple(synth.f32_to_bf16_bits(x) for x in (qf, kf, vf)), target


@pytest.mark.parametrize("cls", [S_, T_])
@pytest.mark.parametrize("permute", [0, 1])
@pytest.mark.parametrize("inside", [True, False])
def test_boundary_spotlight_and_poison(cls, permute, inside):
    wl = synth.small_workload("edge", H=1, D=64, T=6, fh=12, fw=11, L=37, wf=1, ws=20)
    (q, k, v), target = planted_boundary_inputs(wl, cls, inside)
    run = gu.Run(wl, qkv=(q[None, None], k[None, None], v[None, None]), temporal_permute=permute)
    run.force_classes([cls])
    run.build()
    O, lse = run.sparse()
    Or, lr = orc.masked_attention(q, k, v, cls, gu.geom(wl), gu.pparams(wl))
    assert np.abs(Or).max() > 1.0                       # the planted keys matter for the reference
    # the stated bars (max-abs scaled per row by that row's own magnitude; lse 2e-3): a planted key dominates its
    # rows, so the outputs are the planted values themselves and the measured errors are orders below the bars
    gu.check_attention(O[0, 0], lse[0, 0], Or, lr, f"boundary class {cls} permute {permute} inside {inside}", strict=False)


# ------------------------------------------------------------------ degenerate shapes and parameters

@pytest.mark.parametrize("kw", [
    dict(T=1, fh=9, fw=10, L=5),            # a single frame
    dict(T=5, fh=6, fw=7, L=0),             # no text tokens
    dict(T=3, fh=16, fw=8, L=0),            # N = 384: exactly three tiles, no ragged tail
    dict(T=4, fh=5, fw=5, L=3, wf=0, ws=0), # windows of zero
    dict(T=4, fh=5, fw=5, L=3, wf=9, ws=99),# windows wider than the extents: dense masks
    dict(T=4, fh=5, fw=6, L=2, tau=1),      # stride 1: the checkerboard keeps everything
    dict(T=3, fh=3, fw=5, L=2, tau=4),      # stride not dividing the frame
])
def test_edge_shapes_all_patterns(kw):
    wl = synth.small_workload("edge_shape", H=4, D=64, B=2, **kw)
    for permute in (1, 0):
        run = gu.Run(wl, temporal_permute=permute)
        classes = [S_, T_, X_, D_]
        run.force_classes(classes * wl.B)
        run.build()
        O, lse = run.sparse()
        g, pp = gu.geom(wl), gu.pparams(wl)
        for b in range(wl.B):
            for h, cls in enumerate(classes):
                ref = gu.oracle_lists(wl, cls, 128, permute)
                assert run.lists(b, h) == [ref[a] for a in range(run.sched.nQ)]
                Or, lr = orc.masked_attention(run.q_bits[b, h], run.k_bits[b, h], run.v_bits[b, h], cls, g, pp)
                gu.check_attention(O[b, h], lse[b, h], Or, lr, f"{kw} b={b} class {cls} permute={permute}", strict=False)


def test_arm_edge_shapes():
    for kw in (dict(T=1, fh=9, fw=10, L=5, omega=1), dict(T=5, fh=6, fw=7, L=0, omega=3), dict(T=2, fh=20, fw=20, L=4, omega=7)):
        for mode in (0, 1):
            wl = synth.small_workload("arm_edge", H=3, D=64, B=2, mode=mode, wf=1, ws=5, **kw)
            check_arm(wl)


def test_windows_and_stride_far_past_the_extent():
    """frame_window, spatial_window and textural_stride at INT_MAX: the masks are those of the extent itself
    (everything kept; the diagonal y == x), recalls 1, and nothing in the index arithmetic overflows."""
    big = 2**31 - 1
    for mode in (0, 1):
        wl = synth.small_workload("huge_windows", H=3, D=64, T=5, fh=6, fw=7, L=3, mode=mode, omega=3, wf=big, ws=big, tau=big)
        run = gu.Run(wl)
        cls_gpu, cls_ref, _ = check_arm(wl, run)
        assert cls_gpu.tolist() == [[T_] * 3]
        assert np.abs(run.recall.cpu().numpy()[..., :2] - 1.0).max() <= gu.RECALL_ABS
        run.force_classes([S_, T_, X_])
        run.build()
        for h, cls in enumerate([S_, T_, X_]):
            ref = gu.oracle_lists(wl, cls, 128, 1)
            assert run.lists(0, h) == [ref[a] for a in range(run.sched.nQ)]
        O, lse = run.sparse()
        for h, cls in enumerate([S_, T_, X_]):
            Or, lr = orc.masked_attention(run.q_bits[0, h], run.k_bits[0, h], run.v_bits[0, h], cls, gu.geom(wl), gu.pparams(wl))
            gu.check_attention(O[0, h], lse[0, h], Or, lr, f"huge windows class {cls}")
            if cls != X_:
                Od, ld = orc.masked_attention(run.q_bits[0, h], run.k_bits[0, h], run.v_bits[0, h], D_, gu.geom(wl), gu.pparams(wl))
                assert np.array_equal(Or, Od)


def test_scores_with_large_dynamic_range_do_not_overflow():
    """Logits that jump by far more than the lazy-rescale threshold between tiles, and rows whose first
    tiles are fully masked: the running maximum must be raised (and O rescaled) exactly."""
    wl = synth.small_workload("range", H=2, D=64, T=6, fh=12, fw=11, L=37, wf=1, ws=20)
    q, k, v = synth.make_head(wl, 0, 0, kind="none")
    qf, kf = synth.bf16_bits_to_f32(q).copy(), synth.bf16_bits_to_f32(k).copy()
    qf[:, 0] = 8.0
    kf[:, 0] = np.linspace(-40.0, 40.0, wl.N)          # logits grow steadily along the key axis: every tile raises
    qb, kb = synth.f32_to_bf16_bits(qf), synth.f32_to_bf16_bits(kf)
    run = gu.Run(wl, qkv=(np.stack([qb, qb])[None], np.stack([kb, kb])[None], np.stack([v, v])[None]))
    run.force_classes([D_, S_])
    run.build()
    O, lse = run.sparse()
    for h, cls in enumerate([D_, S_]):
        Or, lr = orc.masked_attention(qb, kb, v, cls, gu.geom(wl), gu.pparams(wl))
        gu.check_attention(O[0, h], lse[0, h], Or, lr, f"range class {cls}", strict=False)


def test_bounded_wait_runs_out_cleanly_and_the_context_stays_usable():
    """Failure detection without a fault: a wait on a barrier nobody arrives at gives up after its limit,
    reports RF_ERR_TIMEOUT, later waits of the CTA return at once, the kernel exits, and the next real
    call on the same context works."""
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ret = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    api.rf_selftest_wait_timeout(status, 20, ret)
    t1.record()
    torch.cuda.synchronize()
    assert int(status.item()) == 5            # RF_ERR_TIMEOUT
    assert int(ret.item()) == 4               # neither wait succeeded; abort flag set
    assert 15.0 <= t0.elapsed_time(t1) <= 500.0
    test_dense_tiny()                         # the context is intact


def test_arm_failure_is_reported_and_poisons_the_classes():
    """ARM's reporting of a wait that ran out, exercised without making any wait run out: the self-test runs
    rf_arm_classify's launch sequence with the score kernel's failure flag set in place of the kernel.  The
    decision kernel must then write class -1 for every head and pass RF_ERR_TIMEOUT on; the tile builder and the
    attention kernel, handed those classes, report them through their own status; a normal call afterwards
    clears the flag and classifies as usual."""
    wl = synth.WORKLOADS["tiny"]
    run = gu.Run(wl)
    cls_ok, _ = run.arm()
    assert int(run.status.item()) == 0 and (cls_ok >= 0).all()
    api.rf_selftest_arm_abandoned(run.shape, run.params, run.q, run.k, run.head_class, run.ws, run.status)
    torch.cuda.synchronize()
    assert int(run.status.item()) == 5                         # RF_ERR_TIMEOUT
    assert run.head_class.cpu().numpy().tolist() == [[-1] * wl.H]
    # a caller that gave ARM no status pointer still hears about it from the next stage
    api.rf_selftest_arm_abandoned(run.shape, run.params, run.q, run.k, run.head_class, run.ws, None)
    later = torch.zeros(1, dtype=torch.int32, device="cuda")
    api.rf_build_block_mask(run.shape, run.params, run.head_class, run.sched, later)
    torch.cuda.synchronize()
    assert int(later.item()) == 1                              # RF_ERR_INVALID_ARG: class outside 0..3
    later.zero_()
    o = torch.empty_like(run.q)
    api.rf_sparse_attn_fwd(run.shape, run.params, run.q, run.k, run.v, run.head_class, run.sched, o, None, run.ws, later)
    torch.cuda.synchronize()
    assert int(later.item()) == 1
    # the flag is per call: the next real call classifies normally
    run.status.zero_()
    cls_again, _ = run.arm()
    assert int(run.status.item()) == 0 and np.array_equal(cls_again, cls_ok)


@pytest.mark.parametrize("D", [64, 96, 128])
def test_attention_is_bit_reproducible(D):
    """Same inputs, same schedule: every output bit must repeat (no races between the warp roles, no
    order-dependent accumulation), for the sparse and the dense entry points, across many launches."""
    wl = mid_workload(D=D)
    run = gu.Run(wl)
    run.force_classes([S_, T_, X_, D_])
    run.build()
    outs = []
    for _ in range(4):
        o = torch.empty((wl.B, wl.H, wl.N, wl.D), dtype=torch.bfloat16, device="cuda")
        lse = torch.empty((wl.B, wl.H, wl.N), dtype=torch.float32, device="cuda")
        api.rf_sparse_attn_fwd(run.shape, run.params, run.q, run.k, run.v, run.head_class, run.sched, o, lse, run.ws,
                               run.status)
        od = torch.empty_like(o)
        api.rf_dense_attn_fwd(run.shape, run.q, run.k, run.v, od, None, run.status)
        outs.append((o, lse, od))
    torch.cuda.synchronize()
    assert int(run.status.item()) == 0
    for o, lse, od in outs[1:]:
        assert torch.equal(o.view(torch.int16), outs[0][0].view(torch.int16))
        assert torch.equal(lse.view(torch.int32), outs[0][1].view(torch.int32))
        assert torch.equal(od.view(torch.int16), outs[0][2].view(torch.int16))


@pytest.mark.parametrize("D", [64, 128])
def test_reorder_then_attention_equals_the_fused_call(D):
    """rf_reorder_tokens + rf_sparse_attn_reordered launch the same two kernels as rf_sparse_attn_fwd."""
    wl = mid_workload(D=D)
    run = gu.Run(wl)
    run.force_classes([S_, T_, X_, D_])
    run.build()

    def outputs():
        o = torch.full((wl.B, wl.H, wl.N, wl.D), float("nan"), dtype=torch.bfloat16, device="cuda")
        lse = torch.full((wl.B, wl.H, wl.N), float("nan"), dtype=torch.float32, device="cuda")
        return o, lse
    o1, l1 = outputs()
    api.rf_sparse_attn_fwd(run.shape, run.params, run.q, run.k, run.v, run.head_class, run.sched, o1, l1, run.ws, run.status)
    run.ws.zero_()
    o2, l2 = outputs()
    api.rf_reorder_tokens(run.shape, run.params, run.q, run.k, run.v, run.head_class, run.ws)
    for _ in range(2):   # one reordering serves several attention calls
        api.rf_sparse_attn_reordered(run.shape, run.params, run.q, run.k, run.v, run.head_class, None, run.sched, o2, l2,
                                     run.ws, run.status)
    torch.cuda.synchronize()
    assert int(run.status.item()) == 0
    assert torch.equal(o1.view(torch.int16), o2.view(torch.int16))
    assert torch.equal(l1.view(torch.int32), l2.view(torch.int32))


@pytest.mark.parametrize("D", [64, 96, 128])
def test_row_maximum_growing_in_late_tiles(D):
    """The running maximum is only raised (and O rescaled) when a tile's maximum exceeds it by a wide margin.
    Here it does, repeatedly and at different tiles for neighbouring rows: even rows meet keys whose logit
    steps up by ~30 nats in tiles 2 and 4, odd rows in tiles 1, 3 and 5; every earlier contribution must
    then be scaled down by e^-30 in O and in the row sum alike."""
    wl = mid_workload(D=D, H=2)
    q, k, v = synth.make_head(wl, 0, 0, kind="none")
    qf, kf, vf = (synth.bf16_bits_to_f32(x).copy() for x in (q, k, v))
    qf *= 0.25
    kf *= 0.25
    N = wl.N
    step = 30.0 * np.sqrt(D) / 8.0            # logit = 8 * level * step / sqrt(D) = 30 * level nats
    qf[:, 0] = 0.0
    qf[:, 1] = 0.0
    qf[0::2, 0] = 8.0
    qf[1::2, 1] = 8.0
    kf[:, 0] = 0.0
    kf[:, 1] = 0.0
    rng = np.random.default_rng(11)
    for level, t in enumerate((2, 4), start=1):           # feature 0: even rows
        idx = t * 128 + rng.choice(128, size=5, replace=False)
        kf[idx[idx < N], 0] = level * step
    for level, t in enumerate((1, 3, 5), start=1):        # feature 1: odd rows
        idx = t * 128 + rng.choice(128, size=5, replace=False)
        kf[idx[idx < N], 1] = level * step
    bits = tuple(synth.f32_to_bf16_bits(x) for x in (qf, kf, vf))
    stack = tuple(np.stack([x, x])[None] for x in bits)
    run = gu.Run(wl, qkv=stack)
    run.force_classes([D_, X_])
    run.build()
    g, pp = gu.geom(wl), gu.pparams(wl)
    O, lse = run.sparse()
    Od, lsed = run.dense()
    ref_d = orc.masked_attention(*bits, D_, g, pp)
    ref_x = orc.masked_attention(*bits, X_, g, pp)
    assert ref_d[1].max() > 80.0                       # the staircase really is there
    gu.check_attention(O[0, 0], lse[0, 0], *ref_d, "staircase sparse/dense-class", strict=False)
    gu.check_attention(O[0, 1], lse[0, 1], *ref_x, "staircase textural", strict=False)
    gu.check_attention(Od[0, 1], lsed[0, 1], *ref_d, "staircase dense entry", strict=False)


# ------------------------------------------------------------------ Spatial heads with the first frame as key frame

@pytest.mark.parametrize("mode", [0, 1])
def test_first_frame_as_key_frame(mode):
    """Sec. 3.2 lets a Spatial head attend adjacent or key frames: with spatial_key_first_frame every query also keeps
    the keys of frame 0.  ARM's Spatial recall, the tile lists at several tile sizes and the attention output against the
    oracle; the other patterns must not change."""
    for kw in (dict(T=6, fh=12, fw=11, L=37, wf=1, ws=20, omega=6), dict(T=9, fh=5, fw=8, L=0, wf=0, ws=3, omega=7),
               dict(T=4, fh=20, fw=20, L=9, wf=2, ws=50, omega=3)):
        wl = synth.small_workload("key_first", H=4, D=64, mode=mode, amp=1.5, **kw)
        g, pp = gu.geom(wl), gu.pparams(wl, True)
        run = gu.Run(wl, key_first=1)
        cls_gpu, rec_gpu = run.arm()
        cls_ref, rec_ref, margin = orc.arm_classify(run.q_bits, run.k_bits, g, pp, wl.sample_mode, wl.sample_stride, wl.alpha)
        assert np.abs(rec_gpu - rec_ref).max() <= gu.RECALL_ABS, np.abs(rec_gpu - rec_ref).max()
        decided = margin > gu.TIE_MARGIN
        assert np.array_equal(cls_gpu[decided], cls_ref[decided])
        plain = gu.Run(wl)
        _, rec_plain = plain.arm()
        assert (rec_gpu[..., 1] >= rec_plain[..., 1] - 1e-6).all() and np.allclose(rec_gpu[..., 0], rec_plain[..., 0], atol=1e-6)
        classes = [S_, T_, X_, D_]
        run.force_classes(classes)
        run.build()
        O, lse = run.sparse()
        for h, cls in enumerate(classes):
            ref = gu.oracle_lists(wl, cls, 128, 1, key_first=True)
            assert run.lists(0, h) == [ref[a] for a in range(run.sched.nQ)], (kw, cls)
            Or, lr = orc.masked_attention(run.q_bits[0, h], run.k_bits[0, h], run.v_bits[0, h], cls, g, pp)
            gu.check_attention(O[0, h], lse[0, h], Or, lr, f"key first frame, class {cls}", strict=False)
        # dynamic bandwidth: every candidate's Spatial recall carries the key frame too
        bws = [0.2, 0.5]
        plus = gu.Run(wl, key_first=1)
        _, _, rec_plus = plus.arm_plus(bws)
        for h in range(wl.H):
            _, _, _, Rt, Rs = orc.arm_head_plus(run.q_bits[0, h], run.k_bits[0, h], g, bws, wl.textural_stride, wl.sample_mode,
                                                wl.sample_stride, wl.alpha, keep_first_frame=True)
            assert np.abs(rec_plus[0, h, 0] - np.asarray(Rt)).max() <= gu.RECALL_ABS
            assert np.abs(rec_plus[0, h, 1] - np.asarray(Rs)).max() <= gu.RECALL_ABS
        for block in (16, 32, 64):
            small = gu.Run(wl, block=block, key_first=1)
            small.force_classes(classes)
            small.build()
            ref = gu.oracle_lists(wl, S_, block, 1, key_first=True)
            assert small.lists(0, 0) == [ref[a] for a in range(small.sched.nQ)], (kw, block)


# ------------------------------------------------------------------ Temporal heads with a 2-D in-frame window

@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("permute", [0, 1])
def test_temporal_2d_window(mode, permute):
    """The other reading of Sec. 3.2's locality for Temporal heads: a query keeps the keys whose in-frame row and column
    both lie within a window of its own, in every frame.  ARM's Temporal recall under both sampling modes, the tile lists
    at several tile sizes in both slot orders and the attention output against the oracle; the other patterns must not
    change, and the dynamic-bandwidth entry points refuse the combination."""
    for kw, t2d in ((dict(T=6, fh=12, fw=11, L=37, wf=1, ws=20, omega=6), (2, 3)),
                    (dict(T=9, fh=5, fw=8, L=0, wf=0, ws=3, omega=7), (0, 2)),
                    (dict(T=4, fh=20, fw=20, L=9, wf=2, ws=50, omega=3), (4, 1)),
                    (dict(T=3, fh=17, fw=23, L=5, wf=1, ws=9, omega=4), (40, 50))):      # a window past the frame: every key
        wl = synth.small_workload("t2d", H=4, D=64, mode=mode, amp=1.5, **kw)
        g, pp = gu.geom(wl), gu.pparams(wl, t2d=t2d)
        run = gu.Run(wl, temporal_permute=permute, t2d=t2d)
        cls_gpu, rec_gpu = run.arm()
        cls_ref, rec_ref, margin = orc.arm_classify(run.q_bits, run.k_bits, g, pp, wl.sample_mode, wl.sample_stride, wl.alpha)
        assert np.abs(rec_gpu - rec_ref).max() <= gu.RECALL_ABS, (kw, np.abs(rec_gpu - rec_ref).max())
        decided = margin > gu.TIE_MARGIN
        assert np.array_equal(cls_gpu[decided], cls_ref[decided])
        plain = gu.Run(wl, temporal_permute=permute)
        _, rec_plain = plain.arm()
        assert np.allclose(rec_gpu[..., 1:], rec_plain[..., 1:], atol=1e-6)       # Spatial and Textural recalls untouched
        classes = [S_, T_, X_, D_]
        run.force_classes(classes)
        run.build()
        O, lse = run.sparse()
        for h, cls in enumerate(classes):
            ref = gu.oracle_lists(wl, cls, 128, permute, t2d=t2d)
            assert run.lists(0, h) == [ref[a] for a in range(run.sched.nQ)], (kw, cls)
            Or, lr = orc.masked_attention(run.q_bits[0, h], run.k_bits[0, h], run.v_bits[0, h], cls, g, pp)
            gu.check_attention(O[0, h], lse[0, h], Or, lr, f"2-D temporal window {kw}, class {cls}", strict=False)
        for block in (16, 32, 64):
            small = gu.Run(wl, block=block, temporal_permute=permute, t2d=t2d)
            small.force_classes(classes)
            small.build()
            ref = gu.oracle_lists(wl, T_, block, permute, t2d=t2d)
            assert small.lists(0, 1) == [ref[a] for a in range(small.sched.nQ)], (kw, block)
        with pytest.raises(api.RainFusionError, match="unsupported"):
            run.arm_plus([0.2, 0.5])
