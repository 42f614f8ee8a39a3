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


def draw_case(seed):
    rng = np.random.default_rng(9000 + seed)
    D = int(rng.choice([64, 96, 128]))
    T = int(rng.integers(1, 8))
    fh, fw = int(rng.integers(1, 13)), int(rng.integers(1, 13))
    S = fh * fw
    L = int(rng.choice([0, 1, 17, 130]))
    if T * S + L < 2:
        L = 17
    kw = dict(B=int(rng.choice([1, 2])), H=4, D=D, T=T, fh=fh, fw=fw, L=L,
              wf=int(rng.integers(0, T + 1)), ws=int(rng.integers(0, S + 1)), tau=int(rng.integers(1, 5)),
              mode=int(rng.integers(0, 2)), omega=int(rng.integers(1, max(2, S // 2 + 1))),
              amp=float(rng.choice([0.0, 0.8, 1.5, 2.5])))
    wl = synth.small_workload(f"fuzz{seed}", **kw)
    permute = int(rng.integers(0, 2))
    two_mask = int(rng.integers(0, 2))
    classes = rng.integers(0, 4, size=(wl.B, wl.H)).astype(np.int32)
    return wl, permute, two_mask, classes


@pytest.mark.parametrize("seed", range(32))
def test_random_case(seed):
    wl, permute, two_mask, classes = draw_case(seed)
    g, pp = gu.geom(wl), gu.pparams(wl)
    run = gu.Run(wl, temporal_permute=permute, two_mask=two_mask)
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
            ref = gu.oracle_lists(wl, cls, 128, permute)
            assert run.lists(b, h) == [ref[a] for a in range(run.sched.nQ)], (seed, b, h, cls)
            assert int(run.sched.kv_len[b, h]) == orc.kv_len(cls, g, pp)
            Or, lr = orc.masked_attention(run.q_bits[b, h], run.k_bits[b, h], run.v_bits[b, h], cls, g, pp)
            gu.check_attention(O[b, h], lse[b, h], Or, lr, f"fuzz {seed} b{b} h{h} class {cls}", strict=False)
    if seed % 4 == 0:
        Od, lsed = run.dense()
        Or, lr = orc.masked_attention(run.q_bits[0, 1], run.k_bits[0, 1], run.v_bits[0, 1], orc.DENSE, g, pp)
        gu.check_attention(Od[0, 1], lsed[0, 1], Or, lr, f"fuzz {seed} dense", strict=False)
