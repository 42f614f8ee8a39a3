"""Tensors of more than 2^31 elements: every index computation on the path must be 64-bit.

B*H*N*D = 72 * 240 300 * 128 = 2.21e9 elements per tensor (4.4 GB in bf16).  Inputs are drawn on the device
(seeded); the heads that are checked are copied back and go through the oracle on sampled query rows."""
import numpy as np
import pytest
import torch

from oracle import rainfusion_oracle as orc
from paper_2505_21036_b200 import api, synth

import gpu_util as gu

pytestmark = pytest.mark.gpu


def test_more_than_two_to_the_31_elements():
    wl = synth.small_workload("huge", H=72, D=128, T=20, fh=100, fw=120, L=300, tau=2, mode=1, omega=100, amp=0.0)
    assert wl.B * wl.H * wl.N * wl.D > 2 ** 31
    free, _ = torch.cuda.mem_get_info()
    if free < 60 * 2 ** 30:
        pytest.skip("needs 60 GB of free device memory")
    gen = torch.Generator(device="cuda")
    gen.manual_seed(20250521)
    q, k, v = (torch.randn((wl.B, wl.H, wl.N, wl.D), device="cuda", dtype=torch.bfloat16, generator=gen) for _ in range(3))
    shape, params = api.shape_of(wl), api.params_of(wl)
    ws = api.alloc_workspace(shape, params, "cuda")
    sched = api.Schedule(shape, params, "cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    head_class = torch.zeros((wl.B, wl.H), dtype=torch.int32, device="cuda")
    recall = torch.zeros((wl.B, wl.H, 3), dtype=torch.float32, device="cuda")
    g, pp = gu.geom(wl), gu.pparams(wl)
    check_heads = [0, 34, 70, 71]          # classes S, T, T, X below; the last ones sit past the 2^31-element mark

    def bits(t, h):
        return t[0, h].cpu().view(torch.int16).numpy().view(np.uint16)

    # ARM on iid inputs: recalls of the last heads against the oracle (all heads fall through to Textural)
    api.rf_arm_classify(shape, params, q, k, head_class, recall, ws)
    torch.cuda.synchronize()
    rec = recall.cpu().numpy()[0]
    for h in (0, 71):
        cls, R, margin = orc.arm_head(bits(q, h), bits(k, h), g, pp, wl.sample_mode, wl.sample_stride, wl.alpha)
        assert np.abs(rec[h] - np.asarray(R)).max() <= gu.RECALL_ABS, (h, rec[h], R)
        assert int(head_class[0, h]) == cls == orc.TEXTURAL

    classes = np.array([[(0, 1, 2)[h % 3] for h in range(wl.H)]], dtype=np.int32)
    classes[0, 70] = 1
    classes[0, 71] = 2
    head_class.copy_(torch.from_numpy(classes))
    api.rf_build_block_mask(shape, params, head_class, sched, status)
    o = torch.full((wl.B, wl.H, wl.N, wl.D), float("nan"), dtype=torch.bfloat16, device="cuda")
    lse = torch.full((wl.B, wl.H, wl.N), float("nan"), dtype=torch.float32, device="cuda")
    api.rf_sparse_attn_fwd(shape, params, q, k, v, head_class, sched, o, lse, ws, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0

    rows = synth.sample_rows(wl, 24, seed=12)
    tiles = [0, 1, sched.nQ // 2, sched.nQ - 2, sched.nQ - 1]
    for h in check_heads:
        cls = int(classes[0, h])
        cnt = sched.count[0, h].cpu().numpy()
        til = sched.kv_tile[0, h].cpu().numpy().view(np.uint32)
        ref = gu.oracle_lists(wl, cls, 128, 1, tiles)
        for a in tiles:
            assert til[a, :cnt[a]].tolist() == ref[a], (h, a)
        Or, lr = orc.masked_attention(bits(q, h), bits(k, h), bits(v, h), cls, g, pp, rows=rows)
        Og = o[0, h].float().cpu().numpy().astype(np.float64)[rows]
        lg = lse[0, h].cpu().numpy().astype(np.float64)[rows]
        gu.check_attention(Og, lg, Or, lr, f"huge head {h} class {cls}")
    assert not torch.isnan(o[0, -1, -1].float()).any()
