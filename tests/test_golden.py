"""Stored expected values (tests/golden/tiny_expected.json, written by tests/golden/make_golden.py from the
oracle alone): the oracle must still reproduce them (CPU), and the CUDA path must match them (GPU)."""
import json
import os

import numpy as np
import pytest

from oracle import rainfusion_oracle as orc
from paper_2505_21036_b200 import synth

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "tiny_expected.json")))
WL = synth.WORKLOADS["tiny"]


def test_oracle_still_reproduces_the_stored_values():
    g = orc.Geometry(WL.T, WL.frame_h, WL.frame_w, WL.L_text)
    pp = orc.PatternParams(WL.frame_window, WL.spatial_window, WL.textural_stride)
    q, k, v = synth.make_qkv(WL)
    cls, rec, _ = orc.arm_classify(q, k, g, pp, WL.sample_mode, WL.sample_stride, WL.alpha)
    assert cls[0].tolist() == GOLD["classes"]
    assert np.allclose(rec[0], GOLD["recall"], atol=1e-12)
    for key, lists in GOLD["tile_lists"].items():
        pat, perm = (int(x) for x in key.split("/"))
        assert [orc.tile_row(pat, g, pp, bool(perm), 128, 128, a) for a in range(3)] == lists
    for h, att in enumerate(GOLD["attention"]):
        O, lse = orc.masked_attention(q[0, h], k[0, h], v[0, h], GOLD["classes"][h], g, pp, rows=GOLD["rows"])
        assert np.allclose(O, att["O"], atol=1e-9) and np.allclose(lse, att["lse"], atol=1e-9)


@pytest.mark.gpu
def test_cuda_path_matches_the_stored_values():
    import torch
    import gpu_util as gu
    from paper_2505_21036_b200 import api
    for perm in (1, 0):
        run = gu.Run(WL, temporal_permute=perm)
        cls, rec = run.arm()
        assert cls[0].tolist() == GOLD["classes"]
        assert np.abs(rec[0] - np.asarray(GOLD["recall"])).max() <= gu.RECALL_ABS
        run.build()
        for h, c in enumerate(GOLD["classes"]):
            assert run.lists(0, h) == GOLD["tile_lists"][f"{c}/{perm}"]
            assert int(run.sched.kv_len[0, h]) == GOLD["kv_len"][str(c)]
        O, lse = run.sparse()
        for h, att in enumerate(GOLD["attention"]):
            gu.check_attention(O[0, h][GOLD["rows"]], lse[0, h][GOLD["rows"]], np.asarray(att["O"]), np.asarray(att["lse"]),
                               f"golden head {h}", strict=False)
        # every pattern's lists, forced
        for pat in (0, 1, 2, 3):
            run.force_classes([pat] * WL.H)
            run.build()
            assert run.lists(0, 0) == GOLD["tile_lists"][f"{pat}/{perm}"]
