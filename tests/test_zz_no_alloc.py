"""rf_arm_classify_noalloc: the ARM entry point for callers that cannot allocate device memory.

A serving process whose memory pool is frozen after start-up, or a plug-in that must not re-enter its
host framework's allocator, has no workspace to pass and may not cudaMalloc one.  For them the library
keeps the ARM scratch in a fixed array of its own.  This test drives that entry point through the C ABI
and holds it to the workspace-taking rf_arm_classify: same classes, recalls within the tolerance the
other ARM tests use, on two calls in a row (the second on a different shape, so stale contents of the
shared array would show).  It lives in a file that sorts last so that a stop-at-first-failure run has
already been through every other test.
"""
import numpy as np
import pytest
import torch

from paper_2505_21036_b200 import api, synth

import gpu_util as gu


def _both(wl):
    run = gu.Run(wl)
    cls_ws, rec_ws = run.arm()
    cls_ws, rec_ws = cls_ws.copy(), rec_ws.copy()
    head_class = torch.full((wl.B, wl.H), -1, dtype=torch.int32, device="cuda")
    recall = torch.full((wl.B, wl.H, 3), float("nan"), dtype=torch.float32, device="cuda")
    api.rf_arm_classify_noalloc(run.shape, run.params, run.q, run.k, head_class, recall)
    torch.cuda.synchronize()
    return cls_ws, rec_ws, head_class.cpu().numpy(), recall.cpu().numpy()


@pytest.mark.gpu
def test_noalloc_matches_workspace_entry_point_twice_in_a_row():
    first = synth.small_workload("na_a", H=6, D=128, T=6, fh=12, fw=11, L=37, wf=1, ws=20, tau=2, mode=0, omega=6)
    second = synth.WORKLOADS["tiny"]
    for wl in (first, second, first):
        cls_ws, rec_ws, cls_na, rec_na = _both(wl)
        assert np.array_equal(cls_na, cls_ws)
        assert np.isfinite(rec_na).all()
        assert np.abs(rec_na - rec_ws).max() <= gu.RECALL_ABS


@pytest.mark.gpu
def test_noalloc_allocates_no_device_memory():
    wl = synth.WORKLOADS["tiny"]
    run = gu.Run(wl)
    api.rf_arm_classify_noalloc(run.shape, run.params, run.q, run.k, run.head_class, run.recall)  # set-up call
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    for _ in range(3):
        api.rf_arm_classify_noalloc(run.shape, run.params, run.q, run.k, run.head_class, run.recall)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before


def test_noalloc_rejects_problems_beyond_its_scratch():
    # host-side check only: nothing is launched, so this runs without a GPU
    big = api.make_shape(4, 64, 128, 33, 45, 80, 256)
    params = api.make_params(8, 900, sample_stride=36)
    # the pointers are never dereferenced: the size check comes before any CUDA call
    code = api.load().rf_arm_classify_noalloc(big, params, 16, 16, 16, None, None, None)
    assert code == 6          # RF_ERR_STATIC_SCRATCH_TOO_SMALL
    assert b"built-in" in api.load().rf_status_string(code)
