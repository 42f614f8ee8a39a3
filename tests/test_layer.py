"""The per-layer call policy (dense early steps, then ARM -> schedule -> masked attention; optional CUDA graph)."""
import numpy as np
import pytest
import torch

from paper_2505_21036_b200 import api, synth
from paper_2505_21036_b200.layer import RainFusionAttention


def make_layer(device, **kw):
    wl = synth.small_workload("layer", H=4, D=64, T=6, fh=12, fw=11, L=37, wf=1, ws=20, tau=2, mode=0, omega=6, amp=1.5)
    return wl, RainFusionAttention(api.shape_of(wl), api.params_of(wl), device, **kw)


def test_dense_step_policy_and_speedup_arithmetic():
    wl, layer = make_layer("cpu")
    assert layer.dense_steps(50) == 5 and layer.dense_steps(10) == 1 and layer.dense_steps(4) == 1
    assert [layer.is_dense_step(s, 50) for s in (0, 4, 5, 49)] == [True, True, False, False]
    # Sec. 4.2: 50 % sparsity with the first tenth of the steps dense; the paper's attention speed-up figure is 1.85x
    assert layer.expected_attention_speedup(50, 0.5) == pytest.approx(1.0 / (0.1 + 0.9 * 0.5))
    assert 1.8 < layer.expected_attention_speedup(50, 0.5) < 1.86
    wl, none_dense = make_layer("cpu", dense_fraction=0.0)
    assert none_dense.dense_steps(50) == 0
    with pytest.raises(ValueError):
        make_layer("cpu", dense_fraction=1.5)


@pytest.mark.gpu
@pytest.mark.parametrize("plus", [False, True])
def test_layer_equals_the_entry_points_and_graph_replay_equals_eager(plus):
    bws = [0.125, 0.25, 0.5] if plus else None
    wl, eager = make_layer("cuda", bandwidths=bws)
    _, graphed = make_layer("cuda", graph=True, bandwidths=bws)
    q, k, v = (torch.from_numpy(x.view(np.int16)).view(torch.bfloat16).cuda() for x in synth.make_qkv(wl))

    def fresh():
        return (torch.full_like(q, float("nan")), torch.full((wl.B, wl.H, wl.N), float("nan"), device="cuda"))
    # a dense step is rf_dense_attn_fwd
    o0, l0 = fresh()
    eager(q, k, v, o0, l0, step=0, num_steps=20)
    o1, l1 = fresh()
    api.rf_dense_attn_fwd(eager.shape, q, k, v, o1, l1, eager.status)
    assert torch.equal(o0.view(torch.int16), o1.view(torch.int16)) and torch.equal(l0, l1)
    # a sparse step is the three calls in a row
    o2, l2 = fresh()
    eager(q, k, v, o2, l2, step=7, num_steps=20)
    if not plus:
        o3, l3 = fresh()
        api.rf_arm_classify(eager.shape, eager.params, q, k, eager.head_class, None, eager.ws)
        api.rf_build_block_mask(eager.shape, eager.params, eager.head_class, eager.sched, eager.status)
        api.rf_sparse_attn_fwd(eager.shape, eager.params, q, k, v, eager.head_class, eager.sched, o3, l3, eager.ws,
                               eager.status)
        assert torch.equal(o2.view(torch.int16), o3.view(torch.int16)) and torch.equal(l2, l3)
        assert not torch.equal(o2.view(torch.int16), o0.view(torch.int16))     # the masks really drop something
    # graph: capture on first use, then replays follow the CONTENTS of the same buffers
    og, lg = fresh()
    graphed(q, k, v, og, lg, step=7, num_steps=20)
    assert torch.equal(og.view(torch.int16), o2.view(torch.int16)) and torch.equal(lg, l2)
    q2 = q.clone()
    q.copy_(torch.roll(q2, 1, dims=1))          # heads permuted: other classes, other schedule, other output
    graphed(q, k, v, og, lg, step=8, num_steps=20)
    oe, le = fresh()
    eager(q, k, v, oe, le, step=8, num_steps=20)
    torch.cuda.synchronize()
    assert torch.equal(og.view(torch.int16), oe.view(torch.int16)) and torch.equal(lg, le)
    assert not torch.equal(og.view(torch.int16), o2.view(torch.int16))
    assert len(graphed._graphs) == 1
    eager.check()
    graphed.check()


@pytest.mark.gpu
@pytest.mark.parametrize("groups", [1, 2, 4])
def test_host_staged_call_equals_the_resident_pipeline(groups):
    wl, eager = make_layer("cuda", dense_fraction=0.0)
    from paper_2505_21036_b200.layer import HostStagedAttention
    staged = HostStagedAttention(api.shape_of(wl), api.params_of(wl), "cuda", groups=groups)
    host = [torch.from_numpy(x.view(np.int16)).view(torch.bfloat16).pin_memory() for x in synth.make_qkv(wl)]
    oh = torch.full(host[0].shape, float("nan"), dtype=torch.bfloat16).pin_memory()
    for _ in range(2):                                   # back-to-back calls reuse the staging buffers
        staged(*host, oh)
    torch.cuda.synchronize()
    q, k, v = (t.cuda() for t in host)
    o = torch.empty_like(q)
    eager(q, k, v, o, None, step=0, num_steps=1)
    torch.cuda.synchronize()
    assert int(staged.status.item()) == 0
    assert torch.equal(oh.view(torch.int16), o.cpu().view(torch.int16))
    with pytest.raises(ValueError):
        HostStagedAttention(api.shape_of(wl), api.params_of(wl), "cuda", groups=3)


@pytest.mark.gpu
def test_host_staged_calls_back_to_back_with_different_inputs():
    """Consecutive calls overlap (the next call's copy-in runs under this call's kernels): each call's output must
    still belong to its own inputs."""
    wl, eager = make_layer("cuda", dense_fraction=0.0)
    from paper_2505_21036_b200.layer import HostStagedAttention
    staged = HostStagedAttention(api.shape_of(wl), api.params_of(wl), "cuda", groups=2)
    base = [torch.from_numpy(x.view(np.int16)).view(torch.bfloat16) for x in synth.make_qkv(wl)]
    sets = []
    for shift in range(4):                      # heads rotated: other classes, other schedules, other outputs
        sets.append([torch.roll(t, shift, dims=1).contiguous().pin_memory() for t in base])
    outs = [torch.full(base[0].shape, float("nan"), dtype=torch.bfloat16).pin_memory() for _ in sets]
    for inp, out in zip(sets, outs):            # no synchronisation in between
        staged(*inp, out)
    torch.cuda.synchronize()
    assert int(staged.status.item()) == 0
    for inp, out in zip(sets, outs):
        q, k, v = (t.cuda() for t in inp)
        o = torch.empty_like(q)
        eager(q, k, v, o, None, step=0, num_steps=1)
        torch.cuda.synchronize()
        assert torch.equal(out.view(torch.int16), o.cpu().view(torch.int16))
    assert not torch.equal(outs[0].view(torch.int16), outs[1].view(torch.int16))


@pytest.mark.gpu
def test_host_staged_call_with_dynamic_bandwidth():
    """The host pipeline with candidate bandwidths set (Sec. 4.3): classes, per-head windows and output equal the
    resident dynamic-bandwidth entry points bit for bit; invalid lists are refused; clearing the list returns to the
    fixed windows."""
    wl, eager = make_layer("cuda", dense_fraction=0.0)
    shape, params = api.shape_of(wl), api.params_of(wl)
    pipe = api.HostPipeline(shape, params, "cuda", 2 if (wl.B * wl.H) % 2 == 0 else 1)
    bws = [0.125, 0.25, 0.5]
    for bad in ([0.5, 0.25], [0.0], [1.5], [0.1, 0.2, 0.3, 0.4, 0.5]):
        with pytest.raises(api.RainFusionError):
            pipe.set_bandwidths(bad)
    pipe.set_bandwidths(bws)
    host = [torch.from_numpy(x.view(np.int16)).view(torch.bfloat16).pin_memory() for x in synth.make_qkv(wl)]
    oh = torch.full(host[0].shape, float("nan"), dtype=torch.bfloat16).pin_memory()
    pipe.run(*host, oh)
    assert pipe.status() == 0
    q, k, v = (t.cuda() for t in host)
    ws = api.alloc_workspace(shape, params, "cuda")
    sched = api.Schedule(shape, params, "cuda")
    hc = torch.zeros((wl.B, wl.H), dtype=torch.int32, device="cuda")
    hw = torch.zeros((wl.B, wl.H), dtype=torch.int32, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    o = torch.empty_like(q)
    api.rf_arm_classify_plus(shape, params, bws, q, k, hc, hw, None, ws, st)
    api.rf_build_block_mask_plus(shape, params, hc, hw, sched, st)
    api.rf_sparse_attn_fwd_plus(shape, params, q, k, v, hc, hw, sched, o, None, ws, st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    assert np.array_equal(pipe.head_class(), hc.cpu().numpy().reshape(-1))
    assert np.array_equal(pipe.head_window(), hw.cpu().numpy().reshape(-1))
    assert torch.equal(oh.view(torch.int16), o.cpu().view(torch.int16))
    pipe.set_bandwidths([])
    pipe.run(*host, oh)
    assert pipe.status() == 0
    eager(q, k, v, o, None, step=0, num_steps=1)
    torch.cuda.synchronize()
    assert torch.equal(oh.view(torch.int16), o.cpu().view(torch.int16))
    pipe.close()
