"""Pattern-mix and shape sweep: per-head pattern assignment forced to all-Spatial, all-Temporal,
all-Textural and an even mix, with the Temporal token permutation on and off, at the three sweep
shapes (D = 128, H = 24).  Prints one JSON line per case: tile density, ms per attention call,
computed-tile TFLOP/s and its fraction of the measured bf16 peak.

  python -m paper_2505_21036_b200.sweep [--shapes sweep_8x1024 sweep_16x2040 sweep_33x3600] [--reps 5]

Inputs are iid N(0,1) drawn on the device (timing does not depend on the values); parity for these
cases is covered by the GPU tests.
"""
from __future__ import annotations

import argparse
import json
import os

import torch

from . import api, synth


def measured_peak() -> float:
    p = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "MEASURED_PEAKS.json")
    return json.load(open(p))["bf16_tflops"] if os.path.exists(p) else 1590.0


def run_case(wl, classes, permute, q, k, v, o, status, reps):
    dev = q.device
    shape, params = api.shape_of(wl), api.params_of(wl, 128, 128, permute)
    ws = api.alloc_workspace(shape, params, dev)
    sched = api.Schedule(shape, params, dev)
    hc = torch.tensor(classes, dtype=torch.int32, device=dev).reshape(wl.B, wl.H)
    api.rf_build_block_mask(shape, params, hc, sched, status)

    def call():
        api.rf_sparse_attn_fwd(shape, params, q, k, v, hc, sched, o, None, ws, status)
    for _ in range(3):
        call()
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(reps):
        call()
    b.record()
    torch.cuda.synchronize()
    ms = a.elapsed_time(b) / reps
    listed = int(sched.count.sum().item())
    cnt = sched.count.reshape(-1, sched.nQ)
    idx = torch.arange(sched.nKmax, device=dev)[None, None, :]
    partial = int(((sched.kv_tile.reshape(-1, sched.nQ, sched.nKmax) < 0) & (idx < cnt[..., None])).sum().item())
    return ms, listed, partial, sched.nQ * sched.nKmax * wl.B * wl.H


def run_plus(name, bandwidths, reps):
    """Dynamic bandwidth (RainFusion+) on the seeded planted inputs of a workload: ARM picks a window per head."""
    import numpy as np
    wl = synth.WORKLOADS[name]
    q, k, v = (torch.from_numpy(x.view(np.int16)).cuda().view(torch.bfloat16) for x in synth.make_qkv(wl))
    o = torch.empty_like(q)
    shape, params = api.shape_of(wl), api.params_of(wl)
    ws = api.alloc_workspace(shape, params, "cuda")
    sched = api.Schedule(shape, params, "cuda")
    hc = torch.zeros((wl.B, wl.H), dtype=torch.int32, device="cuda")
    hw = torch.zeros((wl.B, wl.H), dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")

    def timed(fn):
        for _ in range(2):
            fn()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(reps):
            fn()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / reps
    arm_ms = timed(lambda: api.rf_arm_classify_plus(shape, params, bandwidths, q, k, hc, hw, None, ws))
    api.rf_build_block_mask_plus(shape, params, hc, hw, sched, status)
    attn_ms = timed(lambda: api.rf_sparse_attn_fwd_plus(shape, params, q, k, v, hc, hw, sched, o, None, ws, status))
    listed = int(sched.count.sum().item())
    tf = 4.0 * 128 * 128 * wl.D * listed / (attn_ms * 1e-3) / 1e12
    assert int(status.item()) == 0
    picks = sorted(zip(hc.cpu().numpy().reshape(-1).tolist(), hw.cpu().numpy().reshape(-1).tolist()))
    hist = {}
    for c, w in picks:
        hist[f"class{c}/window{w}"] = hist.get(f"class{c}/window{w}", 0) + 1
    print(json.dumps({"workload": name, "variant": "dynamic bandwidth", "bandwidths": bandwidths, "arm_ms": arm_ms,
                      "attn_ms": attn_ms, "arm_overhead_pct": 100 * arm_ms / attn_ms, "picks": hist,
                      "tile_density": listed / float(wl.B * wl.H * sched.nQ * sched.nKmax), "computed_tile_tflops": tf,
                      "dense_equiv_tflops": 4.0 * wl.B * wl.H * wl.N ** 2 * wl.D / (attn_ms * 1e-3) / 1e12}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--shapes", nargs="+", default=["sweep_8x1024", "sweep_16x2040", "sweep_33x3600"])
    ap.add_argument("--reps", type=int, default=5)
    ap.add_argument("--plus", metavar="WORKLOAD", help="run the dynamic-bandwidth variant on this workload and exit")
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("sweep: needs a CUDA device")
    if args.plus:
        run_plus(args.plus, [0.125, 0.25, 0.5], args.reps)
        return
    peak = measured_peak()
    for name in args.shapes:
        wl = synth.WORKLOADS[name]
        g = torch.Generator(device="cuda")
        g.manual_seed(5)
        q = torch.randn((wl.B, wl.H, wl.N, wl.D), device="cuda", dtype=torch.bfloat16, generator=g)
        k, v, o = torch.randn_like(q), torch.randn_like(q), torch.empty_like(q)
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        H = wl.H
        cases = [("all-spatial", [0] * H, 1), ("all-temporal", [1] * H, 1), ("all-temporal", [1] * H, 0),
                 ("all-textural", [2] * H, 1), ("even-mix", [0, 1, 2] * (H // 3), 1), ("even-mix", [0, 1, 2] * (H // 3), 0),
                 ("dense", [3] * H, 1)]
        for label, classes, permute in cases:
            ms, listed, partial, total = run_case(wl, classes, permute, q, k, v, o, status, args.reps)
            tf = 4.0 * 128 * 128 * wl.D * listed / (ms * 1e-3) / 1e12
            print(json.dumps({"workload": name, "N": wl.N, "assignment": label, "temporal_permute": permute,
                              "tile_density": listed / total, "partial_share": partial / max(listed, 1),
                              "ms_per_call": ms, "computed_tile_tflops": tf, "frac_of_measured_bf16_peak": tf / peak,
                              "dense_equiv_tflops": 4.0 * wl.B * wl.H * wl.N ** 2 * wl.D / (ms * 1e-3) / 1e12}))
        assert int(status.item()) == 0


if __name__ == "__main__":
    main()
