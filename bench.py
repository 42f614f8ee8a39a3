#!/usr/bin/env python
"""Benchmark of the RainFusion hot path on B200: ARM -> block mask -> pattern-masked attention.

One step = one pass of the whole path (rf_arm_classify, rf_build_block_mask, rf_sparse_attn_fwd
with its token reordering) over one HunyuanVideo-720p-shaped attention layer of seeded synthetic
Q/K/V (118 800 video + 256 text tokens, 24 heads, D = 128, bf16).  Prints one JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

With --impl reference the CPU oracle is timed instead (a bounded row sample per step).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2505_21036_b200 import synth  # noqa: E402

METRIC = "dense_equiv_tflops_sparse_attn"
UNIT = "TFLOP/s"

# dram__bytes_read.sum + dram__bytes_write.sum of one rf_attn_kernel launch, from single-pass ncu captures; None
# where no capture exists.  The figure is a recorded measurement, not taken in this run: TRAFFIC_SOURCE names the
# summary it comes from and the state of the kernel source it was captured on; re-capture when rf_attn.cu changes.
ATTN_DRAM_BYTES = {"hunyuan720p": 4.67e9, "sweep_33x3600": 4.67e9, "sweep_16x2040": 0.734e9}
TRAFFIC_SOURCE = {"file": "profiles/rf_attn_kernel_hunyuan720p_dram_bytes.md",
                  "captured_on": "the kernel as of the commit that last touched profiles/ (its body is that of commit 2bbb852)"}
NOMINAL_BF16_TFLOPS = 2250.0     # NVIDIA's dense bf16 figure for one B200 (the 4.5 PFLOP/s quoted per GPU is with 2:4 sparsity)


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_burst": d["bf16_tflops"], "bf16_sustained": d["bf16_tflops_sustained"],
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_burst": 1590.0, "bf16_sustained": 1400.0, "source": "fallback"}


def dense_flops(wl):
    return 4.0 * wl.B * wl.H * float(wl.N) ** 2 * wl.D


# ------------------------------------------------------------------------------ clocks

class ClockSampler:
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap,power.draw.instant,power.limit")

    def __init__(self, gpu_id: str):
        """gpu_id: what `nvidia-smi -i` takes.  Pass the device's UUID ("GPU-..."): the CUDA ordinal is not the
        nvidia-smi index when CUDA_VISIBLE_DEVICES reorders or hides GPUs of a shared machine."""
        self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", gpu_id, f"--query-gpu={self.QUERY}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=self.tmp, stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.tmp.flush()
        rows = [l.strip().split(", ") for l in open(self.tmp.name) if l.strip()]
        os.unlink(self.tmp.name)
        sm, pw, reasons, mx, limit = [], [], set(), None, None
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            if len(r) < 7:
                continue
            try:
                sm.append(float(r[0]))
                mx = float(r[1])
            except ValueError:
                continue
            try:
                # power.draw is a one-second average on this generation: take the instantaneous reading
                pw.append(float(r[7]))
                limit = float(r[8])
            except (ValueError, IndexError):
                pass
            for n, val in zip(names, r[3:7]):
                if val.strip().lower().startswith("active"):
                    reasons.add(n)
        if sm:
            out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=mx, reasons=sorted(reasons), samples=len(sm))
        if pw:
            # board power over the same samples: with sw_power_cap among the reasons and the median at the board's limit
            # the timed kernels are bound by power, and the SM clock is what the limit leaves
            out.update(power_w=float(np.median(pw)), power_w_max=float(np.max(pw)), power_limit_w=limit)
        return out


# ------------------------------------------------------------------------------ reference arm (CPU oracle)

def oracle_sample(wl, rows_per_step: int, qkv_head=None):
    """One bounded unit of oracle work: ARM for one head plus masked attention for `rows_per_step`
    query rows of that head (its oracle class).  Returns (seconds, dense-equivalent flops covered)."""
    from oracle import rainfusion_oracle as orc
    g = orc.Geometry(wl.T, wl.frame_h, wl.frame_w, wl.L_text)
    pp = orc.PatternParams(wl.frame_window, wl.spatial_window, wl.textural_stride)
    q, k, v = qkv_head if qkv_head is not None else synth.make_head(wl, 0, 0)
    rows = synth.sample_rows(wl, rows_per_step, seed=1)
    t0 = time.perf_counter()
    cls, _, _ = orc.arm_head(q, k, g, pp, wl.sample_mode, wl.sample_stride, wl.alpha)
    orc.masked_attention(q, k, v, cls, g, pp, rows=rows)
    dt = time.perf_counter() - t0
    return dt, 4.0 * len(rows) * float(wl.N) * wl.D, len(rows)


def threads_used():
    try:
        from threadpoolctl import threadpool_info
        n = [d.get("num_threads", 1) for d in threadpool_info() if d.get("user_api") == "blas"]
        if n:
            return int(max(n))
    except Exception:
        pass
    return os.cpu_count() or 1


def run_reference(args, wl):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    head = synth.make_head(wl, 0, 0)
    rows = args.ref_rows
    for _ in range(min(args.warmup, 1)):
        oracle_sample(wl, rows, head)
    times, flops = [], 0.0
    for _ in range(args.steps):
        dt, fl, nrows = oracle_sample(wl, rows, head)
        times.append(dt)
        flops = fl
    ms = 1e3 * float(np.mean(times))
    value = flops / (ms * 1e-3) / 1e12
    sample = f"head 0: ARM + masked attention (oracle class) on {nrows} of {wl.N} query rows per step"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": min(args.warmup, 1), "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": wl.name, "B": wl.B, "H": wl.H, "D": wl.D, "T": wl.T, "frame": [wl.frame_h, wl.frame_w],
                       "L_text": wl.L_text, "N": wl.N},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads_used(), "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ------------------------------------------------------------------------------ CUDA arm

def run_cuda(args, wl):
    import torch
    from paper_2505_21036_b200 import api, dist_util

    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the hot path has no CPU fallback")
    api.load()
    rank, world, local = dist_util.env_rank()
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist_util.init("nccl", dev)

    # inputs: seeded on the host (pinned, for the end-to-end leg), resident copy on the device
    qh, kh, vh = (torch.from_numpy(x.view(np.int16)).view(torch.bfloat16).pin_memory() for x in synth.make_qkv(wl))
    q, k, v = qh.to(dev), kh.to(dev), vh.to(dev)
    shape, params = api.shape_of(wl), api.params_of(wl)
    ws = api.alloc_workspace(shape, params, dev)
    sched = api.Schedule(shape, params, dev)
    head_class = torch.zeros((wl.B, wl.H), dtype=torch.int32, device=dev)
    recall = torch.zeros((wl.B, wl.H, 3), dtype=torch.float32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    o = torch.empty_like(q)
    lse = torch.empty((wl.B, wl.H, wl.N), dtype=torch.float32, device=dev)
    oh = torch.empty(o.shape, dtype=torch.bfloat16).pin_memory()

    def ev():
        return torch.cuda.Event(enable_timing=True)

    def step(events=None):
        if events:
            events[0].record()
        api.rf_arm_classify(shape, params, q, k, head_class, None, ws, status)   # classes only, as Algorithm 1 needs
        if events:
            events[1].record()
        api.rf_build_block_mask(shape, params, head_class, sched, status)
        if events:
            events[2].record()
        # rf_sparse_attn_fwd as its two launches, so that the attention kernel is timed by itself
        api.rf_reorder_tokens(shape, params, q, k, v, head_class, ws)
        if events:
            events[3].record()
        api.rf_sparse_attn_reordered(shape, params, q, k, v, head_class, None, sched, o, lse, ws, status)
        if events:
            events[4].record()

    def barrier():
        torch.cuda.synchronize()
        dist_util.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    barrier()
    if int(status.item()) != 0:
        raise SystemExit(f"bench.py: device status {int(status.item())}")

    try:
        gpu_uuid = "GPU-" + str(torch.cuda.get_device_properties(local).uuid)
    except Exception:                      # no uuid attribute: fall back to the ordinal and say so in the line
        gpu_uuid = None
    sampler = ClockSampler(gpu_uuid if gpu_uuid else str(local)) if rank == 0 else None
    per = [[ev() for _ in range(5)] for _ in range(args.steps)]
    t_begin, t_end = ev(), ev()
    barrier()
    t_begin.record()
    for i in range(args.steps):
        step(per[i])
    t_end.record()
    barrier()
    total_ms = t_begin.elapsed_time(t_end)
    clocks = sampler.stop() if sampler else None
    stages = {"arm": [p[0].elapsed_time(p[1]) for p in per], "block_mask": [p[1].elapsed_time(p[2]) for p in per],
              "reorder": [p[2].elapsed_time(p[3]) for p in per], "attn_kernel": [p[3].elapsed_time(p[4]) for p in per],
              "sparse_attn_call": [p[2].elapsed_time(p[4]) for p in per]}
    arm_ms, mask_ms, reorder_ms, attn_kernel_ms, sparse_ms = (float(np.mean(stages[n])) for n in (
        "arm", "block_mask", "reorder", "attn_kernel", "sparse_attn_call"))

    # the dense baseline, timed the same way (not part of the step)
    def timed(fn, n):
        fn()
        torch.cuda.synchronize()
        a, b = ev(), ev()
        a.record()
        for _ in range(n):
            fn()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / n
    dense_ms = timed(lambda: api.rf_dense_attn_fwd(shape, q, k, v, o, lse, status), 2) if args.dense else None

    # end to end with host buffers (pinned): every step moves Q, K, V to the device and O back inside the timed
    # region, through one C-ABI call (rf_host_pipeline_run) that takes host pointers.  The library pipelines groups of
    # heads over a copy-in, a compute and a copy-out stream; the same kernels run as in the device-resident step.
    from paper_2505_21036_b200.layer import HostStagedAttention
    heads = wl.B * wl.H
    groups = args.e2e_groups if args.e2e_groups > 0 else next(g for g in (8, 6, 4, 3, 2, 1) if heads % g == 0)
    staged = HostStagedAttention(shape, params, dev, groups=groups)

    def e2e_step():
        staged(qh, kh, vh, oh)
    e2e_n = max(2, min(args.steps, 10))
    e2e_step()
    barrier()
    a, b = ev(), ev()
    a.record()
    for _ in range(e2e_n):
        e2e_step()
    b.record()
    barrier()
    e2e_ms = a.elapsed_time(b) / e2e_n
    if int(staged.status.item()) != 0:
        raise SystemExit(f"bench.py: device status {int(staged.status.item())} in the host-staged leg")
    step()                                                                           # untimed: o = the resident path's output again
    torch.cuda.synchronize()
    e2e_same = bool(torch.equal(oh.view(torch.int16), o.cpu().view(torch.int16)))   # same bits as the resident path

    api.rf_arm_classify(shape, params, q, k, head_class, recall, ws, status)       # untimed: recalls for the report
    torch.cuda.synchronize()
    rec = recall.cpu().numpy().reshape(-1, 3)
    cls = head_class.cpu().numpy().reshape(-1)
    listed = int(sched.count.sum().item())
    if int(status.item()) != 0:
        raise SystemExit(f"bench.py: device status {int(status.item())}")

    ms_per_step = total_ms / args.steps
    ms_per_step, e2e_ms = dist_util.max_over_ranks([ms_per_step, e2e_ms], dev)

    if rank == 0:
        pk = peaks()
        dflops = dense_flops(wl)
        tile_flops = 4.0 * 128 * 128 * wl.D * listed
        achieved = tile_flops / (attn_kernel_ms * 1e-3) / 1e12
        line = {
            "metric": METRIC, "value": dist_util.replica_throughput(dflops, ms_per_step, world) / 1e12, "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": wl.name, "B": wl.B, "H": wl.H, "D": wl.D, "T": wl.T, "frame": [wl.frame_h, wl.frame_w],
                       "L_text": wl.L_text, "N": wl.N, "block": 128, "temporal_permute": 1,
                       "frame_window": wl.frame_window, "spatial_window": wl.spatial_window,
                       "textural_stride": wl.textural_stride, "sample_stride": wl.sample_stride,
                       "l2": f"inputs ({3 * wl.B * wl.H * wl.N * wl.D * 2 / 1e9:.2f} GB of Q/K/V) exceed the 126 MB L2; no flush", "parallelism": f"replicas x{world}"},
            "clocks": dict(clocks or {}, gpu=gpu_uuid if gpu_uuid else f"ordinal {local}"),
            "e2e": {"value": dist_util.replica_throughput(dflops, e2e_ms, world) / 1e12, "unit": UNIT, "ms_per_step": e2e_ms,
                    "h2d_bytes_per_step": staged.h2d_bytes, "d2h_bytes_per_step": staged.d2h_bytes,
                    "head_groups": groups, "equals_resident_output": e2e_same, "steps": e2e_n,
                    "api": "rf_host_pipeline_run: one C-ABI call per step with host pointers; the copies are issued inside the library",
                    "overlap": "head groups inside a step; copy-in of the next step under the kernels of this one"},
            "gpu_launches": args.steps * 5,   # rf_arm_kernel, rf_arm_decide_kernel, rf_build_tiles_kernel, rf_gather_kernel, rf_attn_kernel
            "breakdown_ms": {"arm": arm_ms, "block_mask": mask_ms, "sparse_attn_call": sparse_ms, "reorder": reorder_ms,
                             "attn_kernel": attn_kernel_ms, "dense_attn_call": dense_ms},
            "breakdown_ms_median": {n: float(np.median(x)) for n, x in stages.items()},
            "breakdown_ms_min": {n: float(np.min(x)) for n, x in stages.items()},
            "arm_overhead_pct": 100.0 * arm_ms / sparse_ms,
            "arm_plus_mask_overhead_pct": 100.0 * (arm_ms + mask_ms) / sparse_ms,
            "head_classes": {"spatial": int((cls == 0).sum()), "temporal": int((cls == 1).sum()),
                             "textural": int((cls == 2).sum())},
            "recall_mean_by_class": {name: [float(x) for x in rec[cls == c].mean(axis=0)] if (cls == c).any() else None
                                     for c, name in ((0, "spatial"), (1, "temporal"), (2, "textural"))},
            "tile_density": listed / float(wl.B * wl.H * sched.nQ * sched.nKmax),
            "computed_tile_tflops": achieved,
            "dense_equiv_tflops_attn_call": dflops / (sparse_ms * 1e-3) / 1e12,
            "dense_baseline_tflops": (dflops / (dense_ms * 1e-3) / 1e12) if dense_ms else None,
            "roofline": {"kernel": "rf_attn_kernel", "bound": "tensor", "achieved": achieved, "peak": pk["bf16_sustained"],
                         "unit": "TFLOP/s", "frac": achieved / pk["bf16_sustained"], "traffic": ATTN_DRAM_BYTES.get(wl.name),
                         "traffic_unit": "bytes per launch (ncu, dram read + write)",
                         "algorithmic_bytes_per_launch": 4 * wl.B * wl.H * wl.N * wl.D * 2,
                         "traffic_source": TRAFFIC_SOURCE if ATTN_DRAM_BYTES.get(wl.name) else None,
                         "peak_kind": f"bf16 sustained, of {pk['source']}", "frac_of_burst": achieved / pk["bf16_burst"],
                         "frac_of_nominal": achieved / NOMINAL_BF16_TFLOPS,
                         "nominal_peak": f"{NOMINAL_BF16_TFLOPS:.0f} TFLOP/s, NVIDIA's dense bf16 figure for one B200",
                         "algorithmic_flops_per_launch": tile_flops},
        }
        # The second pipe the kernel leans on: one exponential per score, 16 ex2 per SM and clock (the MUFU pipe: four
        # lanes per SM sub-partition).  4 * D flops go with every exponential, so at D = 64 this roof, not the tensor
        # pipe, is the lower one (1191 TFLOP/s at the maximum clock against 2383 at D = 128, where the two meet).
        sms = torch.cuda.get_device_properties(dev).multi_processor_count
        exps = 128.0 * 128.0 * listed
        exp_peak = 16.0 * sms * ((clocks or {}).get("sm_max_mhz") or 1965.0) * 1e6
        line["roofline"]["exp2"] = {"per_launch": exps, "achieved_per_s": exps / (attn_kernel_ms * 1e-3),
                                    "peak_per_s": exp_peak, "frac": exps / (attn_kernel_ms * 1e-3) / exp_peak,
                                    "peak_kind": "16 ex2 per SM per clock at the maximum SM clock",
                                    "flops_per_exp": 4 * wl.D,
                                    "roof_tflops": exp_peak * 4 * wl.D / 1e12}
        # the small kernels against the HBM roofline (algorithmic bytes / measured time)
        nS, nT, nX = (int((cls == c).sum()) for c in (0, 1, 2))
        head_bytes = wl.N * wl.D * 2
        n_glb = -(-wl.Nv // wl.sample_stride)
        arm_bytes = wl.B * wl.H * 2 * (n_glb + (wl.S if wl.sample_mode == 0 else 0)) * wl.D * 2
        mask_bytes = 4 * listed + 4 * wl.B * wl.H * sched.nQ
        kept = sum(-(-(wl.frame_h - r) // wl.textural_stride) * -(-(wl.frame_w - r) // wl.textural_stride)
                   for r in range(min(wl.textural_stride, wl.frame_h, wl.frame_w)))
        tex_rows = wl.T * kept + wl.L_text
        reorder_bytes = nT * 3 * 2 * head_bytes + nX * 2 * (head_bytes + tex_rows * wl.D * 2)
        line["aux_kernels"] = {
            name: {"ms": ms, "algorithmic_bytes": int(nbytes), "achieved_gbs": nbytes / (ms * 1e-3) / 1e9,
                   "frac_of_hbm_peak": nbytes / (ms * 1e-3) / 1e9 / pk["hbm_gbs"], "bound": bound}
            for name, ms, nbytes, bound in (
                ("rf_arm_classify", arm_ms, arm_bytes, "exponentials / tensor (n/2 flop per byte), not HBM"),
                ("rf_build_block_mask", mask_ms, mask_bytes, "latency (closed-form integer work, 4 B per listed tile)"),
                ("rf_reorder_tokens", reorder_ms, reorder_bytes, "hbm"))}
        if not args.no_cpu:
            dt, fl, nrows = oracle_sample(wl, args.ref_rows)
            line["cpu_baseline"] = {"value": fl / dt / 1e12, "unit": UNIT, "cores": threads_used(), "kind": "oracle",
                                    "sample": f"head 0: ARM + masked attention on {nrows} of {wl.N} query rows, "
                                              f"{dt:.1f} s, extrapolated by rows"}
        print(json.dumps(line))
    dist_util.shutdown()


def run_stub(args, wl):
    """The rank bookkeeping of the CUDA arm without a GPU (used by the CPU tests of the N > 1 path): gloo
    backend, a step that only sleeps, the same barrier / max-over-ranks / replica-throughput arithmetic and
    the same "rank 0 prints one line" rule.  Nothing of the method runs here and no number it prints is a
    measurement."""
    from paper_2505_21036_b200 import dist_util
    rank, world, _ = dist_util.env_rank()
    dist_util.init("gloo")
    dist_util.barrier()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        time.sleep(0.01 * (1 + rank))
    ms = 1e3 * (time.perf_counter() - t0) / args.steps
    dist_util.barrier()
    (ms_max,) = dist_util.max_over_ranks([ms])
    if rank == 0:
        print(json.dumps({"impl": "stub", "metric": METRIC, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                          "warmup": args.warmup, "ms_per_step": ms_max, "scaling": "weak",
                          "value": dist_util.replica_throughput(dense_flops(wl), ms_max, world) / 1e12,
                          "config": {"workload": wl.name, "parallelism": f"replicas x{world}"}}))
    dist_util.shutdown()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--workload", default="hunyuan720p", choices=sorted(synth.WORKLOADS))
    ap.add_argument("--ref-rows", type=int, default=4096, help="query rows per oracle sample (about 10-20 s of CPU work)")
    ap.add_argument("--e2e-groups", type=int, default=0, help="head groups of the host-staged leg (0: automatic)")
    ap.add_argument("--no-cpu", action="store_true", help="skip the cpu_baseline leg")
    ap.add_argument("--no-dense", dest="dense", action="store_false", help="skip the dense-baseline timing")
    ap.add_argument("--stub", action="store_true", help=argparse.SUPPRESS)   # CPU test of the N > 1 bookkeeping
    args = ap.parse_args()
    wl = synth.WORKLOADS[args.workload]
    if args.impl == "reference":
        run_reference(args, wl)                    # rank 0 alone works; started bare, this process is rank 0
        return
    from paper_2505_21036_b200 import dist_util
    if args.gpus > 1 and not dist_util.launched_by_torchrun():
        # started bare: become the launcher of N independent replicas, one process per GPU
        sys.exit(dist_util.spawn_replicas([sys.executable, os.path.abspath(__file__)] + sys.argv[1:], args.gpus))
    _, world, _ = dist_util.env_rank()
    if world != args.gpus:
        raise SystemExit(f"bench.py: --gpus {args.gpus} but WORLD_SIZE={world}")
    if args.stub:
        run_stub(args, wl)
    else:
        run_cuda(args, wl)


if __name__ == "__main__":
    main()
