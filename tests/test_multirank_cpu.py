"""The N > 1 bookkeeping of bench.py on CPU: two gloo ranks, max-over-ranks timing, replica throughput,
and the reference arm's "rank 0 only" rule."""
import json
import os
import socket
import subprocess
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    sys.path.insert(0, ROOT)
    from paper_2505_21036_b200 import dist_util
    r, w = dist_util.init("gloo")
    dist_util.barrier()
    ms = [10.0 + 5.0 * rank, 100.0 - rank]           # rank 1 is slower on the first, faster on the second
    mx = dist_util.max_over_ranks(ms)
    out.put((rank, r, w, mx, dist_util.replica_throughput(1e3, mx[0], w)))
    dist_util.barrier()
    dist_util.shutdown()


def test_two_gloo_ranks_take_the_max_and_sum_the_replicas():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, r, w, mx, thr in res:
        assert (r, w) == (rank, 2)
        assert mx == [15.0, 100.0]
        assert abs(thr - 2 * 1e3 / 15e-3) < 1e-6


def test_bare_bench_command_with_gpus_2_starts_two_replicas():
    """`python bench.py --gpus 2` without a launcher spawns its own two ranks (gloo and a stub step here): rank 0
    prints one line whose n_gpus is 2 and whose time is the slower rank's."""
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--stub", "--workload", "tiny",
                        "--steps", "3", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr
    lines = [l for l in r.stdout.strip().splitlines() if l.startswith("{")]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["n_gpus"] == 2 and line["config"]["parallelism"] == "replicas x2"
    assert line["ms_per_step"] >= 19.0             # rank 1 sleeps 20 ms per step, rank 0 only 10
    # under a launcher (WORLD_SIZE set) a mismatching --gpus is an error, not a silent single replica
    env2 = dict(env, RANK="0", WORLD_SIZE="1", LOCAL_RANK="0")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--stub", "--workload", "tiny"],
                       env=env2, capture_output=True, text=True, timeout=300)
    assert r.returncode != 0 and "WORLD_SIZE" in r.stderr


def test_a_failing_rank_ends_the_launcher_with_its_code():
    sys.path.insert(0, ROOT)
    from paper_2505_21036_b200 import dist_util
    prog = "import os, sys, time; r = int(os.environ['RANK']); sys.exit(7) if r == 1 else time.sleep(60)"
    import time
    t0 = time.time()
    assert dist_util.spawn_replicas([sys.executable, "-c", prog], 2) == 7
    assert time.time() - t0 < 30.0                  # rank 0 was not left sleeping


def test_single_rank_is_identity():
    sys.path.insert(0, ROOT)
    from paper_2505_21036_b200 import dist_util
    assert dist_util.max_over_ranks([3.0, 4.0]) == [3.0, 4.0]
    assert dist_util.replica_throughput(2.0, 1000.0, 1) == 2.0


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--workload", "tiny", "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True,
                       timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env["RANK"] = "0"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--workload", "tiny", "--steps", "1", "--warmup", "0", "--ref-rows", "32"], env=env,
                       capture_output=True, text=True, timeout=300)
    assert r.returncode == 0
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle" and line["n_gpus"] == 2
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0
