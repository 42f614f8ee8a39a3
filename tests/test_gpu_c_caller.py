"""The library driven from plain C (paper_2505_21036_b200/examples/rf_c_caller.c: CUDA runtime, no Python, no torch in
the process): compiled with gcc, run as a child process, its classes, recalls and output checked against the oracle
on inputs rebuilt bit for bit from the example's generator."""
import os
import shutil
import subprocess

import numpy as np
import pytest

from oracle import rainfusion_oracle as orc
from paper_2505_21036_b200 import api, synth

import gpu_util as gu

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def lcg_bf16(n, seed, scale):
    """The example's fill(): a 32-bit LCG, its top 16 bits as a value in [-1, 1), times scale, rounded to bf16."""
    state, raw = seed, np.empty(n, dtype=np.int64)
    for i in range(n):
        state = (state * 1664525 + 1013904223) & 0xFFFFFFFF
        raw[i] = state >> 16
    x = (raw.astype(np.float32) - np.float32(32768.0)) * np.float32(1.0 / 32768.0) * np.float32(scale)
    return synth.f32_to_bf16_bits(x)


def test_c_caller_matches_the_oracle(tmp_path):
    if shutil.which("gcc") is None:
        pytest.skip("no gcc")
    cuda = os.environ.get("CUDA_HOME", "/usr/local/cuda")
    libdir, exe, out = os.path.dirname(api.lib_path()), str(tmp_path / "rf_c_caller"), str(tmp_path / "o.bin")
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Wextra", "-Werror", "-I", os.path.join(ROOT, "include"),
                    "-I", os.path.join(cuda, "include"),
                    os.path.join(ROOT, "paper_2505_21036_b200", "examples", "rf_c_caller.c"), "-o", exe,
                    "-L", libdir, "-l:" + os.path.basename(api.lib_path()), "-L", os.path.join(cuda, "lib64"), "-lcudart",
                    "-Wl,-rpath," + libdir], check=True, capture_output=True, text=True)
    res = subprocess.run([exe, out], capture_output=True, text=True, timeout=300)
    assert res.returncode == 0, res.stdout + res.stderr
    lines = res.stdout.strip().splitlines()
    assert lines[0] == "status 0"
    H, D, T, fh, fw, L = 3, 64, 5, 6, 7, 3
    g = orc.Geometry(T, fh, fw, L)
    pp = orc.PatternParams(1, 10, 2)
    N = g.N
    q, k, v = (lcg_bf16(H * N * D, seed, scale).reshape(H, N, D) for seed, scale in ((1, 2.0), (2, 2.0), (3, 1.0)))
    O = np.fromfile(out, dtype=np.uint16).reshape(H, N, D)
    O = synth.bf16_bits_to_f32(O).astype(np.float64)
    for h in range(H):
        f = lines[1 + h].split()
        cls_c, rec_c = int(f[3]), np.array([float(f[5]), float(f[7]), float(f[9])])
        cls, rec, margin = orc.arm_head(q[h], k[h], g, pp, orc.SAMPLE_ALG1, 4, 0.9)
        assert np.abs(rec_c - np.asarray(rec)).max() <= gu.RECALL_ABS + 1e-6, (h, rec_c, rec)     # six printed decimals
        if margin > gu.TIE_MARGIN:
            assert cls_c == cls, h
        Or, _ = orc.masked_attention(q[h], k[h], v[h], cls_c, g, pp)
        err = np.abs(O[h] - Or)
        assert np.isfinite(O[h]).all() and err.max() <= gu.O_MAX_ABS and err.mean() <= gu.O_MEAN_ABS, (h, err.max(), err.mean())
