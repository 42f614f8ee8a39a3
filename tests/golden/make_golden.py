"""Writes tests/golden/tiny_expected.json from the CPU oracle alone (never from the CUDA path).

  python tests/golden/make_golden.py

Stored: for the tiny workload, ARM recalls and classes per head, every tile list of every pattern
(128 x 128 tiles, Temporal permutation on and off), kv_len per pattern, and the attention output and lse
of each head under its oracle class on a few query rows.  The file pins the oracle against silent drift
and gives the GPU tests expected values that do not depend on running the oracle at test time.
"""
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import rainfusion_oracle as orc          # noqa: E402
from paper_2505_21036_b200 import synth              # noqa: E402  (seeded inputs only)

ROWS = [0, 63, 64, 127, 128, 200, 255, 256, 263, 271]


def main():
    wl = synth.WORKLOADS["tiny"]
    g = orc.Geometry(wl.T, wl.frame_h, wl.frame_w, wl.L_text)
    pp = orc.PatternParams(wl.frame_window, wl.spatial_window, wl.textural_stride)
    q, k, v = synth.make_qkv(wl)
    cls, rec, margin = orc.arm_classify(q, k, g, pp, wl.sample_mode, wl.sample_stride, wl.alpha)
    out = {"workload": "tiny", "classes": cls[0].tolist(), "recall": rec[0].tolist(), "margin": margin[0].tolist(),
           "rows": ROWS, "tile_lists": {}, "kv_len": {}, "attention": []}
    for pat in (orc.SPATIAL, orc.TEMPORAL, orc.TEXTURAL, orc.DENSE):
        out["kv_len"][str(pat)] = orc.kv_len(pat, g, pp)
        for perm in (0, 1):
            out["tile_lists"][f"{pat}/{perm}"] = [orc.tile_row(pat, g, pp, bool(perm), 128, 128, a) for a in range(3)]
    for h in range(wl.H):
        O, lse = orc.masked_attention(q[0, h], k[0, h], v[0, h], int(cls[0, h]), g, pp, rows=ROWS)
        out["attention"].append({"O": np.round(O, 10).tolist(), "lse": np.round(lse, 10).tolist()})
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "tiny_expected.json")
    with open(path, "w") as f:
        json.dump(out, f)
    print(path, os.path.getsize(path), "bytes")


if __name__ == "__main__":
    main()
