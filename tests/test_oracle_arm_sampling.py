"""Pins for WHICH sample feeds WHICH recall in the oracle's ARM (Sec. 3.3, Algorithm 1) and for the
bandwidth -> window rounding (Sec. 4.1).  CPU only.

Algorithm 1 measures the Temporal mask's recall on the local sample (the first frame's tokens) and the
Spatial mask's recall on the global sample (every omega-th video token); the ablation of Table 2 uses the
global sample for both.  The checks below rebuild both recalls without any oracle code: the sampled
tokens are sliced by hand, the restricted masks come from nested loops over the one-line definitions, and
the softmax is torch's scaled_dot_product_attention in fp64 (values = the transposed mask, so that the
diagonal of the output is each row's kept mass).  A wiring mistake (Temporal recall taken from the stride
sample, Spatial recall from the first frame, the two swapped) fails them, and so does a planted case
whose position-local structure exists in the first frame only."""
import math

import numpy as np
import pytest
import torch

from oracle import rainfusion_oracle as orc
from oracle.rainfusion_oracle import SPATIAL, TEMPORAL, TEXTURAL, Geometry, PatternParams
from paper_2505_21036_b200 import synth


def rand_bits(rng, n, d, scale=1.0):
    return synth.f32_to_bf16_bits(rng.standard_normal((n, d)).astype(np.float32) * np.float32(scale))


def f64(bits):
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def recall_by_library(q_bits, k_bits, tokens, kept):
    """Mean over sampled rows of the softmax mass on kept keys, via torch SDPA: with V = kept^T the output's
    diagonal entry r is sum_j P[r, j] * kept[r, j]."""
    q = torch.from_numpy(f64(q_bits[tokens]))[None]
    k = torch.from_numpy(f64(k_bits[tokens]))[None]
    v = torch.from_numpy(np.ascontiguousarray(kept.T.astype(np.float64)))[None]
    out = torch.nn.functional.scaled_dot_product_attention(q, k, v)[0].numpy()
    return float(np.diag(out).mean())


def temporal_kept_by_loops(tokens, S, ws):
    n = len(tokens)
    kept = np.zeros((n, n), dtype=bool)
    for a in range(n):
        for b in range(n):
            kept[a, b] = abs(tokens[a] % S - tokens[b] % S) <= ws
    return kept


def spatial_kept_by_loops(tokens, S, wf):
    n = len(tokens)
    kept = np.zeros((n, n), dtype=bool)
    for a in range(n):
        for b in range(n):
            kept[a, b] = abs(tokens[a] // S - tokens[b] // S) <= wf
    return kept


G = Geometry(5, 4, 6, 7)          # S = 24, Nv = 120
PP = PatternParams(1, 3, 2)
OMEGA = 5                          # does not divide S: the stride sample hits different positions in every frame


@pytest.fixture(scope="module")
def qk():
    rng = np.random.default_rng(20250521)
    # a shared per-position component, stronger in the first frame, so that the two samples give clearly
    # different Temporal recalls
    q = rng.standard_normal((G.N, 32)).astype(np.float32)
    k = rng.standard_normal((G.N, 32)).astype(np.float32)
    pos = rng.standard_normal((G.S, 32)).astype(np.float32)
    for f in range(G.T):
        q[f * G.S:(f + 1) * G.S] += pos * np.float32(1.4 if f == 0 else 0.5)
        k[f * G.S:(f + 1) * G.S] += pos * np.float32(1.4 if f == 0 else 0.5)
    return synth.f32_to_bf16_bits(q), synth.f32_to_bf16_bits(k)


def test_algorithm1_wiring_local_sample_feeds_temporal_global_sample_feeds_spatial(qk):
    q, k = qk
    first_frame = list(range(G.S))
    strided = list(range(0, G.Nv, OMEGA))
    Rt_loc = recall_by_library(q, k, first_frame, temporal_kept_by_loops(first_frame, G.S, PP.spatial_window))
    Rt_glb = recall_by_library(q, k, strided, temporal_kept_by_loops(strided, G.S, PP.spatial_window))
    Rs_glb = recall_by_library(q, k, strided, spatial_kept_by_loops(strided, G.S, PP.frame_window))
    # the three quantities are well apart, so a swap cannot hide inside the tolerance
    assert abs(Rt_loc - Rt_glb) > 0.02 and abs(Rt_loc - Rs_glb) > 0.02 and abs(Rt_glb - Rs_glb) > 0.02
    _, (rt, rs, _), _ = orc.arm_head(q, k, G, PP, orc.SAMPLE_ALG1, OMEGA, 0.9)
    assert rt == pytest.approx(Rt_loc, abs=1e-12)
    assert rs == pytest.approx(Rs_glb, abs=1e-12)
    _, (rt, rs, _), _ = orc.arm_head(q, k, G, PP, orc.SAMPLE_GLOBAL, OMEGA, 0.9)
    assert rt == pytest.approx(Rt_glb, abs=1e-12)
    assert rs == pytest.approx(Rs_glb, abs=1e-12)


def test_textural_recall_is_measured_on_the_global_sample(qk):
    q, k = qk
    strided = list(range(0, G.Nv, OMEGA))
    n = len(strided)
    kept = np.zeros((n, n), dtype=bool)
    for b, tok in enumerate(strided):
        p = tok % G.S
        kept[:, b] = (p // G.frame_w) % PP.textural_stride == (p % G.frame_w) % PP.textural_stride
    expect = recall_by_library(q, k, strided, kept)
    for mode in (orc.SAMPLE_ALG1, orc.SAMPLE_GLOBAL):
        _, (_, _, rte), _ = orc.arm_head(q, k, G, PP, mode, OMEGA, 0.9)
        assert rte == pytest.approx(expect, abs=1e-12)


def test_dynamic_bandwidth_wiring_per_candidate(qk):
    q, k = qk
    first_frame = list(range(G.S))
    strided = list(range(0, G.Nv, OMEGA))
    bws = [0.2, 0.45, 0.7]
    # windows by hand: floor(b * T) frames, floor(b * S) positions
    hand = {0.2: (1, 4), 0.45: (2, 10), 0.7: (3, 16)}
    for mode, t_tokens in ((orc.SAMPLE_ALG1, first_frame), (orc.SAMPLE_GLOBAL, strided)):
        _, _, _, Rt, Rs = orc.arm_head_plus(q, k, G, bws, 2, mode, OMEGA, 0.9)
        for i, b in enumerate(bws):
            wf, ws = hand[b]
            assert Rt[i] == pytest.approx(recall_by_library(q, k, t_tokens, temporal_kept_by_loops(t_tokens, G.S, ws)), abs=1e-12)
            assert Rs[i] == pytest.approx(recall_by_library(q, k, strided, spatial_kept_by_loops(strided, G.S, wf)), abs=1e-12)


def first_frame_only_position_structure(g, d=32, amp=3.0, seed=5):
    """Frame 0: query and key of position p share one strong random vector (a query's mass sits on its own
    position).  Frames >= 1: iid N(0,1), no structure at all."""
    rng = np.random.default_rng(seed)
    q = rng.standard_normal((g.N, d)).astype(np.float32)
    k = rng.standard_normal((g.N, d)).astype(np.float32)
    v = rng.standard_normal((g.S, d)).astype(np.float32) * np.float32(amp)
    q[:g.S] = v
    k[:g.S] = v
    return synth.f32_to_bf16_bits(q), synth.f32_to_bf16_bits(k)


def test_structure_planted_in_the_first_frame_only_is_seen_by_algorithm1_and_missed_by_global_sampling():
    g = Geometry(6, 6, 6, 4)
    pp = PatternParams(1, 1, 2)
    q, k = first_frame_only_position_structure(g)
    cls, (rt, rs, _), _ = orc.arm_head(q, k, g, pp, orc.SAMPLE_ALG1, 6, 0.9)
    assert cls == TEMPORAL and rt > 0.999
    cls_g, (rt_g, rs_g, _), _ = orc.arm_head(q, k, g, pp, orc.SAMPLE_GLOBAL, 6, 0.9)
    assert cls_g != TEMPORAL and rt_g < 0.5
    assert rs == rs_g                                         # the Spatial recall is the global one in both modes
    # the same through the dynamic-bandwidth path: the narrowest candidate already qualifies on the local sample
    cls_p, idx, window, Rt, _ = orc.arm_head_plus(q, k, g, [0.05, 0.5], 2, orc.SAMPLE_ALG1, 6, 0.9)
    assert (cls_p, idx, window) == (TEMPORAL, 0, 1) and Rt[0] > 0.999
    cls_p, _, _, Rt, _ = orc.arm_head_plus(q, k, g, [0.05, 0.5], 2, orc.SAMPLE_GLOBAL, 6, 0.9)
    assert cls_p != TEMPORAL and Rt[0] < 0.5


def test_spatial_recall_never_comes_from_the_first_frame():
    """On the first frame alone every pair is within the frame window, so a Spatial recall taken there
    would be exactly 1 whatever the head does.  Frame-free iid inputs must give the mask's density instead."""
    g = Geometry(8, 3, 4, 0)
    pp = PatternParams(1, 2, 2)
    z = np.zeros((g.N, 16), dtype=np.uint16)                  # Q = 0: uniform softmax, recall = mask density
    rng = np.random.default_rng(9)
    k = rand_bits(rng, g.N, 16)
    _, (rt, rs, _), _ = orc.arm_head(z, k, g, pp, orc.SAMPLE_ALG1, 3, 0.9)
    # stride 3 on S = 12: four samples per frame, 8 frames; frame band of half-width 1: (8*3 - 2)/64 of frame pairs
    assert rs == pytest.approx(22 / 64, abs=1e-13)
    # first frame, 12 positions, position band of half-width 2: (12*5 - 6)/144
    assert rt == pytest.approx(54 / 144, abs=1e-13)


@pytest.mark.parametrize("b,T,fh,fw,expect", [
    (0.13, 13, 30, 45, (1, 175)),     # 0.13 * 1350 = 175.5: floor, not round-half-up or round-half-even (176)
    (0.18, 13, 30, 45, (2, 243)),     # 2.34 and 243.0
    (0.125, 13, 30, 45, (1, 168)),    # 1.625 -> 1 (rounding would give 2), 168.75 -> 168 (rounding: 169)
    (0.7, 5, 4, 6, (3, 16)),          # 3.5 -> 3 (round-half-even would give 4), 16.8 -> 16
    (0.25, 33, 45, 80, (8, 900)),
    (1.0, 7, 3, 5, (7, 15)),
])
def test_bandwidth_to_window_takes_the_floor(b, T, fh, fw, expect):
    assert orc.windows_of(b, Geometry(T, fh, fw, 0)) == expect


def test_spatial_recall_with_the_first_frame_as_key_frame(qk):
    """Option of Sec. 3.2's "adjacent or key frames": the sampled Spatial mask also keeps the sampled keys of frame 0;
    the Temporal recall does not change."""
    q, k = qk
    strided = list(range(0, G.Nv, OMEGA))
    n = len(strided)
    kept = np.zeros((n, n), dtype=bool)
    for a in range(n):
        for b in range(n):
            kept[a, b] = abs(strided[a] // G.S - strided[b] // G.S) <= PP.frame_window or strided[b] // G.S == 0
    expect = recall_by_library(q, k, strided, kept)
    pp_on = PatternParams(PP.frame_window, PP.spatial_window, PP.textural_stride, True)
    _, (rt_on, rs_on, _), _ = orc.arm_head(q, k, G, pp_on, orc.SAMPLE_ALG1, OMEGA, 0.9)
    _, (rt_off, rs_off, _), _ = orc.arm_head(q, k, G, PP, orc.SAMPLE_ALG1, OMEGA, 0.9)
    assert rs_on == pytest.approx(expect, abs=1e-12) and rs_on > rs_off + 1e-3 and rt_on == rt_off
    _, _, _, Rt, Rs = orc.arm_head_plus(q, k, G, [0.2, 0.45], 2, orc.SAMPLE_ALG1, OMEGA, 0.9, keep_first_frame=True)
    kept2 = np.zeros((n, n), dtype=bool)
    for a in range(n):
        for b in range(n):
            kept2[a, b] = abs(strided[a] // G.S - strided[b] // G.S) <= 2 or strided[b] // G.S == 0     # floor(0.45 * 5) = 2
    assert Rs[0] == pytest.approx(expect, abs=1e-12)                                                  # floor(0.2 * 5) = 1 = PP's window
    assert Rs[1] == pytest.approx(recall_by_library(q, k, strided, kept2), abs=1e-12)


def test_temporal_recall_with_a_2d_window(qk):
    """The 2-D reading of the Temporal locality on both samples, rebuilt with loops and the library softmax."""
    q, k = qk
    wy, wx = 1, 2
    pp2 = PatternParams(PP.frame_window, PP.spatial_window, PP.textural_stride, False, (wy, wx))

    def kept_of(tokens):
        n = len(tokens)
        kept = np.zeros((n, n), dtype=bool)
        for a in range(n):
            for b in range(n):
                pa, pb = tokens[a] % G.S, tokens[b] % G.S
                kept[a, b] = abs(pa // G.frame_w - pb // G.frame_w) <= wy and abs(pa % G.frame_w - pb % G.frame_w) <= wx
        return kept

    first_frame = list(range(G.S))
    strided = list(range(0, G.Nv, OMEGA))
    _, (rt, rs, _), _ = orc.arm_head(q, k, G, pp2, orc.SAMPLE_ALG1, OMEGA, 0.9)
    assert rt == pytest.approx(recall_by_library(q, k, first_frame, kept_of(first_frame)), abs=1e-12)
    _, (rt_g, rs_g, _), _ = orc.arm_head(q, k, G, pp2, orc.SAMPLE_GLOBAL, OMEGA, 0.9)
    assert rt_g == pytest.approx(recall_by_library(q, k, strided, kept_of(strided)), abs=1e-12)
    _, (_, rs_plain, _), _ = orc.arm_head(q, k, G, PP, orc.SAMPLE_ALG1, OMEGA, 0.9)
    assert rs == rs_g == rs_plain                      # the Spatial recall does not depend on it
