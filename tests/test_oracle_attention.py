"""Pins for the oracle's ARM recall / decision and masked attention (CPU only).

torch's scaled_dot_product_attention (fp64, CPU) is the independent library routine the
oracle's numpy softmax-attention is held against; the rest are closed forms and invariants."""
import math

import numpy as np
import pytest
import torch

from oracle import rainfusion_oracle as orc
from oracle.rainfusion_oracle import DENSE, SPATIAL, TEMPORAL, TEXTURAL, Geometry, PatternParams
from paper_2505_21036_b200 import synth


def rand_bits(rng, n, d, scale=1.0):
    return synth.f32_to_bf16_bits(rng.standard_normal((n, d)).astype(np.float32) * np.float32(scale))


def sdpa(q_bits, k_bits, v_bits, mask=None):
    q = torch.from_numpy(orc.bf16_to_f64(q_bits))[None]
    k = torch.from_numpy(orc.bf16_to_f64(k_bits))[None]
    v = torch.from_numpy(orc.bf16_to_f64(v_bits))[None]
    m = None if mask is None else torch.from_numpy(mask)[None]
    return torch.nn.functional.scaled_dot_product_attention(q, k, v, attn_mask=m)[0].numpy()


G = Geometry(4, 4, 5, 6)
PP = PatternParams(1, 3, 2)


@pytest.fixture(scope="module")
def qkv():
    rng = np.random.default_rng(7)
    return rand_bits(rng, G.N, 32), rand_bits(rng, G.N, 32), rand_bits(rng, G.N, 32)


def test_bf16_widening_is_exact():
    bits = np.arange(0, 0x7F80, 37, dtype=np.uint16)          # finite positive bf16 values
    t = torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(orc.bf16_to_f64(bits), t)


def test_all_ones_mask_is_naive_dense_attention(qkv):
    q, k, v = qkv
    O, lse = orc.masked_attention(q, k, v, DENSE, G, PP)
    assert np.allclose(O, sdpa(q, k, v), atol=1e-12)
    s = orc.bf16_to_f64(q) @ orc.bf16_to_f64(k).T / math.sqrt(q.shape[1])
    assert np.allclose(lse, torch.logsumexp(torch.from_numpy(s), dim=1).numpy(), atol=1e-12)


@pytest.mark.parametrize("pattern", [SPATIAL, TEMPORAL, TEXTURAL])
def test_masked_attention_matches_library_with_explicit_mask(qkv, pattern):
    q, k, v = qkv
    idx = np.arange(G.N)
    M = orc.keep_mask(pattern, idx, idx, G, PP)
    O, _ = orc.masked_attention(q, k, v, pattern, G, PP, chunk=7)
    assert np.allclose(O, sdpa(q, k, v, M), atol=1e-12)


def test_probability_rows_sum_to_one_and_lse_is_consistent(qkv):
    q, k, v = qkv
    ones = synth.f32_to_bf16_bits(np.ones((G.N, 8), dtype=np.float32))
    for pattern in (SPATIAL, TEMPORAL, TEXTURAL, DENSE):
        O, lse = orc.masked_attention(q, k, ones, pattern, G, PP)
        assert np.allclose(O, 1.0, atol=1e-13)          # V == 1  =>  O == sum of probabilities
        idx = np.arange(G.N)
        s = orc.bf16_to_f64(q) @ orc.bf16_to_f64(k).T / math.sqrt(q.shape[1])
        s[~orc.keep_mask(pattern, idx, idx, G, PP)] = -np.inf
        assert np.allclose(np.exp(s - lse[:, None]).sum(axis=1), 1.0, atol=1e-12)


def test_one_key_per_row_returns_that_value(qkv):
    # w_f = 0 with one-token frames and no text: every query sees exactly its own key
    g = Geometry(9, 1, 1, 0)
    rng = np.random.default_rng(3)
    q, k, v = rand_bits(rng, g.N, 16), rand_bits(rng, g.N, 16), rand_bits(rng, g.N, 16)
    O, lse = orc.masked_attention(q, k, v, SPATIAL, g, PatternParams(0, 0, 2))
    assert np.allclose(O, orc.bf16_to_f64(v), atol=1e-14)
    diag = (orc.bf16_to_f64(q) * orc.bf16_to_f64(k)).sum(axis=1) / 4.0
    assert np.allclose(lse, diag, atol=1e-12)


def test_textural_equals_dense_attention_on_gathered_keys(qkv):
    q, k, v = qkv
    kept = orc.key_order(TEXTURAL, G, PP, False)
    O, _ = orc.masked_attention(q, k, v, TEXTURAL, G, PP)
    assert np.allclose(O, sdpa(q, k[kept], v[kept]), atol=1e-12)


def test_spatial_window_zero_is_per_frame_attention():
    g = Geometry(3, 3, 4, 0)
    rng = np.random.default_rng(5)
    q, k, v = rand_bits(rng, g.N, 16), rand_bits(rng, g.N, 16), rand_bits(rng, g.N, 16)
    O, _ = orc.masked_attention(q, k, v, SPATIAL, g, PatternParams(0, 0, 2))
    for f in range(g.T):
        sl = slice(f * g.S, (f + 1) * g.S)
        assert np.allclose(O[sl], sdpa(q[sl], k[sl], v[sl]), atol=1e-12)


def test_temporal_window_zero_is_per_position_attention():
    g = Geometry(5, 2, 3, 0)
    rng = np.random.default_rng(6)
    q, k, v = rand_bits(rng, g.N, 16), rand_bits(rng, g.N, 16), rand_bits(rng, g.N, 16)
    O, _ = orc.masked_attention(q, k, v, TEMPORAL, g, PatternParams(0, 0, 2))
    for p in range(g.S):
        sl = slice(p, g.N, g.S)
        assert np.allclose(O[sl], sdpa(q[sl], k[sl], v[sl]), atol=1e-12)


def test_joint_permutation_of_keys_and_values_inside_a_frame_cell(qkv):
    # Spatial mask depends on the key's frame only: shuffling keys+values within each frame changes nothing
    q, k, v = qkv
    rng = np.random.default_rng(11)
    perm = np.arange(G.N)
    for f in range(G.T):
        perm[f * G.S:(f + 1) * G.S] = f * G.S + rng.permutation(G.S)
    O1, l1 = orc.masked_attention(q, k, v, SPATIAL, G, PP)
    O2, l2 = orc.masked_attention(q, k[perm], v[perm], SPATIAL, G, PP)
    assert np.allclose(O1, O2, atol=1e-12) and np.allclose(l1, l2, atol=1e-12)


def test_row_subset_equals_full(qkv):
    q, k, v = qkv
    rows = [0, 5, G.Nv - 1, G.Nv, G.N - 1]
    O, lse = orc.masked_attention(q, k, v, TEMPORAL, G, PP)
    Os, ls = orc.masked_attention(q, k, v, TEMPORAL, G, PP, rows=rows)
    assert np.array_equal(O[rows], Os) and np.array_equal(lse[rows], ls)


# ---------------------------------------------------------------- ARM

def test_sampling_index_sets():
    g = Geometry(4, 8, 8, 16)
    assert orc.local_sample(g).tolist() == list(range(64))
    assert orc.global_sample(g, 4).tolist() == list(range(0, 256, 4))
    assert len(orc.global_sample(Geometry(33, 45, 80, 256), 36)) == 3300
    assert orc.global_sample(Geometry(2, 1, 5, 3), 3).tolist() == [0, 3, 6, 9]   # never a text token


def test_local_sampling_cost_is_one_over_t_squared():
    g = Geometry(33, 45, 80, 256)
    assert len(orc.local_sample(g)) ** 2 * g.T ** 2 == g.Nv ** 2


def test_recall_full_empty_and_complement(qkv):
    q, k, _ = qkv
    I = orc.global_sample(G, 3)
    P = orc.approx_scores(q, k, I)
    assert np.allclose(P.sum(axis=1), 1.0, atol=1e-14)
    full = np.ones_like(P, dtype=bool)
    assert orc.recall(P, full) == pytest.approx(1.0, abs=1e-14)
    assert orc.recall(P, ~full) == 0.0
    M = orc.keep_mask(SPATIAL, I, I, G, PP)
    assert orc.recall(P, M) + orc.recall(P, ~M) == pytest.approx(1.0, abs=1e-13)


def test_recall_of_uniform_scores_is_mask_density():
    g = Geometry(6, 2, 3, 0)
    z = np.zeros((g.N, 16), dtype=np.uint16)           # Q' = 0  =>  uniform softmax
    rng = np.random.default_rng(2)
    k = rand_bits(rng, g.N, 16)
    I = orc.global_sample(g, 2)
    P = orc.approx_scores(z, k, I)
    M = orc.keep_mask(SPATIAL, I, I, g, PatternParams(1, 0, 2))
    assert orc.recall(P, M) == pytest.approx(M.mean(), abs=1e-14)
    # Spatial band of half-width 1 over 6 frames keeps (6*3 - 2)/36 of the frame pairs
    assert M.mean() == pytest.approx(16 / 36)


def test_recall_equals_dense_attention_on_indicator_values(qkv):
    # V[:, 0] = [key kept for this row's frame]: dense attention's output column is that row's recall
    q, k, _ = qkv
    I = orc.local_sample(G)
    M = orc.keep_mask(TEMPORAL, I, I, G, PP)
    P = orc.approx_scores(q, k, I)
    per_row = (P * M).sum(axis=1)
    for r in (0, 7, len(I) - 1):
        ind = synth.f32_to_bf16_bits(M[r].astype(np.float32)[:, None])
        out = sdpa(q[I][r:r + 1], k[I], ind)
        assert out[0, 0] == pytest.approx(per_row[r], abs=1e-13)


def test_recall_with_one_dominant_key():
    g = Geometry(4, 2, 2, 0)
    q = np.zeros((g.N, 8), dtype=np.float32)
    k = np.zeros((g.N, 8), dtype=np.float32)
    q[:, 0] = 16.0
    k[0, 0] = 16.0                                     # every query puts ~all mass on key 0 (frame 0)
    qb, kb = synth.f32_to_bf16_bits(q), synth.f32_to_bf16_bits(k)
    I = orc.global_sample(g, 1)
    P = orc.approx_scores(qb, kb, I)
    M = orc.keep_mask(SPATIAL, I, I, g, PatternParams(0, 0, 2))
    # rows of frame 0 keep key 0, rows of the other three frames lose it
    assert orc.recall(P, M) == pytest.approx(0.25, abs=1e-6)


@pytest.mark.parametrize("Rt,Rs,expect", [
    (0.95, 0.10, TEMPORAL), (0.95, 0.95, TEMPORAL), (0.10, 0.95, SPATIAL), (0.10, 0.10, TEXTURAL),
    (0.90, 0.00, TEMPORAL), (0.8999, 0.90, SPATIAL), (0.8999, 0.8999, TEXTURAL)])
def test_algorithm1_truth_table(Rt, Rs, expect):
    assert orc.decide(Rt, Rs, 0.9) == expect


def test_two_mask_ablation_never_picks_textural_and_agrees_with_algorithm1_elsewhere():
    """Table 2's rows without the Textural mask: same decision wherever Algorithm 1 picks Spatial or Temporal,
    the mask of larger recall (Temporal on equality) where it would have picked Textural."""
    grid = [i / 20.0 for i in range(21)]
    for alpha in (0.5, 0.9, 1.0):
        for Rt in grid:
            for Rs in grid:
                three, two = orc.decide(Rt, Rs, alpha), orc.decide(Rt, Rs, alpha, two_mask=True)
                assert two in (TEMPORAL, SPATIAL)
                if three != TEXTURAL:
                    assert two == three
                else:
                    assert two == (TEMPORAL if Rt >= Rs else SPATIAL)
    assert orc.decide_plus([0.1, 0.2, 0.3], [0.2, 0.3, 0.25], 0.9, two_mask=True) == (TEMPORAL, 2)
    assert orc.decide_plus([0.1, 0.2, 0.3], [0.2, 0.3, 0.35], 0.9, two_mask=True) == (SPATIAL, 2)
    assert orc.decide_plus([0.1, 0.95, 0.99], [0.2, 0.3, 0.35], 0.9, two_mask=True) == (TEMPORAL, 1)
    assert orc.decide_plus([0.1, 0.2, 0.3], [0.2, 0.3, 0.35], 0.9) == (TEXTURAL, -1)
    assert orc.decision_margin(0.5, 0.52, 0.9, two_mask=True) == pytest.approx(0.02)
    assert orc.decision_margin(0.5, 0.93, 0.9, two_mask=True) == pytest.approx(0.03)


def test_margin():
    assert orc.decision_margin(0.95, 0.2, 0.9) == pytest.approx(0.05)
    assert orc.decision_margin(0.5, 0.93, 0.9) == pytest.approx(0.03)
    assert orc.decision_margin(0.895, 0.2, 0.9) == pytest.approx(0.005)


def test_planted_heads_of_tiny_config_pick_their_patterns():
    wl = synth.WORKLOADS["tiny"]
    q, k, _ = synth.make_qkv(wl)
    g = Geometry(wl.T, wl.frame_h, wl.frame_w, wl.L_text)
    pp = PatternParams(wl.frame_window, wl.spatial_window, wl.textural_stride)
    cls, rec, mar = orc.arm_classify(q, k, g, pp, wl.sample_mode, wl.sample_stride, wl.alpha)
    assert cls[0].tolist() == [SPATIAL, TEMPORAL, TEXTURAL]
    assert mar.min() > 1e-3
    # global-only mode on a first-frame-only question: both modes agree when T == 1
    g1 = Geometry(1, 8, 8, 0)
    a = orc.arm_head(q[0, 1, :64], k[0, 1, :64], g1, pp, orc.SAMPLE_ALG1, 1, 0.9)
    b = orc.arm_head(q[0, 1, :64], k[0, 1, :64], g1, pp, orc.SAMPLE_GLOBAL, 1, 0.9)
    assert a[1][0] == pytest.approx(b[1][0], abs=1e-14)


# ---------------------------------------------------------------- RainFusion+ (dynamic bandwidth)

@pytest.mark.parametrize("Rt,Rs,expect", [
    ([0.5, 0.95, 0.99], [0.1, 0.2, 0.3], (TEMPORAL, 1)),      # smallest qualifying Temporal bandwidth
    ([0.95, 0.96, 0.97], [0.99, 0.99, 0.99], (TEMPORAL, 0)),  # Temporal has priority even if Spatial is better
    ([0.1, 0.2, 0.89], [0.2, 0.5, 0.9], (SPATIAL, 2)),        # >= alpha counts
    ([0.1, 0.2, 0.3], [0.91, 0.95, 0.99], (SPATIAL, 0)),
    ([0.1, 0.2, 0.3], [0.2, 0.5, 0.8999], (TEXTURAL, -1))])
def test_dynamic_bandwidth_truth_table(Rt, Rs, expect):
    assert orc.decide_plus(Rt, Rs, 0.9) == expect


def test_windows_of_bandwidth():
    g = Geometry(33, 45, 80, 256)
    assert orc.windows_of(0.25, g) == (8, 900)
    assert orc.windows_of(0.125, g) == (4, 450)
    assert orc.windows_of(0.5, g) == (16, 1800)


def test_dynamic_bandwidth_recalls_grow_with_the_window_and_match_the_fixed_bandwidth_path():
    wl = synth.WORKLOADS["tiny"]
    q, k, _ = synth.make_qkv(wl)
    g = Geometry(wl.T, wl.frame_h, wl.frame_w, wl.L_text)
    bws = [0.125, 0.25, 0.5]
    for h in range(wl.H):
        cls, idx, window, Rt, Rs = orc.arm_head_plus(q[0, h], k[0, h], g, bws, 2, orc.SAMPLE_ALG1, 4, 0.9)
        assert all(a <= b + 1e-15 for a, b in zip(Rt, Rt[1:]))     # nested masks: recall is monotone
        assert all(a <= b + 1e-15 for a, b in zip(Rs, Rs[1:]))
        for i, b in enumerate(bws):                                  # each candidate equals the fixed-window ARM
            wf, ws = orc.windows_of(b, g)
            _, (rt, rs, _), _ = orc.arm_head(q[0, h], k[0, h], g, PatternParams(wf, ws, 2), orc.SAMPLE_ALG1, 4, 0.9)
            assert rt == pytest.approx(Rt[i], abs=1e-15) and rs == pytest.approx(Rs[i], abs=1e-15)
        assert (cls, idx) == orc.decide_plus(Rt, Rs, 0.9)
        if cls == TEMPORAL:
            assert window == orc.windows_of(bws[idx], g)[1]
        elif cls == SPATIAL:
            assert window == orc.windows_of(bws[idx], g)[0]
        else:
            assert window == -1
    # a bandwidth of 1 keeps everything: recall 1 and Temporal always qualifies
    cls, idx, window, Rt, Rs = orc.arm_head_plus(q[0, 2], k[0, 2], g, [1.0], 2, orc.SAMPLE_ALG1, 4, 0.9)
    assert Rt[0] == pytest.approx(1.0) and Rs[0] == pytest.approx(1.0) and cls == TEMPORAL
