"""Pins for the oracle's pattern masks, coordinate spaces and tile lists (CPU only).

Each check compares the oracle with something fixed outside it: an independent
enumeration of the token layout, a Kronecker construction, a closed form, or an
arithmetic fact the paper states (tests/golden/paper_arithmetic.txt)."""
import math
import os

import numpy as np
import pytest

from oracle import rainfusion_oracle as orc
from oracle.rainfusion_oracle import DENSE, SPATIAL, TEMPORAL, TEXTURAL, Geometry, PatternParams


def golden():
    path = os.path.join(os.path.dirname(__file__), "golden", "paper_arithmetic.txt")
    out = {}
    for line in open(path):
        line = line.split("#")[0].split()
        if len(line) == 2:
            out[line[0]] = float(line[1])
    return out


def token_table(g):
    """Independent enumeration of the token layout: nested loops, no div/mod."""
    tab = []
    for f in range(g.T):
        for y in range(g.frame_h):
            for x in range(g.frame_w):
                tab.append((f, y, x, y * g.frame_w + x, False))
    for _ in range(g.L_text):
        tab.append((-1, -1, -1, -1, True))
    return tab


def brute_mask(pattern, g, pp):
    tab = token_table(g)
    N = len(tab)
    M = np.zeros((N, N), dtype=bool)
    for i, (fi, yi, xi, pi, ti) in enumerate(tab):
        for j, (fj, yj, xj, pj, tj) in enumerate(tab):
            if pattern == DENSE:
                k = True
            elif pattern == SPATIAL:
                k = ti or tj or abs(fi - fj) <= pp.frame_window
            elif pattern == TEMPORAL:
                k = ti or tj or abs(pi - pj) <= pp.spatial_window
            else:
                k = tj or any(yj % pp.textural_stride == r and xj % pp.textural_stride == r
                              for r in range(pp.textural_stride))
            M[i, j] = k
    return M


@pytest.mark.parametrize("geom", [Geometry(3, 3, 4, 2), Geometry(4, 2, 5, 0), Geometry(1, 4, 4, 3)])
@pytest.mark.parametrize("pp", [PatternParams(1, 2, 2), PatternParams(0, 0, 3), PatternParams(2, 5, 1)])
@pytest.mark.parametrize("pattern", [SPATIAL, TEMPORAL, TEXTURAL, DENSE])
def test_masks_match_loop_enumeration(geom, pp, pattern):
    idx = np.arange(geom.N)
    assert np.array_equal(orc.keep_mask(pattern, idx, idx, geom, pp), brute_mask(pattern, geom, pp))


def test_spatial_is_block_diagonal_per_frame_when_window_zero():
    g = Geometry(4, 3, 5, 0)
    idx = np.arange(g.N)
    M = orc.keep_mask(SPATIAL, idx, idx, g, PatternParams(0, 0, 2))
    assert np.array_equal(M, np.kron(np.eye(g.T, dtype=bool), np.ones((g.S, g.S), dtype=bool)))


def test_temporal_is_per_position_when_window_zero():
    g = Geometry(4, 3, 5, 0)
    idx = np.arange(g.N)
    M = orc.keep_mask(TEMPORAL, idx, idx, g, PatternParams(0, 0, 2))
    assert np.array_equal(M, np.kron(np.ones((g.T, g.T), dtype=bool), np.eye(g.S, dtype=bool)))


def test_band_structure_is_toeplitz_kron():
    g = Geometry(6, 2, 4, 0)
    idx = np.arange(g.N)
    w = 2
    bandT = np.abs(np.subtract.outer(np.arange(g.T), np.arange(g.T))) <= w
    bandS = np.abs(np.subtract.outer(np.arange(g.S), np.arange(g.S))) <= w
    assert np.array_equal(orc.keep_mask(SPATIAL, idx, idx, g, PatternParams(w, 0, 2)),
                          np.kron(bandT, np.ones((g.S, g.S), dtype=bool)))
    assert np.array_equal(orc.keep_mask(TEMPORAL, idx, idx, g, PatternParams(0, w, 2)),
                          np.kron(np.ones((g.T, g.T), dtype=bool), bandS))


@pytest.mark.parametrize("n,w", [(13, 3), (33, 8), (4, 1), (7, 0), (5, 9)])
def test_band_kept_fraction_closed_form(n, w):
    # a symmetric band of half-width w in an n x n grid keeps n(2w+1) - w(w+1) cells (w clipped to n-1)
    g = Geometry(n, 2, 3, 0)
    idx = np.arange(g.N)
    M = orc.keep_mask(SPATIAL, idx, idx, g, PatternParams(w, 0, 2))
    wc = min(w, n - 1)
    assert M.sum() == (n * (2 * wc + 1) - wc * (wc + 1)) * g.S * g.S
    g2 = Geometry(2, 1, n, 0)
    idx2 = np.arange(g2.N)
    M2 = orc.keep_mask(TEMPORAL, idx2, idx2, g2, PatternParams(0, w, 2))
    assert M2.sum() == (n * (2 * wc + 1) - wc * (wc + 1)) * g2.T * g2.T


def test_paper_bandwidth_quarter_gives_nine_sixteenths_reduction():
    gold = golden()
    b = gold["bandwidth"]
    n = 4000
    w = int(b * n)
    kept = (n * (2 * w + 1) - w * (w + 1)) / n ** 2      # closed form pinned above against the mask
    assert abs((1 - kept) - gold["band_compute_reduction"]) < 1e-3
    # and on a real (small) mask: T = 64 frames, w_f = 16
    g = Geometry(64, 1, 2, 0)
    idx = np.arange(g.N)
    frac = orc.keep_mask(SPATIAL, idx, idx, g, PatternParams(16, 0, 2)).mean()
    assert abs((1 - frac) - gold["band_compute_reduction"]) < 0.02


def test_paper_default_speedup_arithmetic():
    # 10 % dense steps + kept fraction between 7/16 (band heads) and 1/2 (textural heads)
    gold = golden()
    lo = 1 / (gold["dense_step_fraction"] + (1 - gold["dense_step_fraction"]) * 0.5)
    hi = 1 / (gold["dense_step_fraction"] + (1 - gold["dense_step_fraction"]) * (1 - gold["band_compute_reduction"]))
    assert lo <= gold["attention_speedup"] + 0.04 and gold["attention_speedup"] <= hi


@pytest.mark.parametrize("fh,fw,tau,expect", [
    (8, 8, 2, 32), (30, 45, 2, 675), (45, 80, 2, 1800), (30, 45, 3, 450), (45, 80, 3, 1200),
    (30, 45, 4, 338), (45, 80, 4, 900), (5, 7, 1, 35)])
def test_checkerboard_counts(fh, fw, tau, expect):
    g = Geometry(2, fh, fw, 0)
    c = orc.kept_per_frame(g, tau)
    # sum over residues k of ceil((fh-k)/tau) * ceil((fw-k)/tau)
    closed = sum(math.ceil((fh - k) / tau) * math.ceil((fw - k) / tau) for k in range(tau))
    assert len(c) == closed == expect
    assert np.all(np.diff(c) > 0)


def test_checkerboard_tau2_halves_and_neighbours_are_kept():
    gold = golden()
    g = Geometry(1, 30, 45, 0)
    kept = np.zeros(g.S, dtype=bool)
    kept[orc.kept_per_frame(g, 2)] = True
    assert abs(kept.mean() - gold["textural_kept_fraction"]) < 1e-3
    grid = kept.reshape(g.frame_h, g.frame_w)
    for y in range(1, g.frame_h - 1):
        for x in range(1, g.frame_w - 1):
            if not grid[y, x]:
                assert grid[y - 1, x] and grid[y + 1, x] and grid[y, x - 1] and grid[y, x + 1]


def test_degenerate_parameters_give_all_ones():
    g = Geometry(3, 2, 3, 2)
    idx = np.arange(g.N)
    assert orc.keep_mask(SPATIAL, idx, idx, g, PatternParams(g.T - 1, 0, 2)).all()
    assert orc.keep_mask(TEMPORAL, idx, idx, g, PatternParams(0, g.S - 1, 2)).all()
    assert orc.keep_mask(TEXTURAL, idx, idx, g, PatternParams(0, 0, 1)).all()


def test_text_rows_and_columns():
    g = Geometry(3, 2, 3, 4)
    pp = PatternParams(0, 0, 2)
    idx = np.arange(g.N)
    for pat in (SPATIAL, TEMPORAL):
        M = orc.keep_mask(pat, idx, idx, g, pp)
        assert M[g.Nv:, :].all() and M[:, g.Nv:].all()
    M = orc.keep_mask(TEXTURAL, idx, idx, g, pp)
    assert M[:, g.Nv:].all()
    assert np.array_equal(M[g.Nv:, :g.Nv], M[:g.L_text, :g.Nv])   # text queries see C, like everyone


# ---------------------------------------------------------------- coordinate spaces

def test_temporal_permutation_is_position_major_bijection():
    g = Geometry(3, 2, 2, 2)
    pq = orc.query_order(TEMPORAL, g, True)
    assert sorted(pq.tolist()) == list(range(g.N))
    # slots enumerate positions outermost, frames innermost
    expect = [f * g.S + p for p in range(g.S) for f in range(g.T)] + list(range(g.Nv, g.N))
    assert pq.tolist() == expect
    assert np.array_equal(orc.query_order(TEMPORAL, g, False), np.arange(g.N))
    assert np.array_equal(orc.query_order(SPATIAL, g, True), np.arange(g.N))


def test_textural_key_order_is_ascending_kept_then_text():
    g = Geometry(3, 4, 5, 2)
    pp = PatternParams(1, 1, 2)
    pk = orc.key_order(TEXTURAL, g, pp, True)
    tab = token_table(g)
    expect = [i for i, (f, y, x, p, t) in enumerate(tab) if t or (y % 2 == x % 2)]
    assert pk.tolist() == expect
    assert orc.kv_len(TEXTURAL, g, pp) == len(expect)
    assert orc.kv_len(SPATIAL, g, pp) == g.N


# ---------------------------------------------------------------- tile lists

def flags(lst):
    return [(e & 0x7FFFFFFF, bool(e >> 31)) for e in lst]


def test_tile_lists_textural_and_dense_list_everything():
    g = Geometry(4, 8, 8, 16)
    pp = PatternParams(1, 2, 2)
    for pat in (TEXTURAL, DENSE):
        L = orc.kv_len(pat, g, pp)
        for BN in (16, 32, 64, 128):
            nK = -(-L // BN)
            for a in range(-(-g.N // 64)):
                lst = flags(orc.tile_row(pat, g, pp, True, 64, BN, a))
                assert [b for b, _ in lst] == list(range(nK))
                assert all(not p for _, p in lst[:-1])
                assert lst[-1][1] == (L % BN != 0)


def test_tile_lists_block_diagonal_case():
    # w_f = 0, no text, S a multiple of the block: exactly the diagonal frame blocks, all FULL
    g = Geometry(4, 8, 8, 0)
    pp = PatternParams(0, 0, 2)
    BM = BN = 32
    for a in range(g.N // BM):
        f = (a * BM) // g.S
        expect = [(b, False) for b in range(f * g.S // BN, (f + 1) * g.S // BN)]
        assert flags(orc.tile_row(SPATIAL, g, pp, False, BM, BN, a)) == expect


def test_tile_lists_against_loop_enumeration():
    g = Geometry(5, 6, 7, 3)
    pp = PatternParams(1, 5, 2)
    tab = token_table(g)
    BM, BN = 16, 32
    for pat, perm in ((SPATIAL, False), (TEMPORAL, False), (TEMPORAL, True), (TEXTURAL, False)):
        M = brute_mask(pat, g, pp)
        if pat == TEMPORAL and perm:
            order = [f * g.S + p for p in range(g.S) for f in range(g.T)] + list(range(g.Nv, g.N))
            qo = ko = order
        elif pat == TEXTURAL:
            qo = list(range(g.N))
            ko = [i for i, (f, y, x, p, t) in enumerate(tab) if t or (y % 2 == x % 2)]
        else:
            qo = ko = list(range(g.N))
        Mh = M[np.ix_(qo, ko)]
        for a in range(-(-g.N // BM)):
            expect = []
            for b in range(-(-len(ko) // BN)):
                sub = Mh[a * BM:(a + 1) * BM, b * BN:(b + 1) * BN]
                if sub.any():
                    expect.append((b, not (sub.all() and (b + 1) * BN <= len(ko))))
            assert flags(orc.tile_row(pat, g, pp, perm, BM, BN, a)) == expect


def test_tiny_config_tile_density():
    # 4 frames of 8x8 + 16 text, 128x128 tiles: Spatial/Temporal list all 3x3 tiles,
    # Textural's key space is 4*32+16 = 144 slots = 2 tiles of 3 -> density 2/3
    g = Geometry(4, 8, 8, 16)
    pp = PatternParams(1, 2, 2)
    for pat, n in ((SPATIAL, 9), (TEMPORAL, 9), (TEXTURAL, 6), (DENSE, 9)):
        tot = sum(len(orc.tile_row(pat, g, pp, True, 128, 128, a)) for a in range(3))
        assert tot == n


def test_permutation_makes_temporal_mask_banded():
    # in position-major order a Temporal row's kept video keys form ONE contiguous run
    g = Geometry(4, 3, 5, 2)
    pp = PatternParams(0, 2, 2)
    pq = orc.query_order(TEMPORAL, g, True)
    M = orc.keep_mask(TEMPORAL, pq, pq, g, pp)[:, :g.Nv]
    for r in range(g.Nv):
        nz = np.flatnonzero(M[r])
        assert nz[-1] - nz[0] + 1 == len(nz)


# ---------------------------------------------------------------- Spatial head with the first frame as a key frame

def test_key_first_frame_mask_by_enumeration():
    """Sec. 3.2 lets a Spatial head attend adjacent OR key frames; with the option on, every query also keeps the keys
    of frame 0.  Nested loops over the definition, all patterns (only Spatial may change)."""
    g = Geometry(5, 2, 3, 2)
    idx = np.arange(g.N)
    for wf in (0, 1, 2):
        on, off = PatternParams(wf, 1, 2, True), PatternParams(wf, 1, 2, False)
        M = orc.keep_mask(SPATIAL, idx, idx, g, on)
        for i in range(g.N):
            for j in range(g.N):
                if i >= g.Nv or j >= g.Nv:
                    want = True
                else:
                    want = abs(i // g.S - j // g.S) <= wf or j // g.S == 0
                assert M[i, j] == want, (wf, i, j)
        for pattern in (TEMPORAL, TEXTURAL, DENSE):
            assert np.array_equal(orc.keep_mask(pattern, idx, idx, g, on), orc.keep_mask(pattern, idx, idx, g, off))
        # a superset of the plain Spatial mask that differs only in key columns of frame 0
        P = orc.keep_mask(SPATIAL, idx, idx, g, off)
        assert (M | P).sum() == M.sum() and np.array_equal(M[:, g.S:], P[:, g.S:])


def test_key_first_frame_kept_fraction_closed_form():
    # frame pairs kept: the band T(2w+1) - w(w+1) plus, in key column 0, the query frames the band does not reach: T - 1 - w
    for T, w in ((8, 1), (13, 3), (6, 0), (5, 4), (5, 9)):
        g = Geometry(T, 2, 2, 0)
        idx = np.arange(g.N)
        M = orc.keep_mask(SPATIAL, idx, idx, g, PatternParams(w, 0, 2, True))
        wc = min(w, T - 1)
        frames = T * (2 * wc + 1) - wc * (wc + 1) + (T - 1 - wc)
        assert M.sum() == frames * g.S * g.S


def test_key_first_frame_tile_lists_follow_the_mask():
    g = Geometry(6, 4, 8, 5)                     # S = 32: a 16-slot tile never straddles two frames, a 64-slot tile always does
    pp = PatternParams(1, 3, 2, True)
    pq = orc.query_order(SPATIAL, g, False)
    kept = orc.keep_mask(SPATIAL, pq, pq, g, pp)
    for block in (16, 64):
        nQ = -(-g.N // block)
        for a in range(nQ):
            row = orc.tile_row(SPATIAL, g, pp, False, block, block, a)
            tiles = [e & ~orc.PARTIAL_BIT for e in row]
            assert 0 in tiles                      # the first key tile lies in frame 0: every query tile lists it
            for b in range(nQ):
                sub = kept[a * block:(a + 1) * block, b * block:(b + 1) * block]
                assert (b in tiles) == bool(sub.any())


# ---------------------------------------------------------------- Temporal head with a 2-D in-frame window

def test_temporal_2d_window_by_enumeration():
    """The other reading of Sec. 3.2's locality inside a frame: a window on rows and columns of the frame rather than a
    band on the flattened index.  Nested loops over the definition; the other patterns do not change."""
    g = Geometry(3, 4, 5, 2)
    idx = np.arange(g.N)
    for wy, wx in ((0, 0), (1, 2), (0, 4), (3, 0), (9, 9)):
        pp = PatternParams(1, 2, 2, False, (wy, wx))
        M = orc.keep_mask(TEMPORAL, idx, idx, g, pp)
        for i in range(g.N):
            for j in range(g.N):
                if i >= g.Nv or j >= g.Nv:
                    want = True
                else:
                    pi, pj = i % g.S, j % g.S
                    want = abs(pi // g.frame_w - pj // g.frame_w) <= wy and abs(pi % g.frame_w - pj % g.frame_w) <= wx
                assert M[i, j] == want, (wy, wx, i, j)
        for pattern in (SPATIAL, TEXTURAL, DENSE):
            assert np.array_equal(orc.keep_mask(pattern, idx, idx, g, pp), orc.keep_mask(pattern, idx, idx, g, PatternParams(1, 2, 2)))
    # a window covering the frame keeps everything
    assert orc.keep_mask(TEMPORAL, idx, idx, g, PatternParams(1, 0, 2, False, (3, 4))).all()


def test_temporal_2d_window_is_a_kronecker_product_of_two_bands():
    # video x video part = ones(T, T) (x) band_y(H) (x) band_x(W)
    g = Geometry(3, 5, 6, 0)
    wy, wx = 1, 2
    idx = np.arange(g.N)
    M = orc.keep_mask(TEMPORAL, idx, idx, g, PatternParams(0, 0, 2, False, (wy, wx)))
    by = np.abs(np.subtract.outer(np.arange(g.frame_h), np.arange(g.frame_h))) <= wy
    bx = np.abs(np.subtract.outer(np.arange(g.frame_w), np.arange(g.frame_w))) <= wx
    assert np.array_equal(M, np.kron(np.ones((g.T, g.T), dtype=bool), np.kron(by, bx)))
    # kept count: product of the two band counts, for every frame pair
    cy = g.frame_h * (2 * wy + 1) - wy * (wy + 1)
    cx = g.frame_w * (2 * wx + 1) - wx * (wx + 1)
    assert M.sum() == g.T * g.T * cy * cx


def test_temporal_2d_tile_lists_follow_the_mask():
    g = Geometry(4, 6, 10, 7)
    pp = PatternParams(1, 3, 2, False, (1, 3))
    for permute in (False, True):
        pq = orc.query_order(TEMPORAL, g, permute)
        kept = orc.keep_mask(TEMPORAL, pq, pq, g, pp)
        for block in (16, 64):
            nQ = -(-g.N // block)
            for a in range(0, nQ, 3):
                row = orc.tile_row(TEMPORAL, g, pp, permute, block, block, a)
                tiles = {e & ~orc.PARTIAL_BIT: bool(e & orc.PARTIAL_BIT) for e in row}
                for b in range(nQ):
                    sub = kept[a * block:(a + 1) * block, b * block:(b + 1) * block]
                    assert (b in tiles) == bool(sub.any())
                    if b in tiles:
                        assert tiles[b] == (not (sub.all() and (b + 1) * block <= g.N))
