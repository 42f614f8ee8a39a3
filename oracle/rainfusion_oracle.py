"""CPU oracle for RainFusion's hot path (arxiv 2505.21036): TEST INFRASTRUCTURE ONLY.

A plain, slow numpy restatement, in fp64, of what the method computes:
explicit per-pattern attention masks (Sec. 3.2, Eq. 3-5), the Adaptive
Recognition Module's sampled-softmax recall and head decision (Sec. 3.3, Eq. 6,
Algorithm 1), the block masks / tile lists that follow from those masks, and
masked softmax attention (Eq. 1-2).  Nothing here is blocked, fused or
reordered: every function builds the full mask or score matrix it talks about.

Only tests, the smoke check and the benchmark's cpu_baseline / reference legs
may import this file.  It shares no code with the CUDA path and imports nothing
from the package.  bf16 inputs arrive as uint16 bit patterns and are widened to
fp64 exactly.

Readings taken where the paper is silent (each also listed in the design notes):
  * tokens: frame-major, row-major inside a frame, text tokens appended last;
  * Spatial head keeps |frame(i) - frame(j)| <= w_f (Eq. 3: the significant frames
    of frame f are its neighbours); as an option (Sec. 3.2 speaks of adjacent OR key frames) the
    first frame counts as a key frame that every query keeps as well; Temporal head keeps |pos(i) - pos(j)| <= w_s with
    pos the flattened in-frame index (Sec. 3.2 describes Temporal heads as local inside one
    frame's sub-sequence and periodic across frames); as an option the locality is a 2-D window
    |y(i) - y(j)| <= w_y and |x(i) - x(j)| <= w_x on the frame's rows and columns, the other way to read
    "local" for tokens that are image patches; text rows and text columns are always kept for both;
  * Textural head keeps key/value token (y, x) of every frame iff y mod tau == x mod tau
    (Eq. 4), plus all text keys, for every query (Eq. 5: all-zero mask on K_C, V_C);
  * recall (Eq. 6) is the share of a row's unmasked softmax mass that falls on kept
    positions, averaged over the sampled rows; the down-sampled mask is the
    restriction of the full mask to the sampled tokens;
  * Algorithm 1: Temporal if R_temporal >= alpha, else Spatial if R_spatial >= alpha,
    else Textural.

Parity pins: see tests/test_oracle_*.py.  Unpinned against the authors' own
implementation (none is available): the choices above are "parity unpinned"
with respect to it and pinned only against the definitions written here.
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Optional, Sequence, Tuple

import numpy as np

SPATIAL, TEMPORAL, TEXTURAL, DENSE = 0, 1, 2, 3
SAMPLE_ALG1, SAMPLE_GLOBAL = 0, 1
PARTIAL_BIT = 1 << 31


@dataclasses.dataclass(frozen=True)
class Geometry:
    """Latent video shape (T frames of frame_h x frame_w tokens) plus text tokens."""
    T: int
    frame_h: int
    frame_w: int
    L_text: int

    @property
    def S(self) -> int:
        return self.frame_h * self.frame_w

    @property
    def Nv(self) -> int:
        return self.T * self.S

    @property
    def N(self) -> int:
        return self.Nv + self.L_text


@dataclasses.dataclass(frozen=True)
class PatternParams:
    frame_window: int      # w_f
    spatial_window: int    # w_s
    textural_stride: int   # tau
    keep_first_frame: bool = False   # Spatial heads also keep every key of frame 0 (a "key frame", Sec. 3.2)
    temporal_window_2d: Optional[Tuple[int, int]] = None   # (w_y, w_x): Temporal heads keep |y(i)-y(j)| <= w_y and
                                                           # |x(i)-x(j)| <= w_x instead of the 1-D band on the flattened index


def bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns (uint16) to fp64."""
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


# ----------------------------------------------------------------------------------------
# Element-level masks in original token order (Sec. 3.2)
# ----------------------------------------------------------------------------------------

def frame_of(i, g: Geometry):
    return i // g.S


def pos_of(i, g: Geometry):
    return i % g.S


def in_checkerboard(j, g: Geometry, tau: int):
    """Eq. 4: video token j at in-frame (y, x) is kept iff y mod tau == x mod tau."""
    p = pos_of(j, g)
    y = p // g.frame_w
    x = p % g.frame_w
    return (y % tau) == (x % tau)


def keep_mask(pattern: int, rows: np.ndarray, cols: np.ndarray, g: Geometry, pp: PatternParams) -> np.ndarray:
    """Boolean [len(rows), len(cols)]: True where query token rows[a] may attend key token cols[b].
    rows and cols hold ORIGINAL token indices in [0, N)."""
    i = np.asarray(rows, dtype=np.int64)[:, None]
    j = np.asarray(cols, dtype=np.int64)[None, :]
    i_text = i >= g.Nv
    j_text = j >= g.Nv
    if pattern == DENSE:
        return np.ones((i.shape[0], j.shape[1]), dtype=bool)
    if pattern == SPATIAL:
        near = np.abs(frame_of(i, g) - frame_of(j, g)) <= pp.frame_window
        if pp.keep_first_frame:
            near = near | (frame_of(j, g) == 0)
        return i_text | j_text | near
    if pattern == TEMPORAL:
        if pp.temporal_window_2d is not None:
            wy, wx = pp.temporal_window_2d
            pi, pj = pos_of(i, g), pos_of(j, g)
            near = (np.abs(pi // g.frame_w - pj // g.frame_w) <= wy) & (np.abs(pi % g.frame_w - pj % g.frame_w) <= wx)
        else:
            near = np.abs(pos_of(i, g) - pos_of(j, g)) <= pp.spatial_window
        return i_text | j_text | near
    if pattern == TEXTURAL:
        kept = j_text | in_checkerboard(j, g, pp.textural_stride)
        return np.broadcast_to(kept, (i.shape[0], j.shape[1])).copy()
    raise ValueError(f"unknown pattern {pattern}")


# ----------------------------------------------------------------------------------------
# ARM: sampled approximate scores, masked recall, head decision (Sec. 3.3, Eq. 6, Alg. 1)
# ----------------------------------------------------------------------------------------

def local_sample(g: Geometry) -> np.ndarray:
    """Local sampling: the tokens of the first frame."""
    return np.arange(g.S, dtype=np.int64)


def global_sample(g: Geometry, omega: int) -> np.ndarray:
    """Global sampling: every omega-th video token, starting at token 0."""
    return np.arange(0, g.Nv, omega, dtype=np.int64)


def softmax_rows(s: np.ndarray) -> np.ndarray:
    e = np.exp(s - s.max(axis=1, keepdims=True))
    return e / e.sum(axis=1, keepdims=True)


def approx_scores(q_bits: np.ndarray, k_bits: np.ndarray, idx: np.ndarray) -> np.ndarray:
    """Eq. 1 on the sampled tokens with the all-zero mask: softmax(Q' K'^T / sqrt(d))."""
    qs = bf16_to_f64(q_bits[idx])
    ks = bf16_to_f64(k_bits[idx])
    d = qs.shape[1]
    return softmax_rows(qs @ ks.T / math.sqrt(d))


def recall(P: np.ndarray, kept: np.ndarray) -> float:
    """Eq. 6: softmax mass that survives the mask, relative to the unmasked mass (rows of P
    sum to 1), averaged over the sampled query rows."""
    return float((P * kept).sum(axis=1).mean())


def decide(R_temporal: float, R_spatial: float, alpha: float, two_mask: bool = False) -> int:
    """Algorithm 1's branch: Temporal has priority, then Spatial, else Textural.
    two_mask: the ablation of Sec. 4.4 (Table 2, rows without Te) that uses only the Spatial and the
    Temporal mask; the paper does not say what a head reaching alpha with neither gets: here the mask of
    larger recall, Temporal on equality."""
    if R_temporal >= alpha:
        return TEMPORAL
    if R_spatial >= alpha:
        return SPATIAL
    if two_mask:
        return TEMPORAL if R_temporal >= R_spatial else SPATIAL
    return TEXTURAL


def decision_margin(R_temporal: float, R_spatial: float, alpha: float, two_mask: bool = False) -> float:
    """Distance of the deciding recall(s) from the threshold (and from each other, where that decides)."""
    if R_temporal >= alpha:
        return abs(R_temporal - alpha)
    m = min(abs(R_temporal - alpha), abs(R_spatial - alpha))
    if two_mask and R_spatial < alpha:
        m = min(m, abs(R_temporal - R_spatial))
    return m


def arm_head(q_bits: np.ndarray, k_bits: np.ndarray, g: Geometry, pp: PatternParams,
             sample_mode: int, omega: int, alpha: float, two_mask: bool = False):
    """ARM for one head.  q_bits, k_bits: [N, D] bf16 bit patterns.
    Returns (class, (R_temporal, R_spatial, R_textural), margin)."""
    I_glb = global_sample(g, omega)
    P_glb = approx_scores(q_bits, k_bits, I_glb)
    R_s = recall(P_glb, keep_mask(SPATIAL, I_glb, I_glb, g, pp))
    R_te = recall(P_glb, keep_mask(TEXTURAL, I_glb, I_glb, g, pp))
    if sample_mode == SAMPLE_ALG1:
        I_loc = local_sample(g)
        P_loc = approx_scores(q_bits, k_bits, I_loc)
        R_t = recall(P_loc, keep_mask(TEMPORAL, I_loc, I_loc, g, pp))
    elif sample_mode == SAMPLE_GLOBAL:
        R_t = recall(P_glb, keep_mask(TEMPORAL, I_glb, I_glb, g, pp))
    else:
        raise ValueError(sample_mode)
    return decide(R_t, R_s, alpha, two_mask), (R_t, R_s, R_te), decision_margin(R_t, R_s, alpha, two_mask)


def arm_classify(q_bits: np.ndarray, k_bits: np.ndarray, g: Geometry, pp: PatternParams,
                 sample_mode: int, omega: int, alpha: float, two_mask: bool = False):
    """ARM over [B, H, N, D] inputs.  Returns (class int32 [B,H], recall f64 [B,H,3], margin f64 [B,H])."""
    B, H = q_bits.shape[:2]
    cls = np.zeros((B, H), dtype=np.int32)
    rec = np.zeros((B, H, 3), dtype=np.float64)
    mar = np.zeros((B, H), dtype=np.float64)
    for b in range(B):
        for h in range(H):
            c, r, m = arm_head(q_bits[b, h], k_bits[b, h], g, pp, sample_mode, omega, alpha, two_mask)
            cls[b, h], rec[b, h], mar[b, h] = c, r, m
    return cls, rec, mar


# ----------------------------------------------------------------------------------------
# RainFusion+ : per-head bandwidth (Sec. 4.3, "Qualitative Analysis and Integrability")
# ----------------------------------------------------------------------------------------

def windows_of(bandwidth: float, g: Geometry) -> Tuple[int, int]:
    """(w_f, w_s) of a bandwidth b: floor(b*T) frames, floor(b*S) in-frame positions."""
    return int(math.floor(bandwidth * g.T)), int(math.floor(bandwidth * g.S))


def decide_plus(R_temporal: Sequence[float], R_spatial: Sequence[float], alpha: float,
                two_mask: bool = False) -> Tuple[int, int]:
    """Recalls per candidate bandwidth (ascending).  The pattern is chosen as in Algorithm 1 (Temporal
    first, then Spatial, else Textural), a pattern qualifying if ANY candidate reaches alpha; its
    bandwidth is the smallest candidate that does.  Returns (class, candidate index or -1).
    two_mask (see decide): if nothing qualifies, the mask of larger recall at the widest candidate."""
    for cls, R in ((TEMPORAL, R_temporal), (SPATIAL, R_spatial)):
        for i, r in enumerate(R):
            if r >= alpha:
                return cls, i
    if two_mask:
        last = len(R_temporal) - 1
        return (TEMPORAL if R_temporal[last] >= R_spatial[last] else SPATIAL), last
    return TEXTURAL, -1


def arm_head_plus(q_bits: np.ndarray, k_bits: np.ndarray, g: Geometry, bandwidths: Sequence[float], tau: int,
                  sample_mode: int, omega: int, alpha: float, two_mask: bool = False, keep_first_frame: bool = False):
    """ARM with dynamic bandwidth for one head: every candidate bandwidth's Temporal and Spatial recall on
    the same approximate scores, then decide_plus.  Returns (class, index, window, R_t list, R_s list),
    window = w_s of the chosen bandwidth for Temporal, w_f for Spatial, -1 for Textural."""
    I_glb = global_sample(g, omega)
    P_glb = approx_scores(q_bits, k_bits, I_glb)
    if sample_mode == SAMPLE_ALG1:
        I_t = local_sample(g)
        P_t = approx_scores(q_bits, k_bits, I_t)
    else:
        I_t, P_t = I_glb, P_glb
    R_t, R_s = [], []
    for b in bandwidths:
        wf, ws = windows_of(b, g)
        pp = PatternParams(wf, ws, tau, keep_first_frame)
        R_t.append(recall(P_t, keep_mask(TEMPORAL, I_t, I_t, g, pp)))
        R_s.append(recall(P_glb, keep_mask(SPATIAL, I_glb, I_glb, g, pp)))
    cls, idx = decide_plus(R_t, R_s, alpha, two_mask)
    window = -1
    if cls == TEMPORAL:
        window = windows_of(bandwidths[idx], g)[1]
    elif cls == SPATIAL:
        window = windows_of(bandwidths[idx], g)[0]
    return cls, idx, window, R_t, R_s


# ----------------------------------------------------------------------------------------
# Head coordinate spaces, block masks and tile lists
# ----------------------------------------------------------------------------------------

def kept_per_frame(g: Geometry, tau: int) -> np.ndarray:
    """In-frame positions of the checkerboard set C (Eq. 4), ascending."""
    p = np.arange(g.S, dtype=np.int64)
    return p[in_checkerboard(p, g, tau)]


def query_order(pattern: int, g: Geometry, temporal_permute: bool) -> np.ndarray:
    """pi_q: original token index held by each query slot of the head's coordinate space."""
    if pattern == TEMPORAL and temporal_permute:
        slot = np.arange(g.Nv, dtype=np.int64)
        p, f = slot // g.T, slot % g.T          # slot = p*T + f  (position-major)
        return np.concatenate([f * g.S + p, np.arange(g.Nv, g.N, dtype=np.int64)])
    return np.arange(g.N, dtype=np.int64)


def key_order(pattern: int, g: Geometry, pp: PatternParams, temporal_permute: bool) -> np.ndarray:
    """pi_k: original token index held by each key/value slot; its length is Lkv."""
    if pattern == TEXTURAL:
        c = kept_per_frame(g, pp.textural_stride)
        video = (np.arange(g.T, dtype=np.int64)[:, None] * g.S + c[None, :]).reshape(-1)
        return np.concatenate([video, np.arange(g.Nv, g.N, dtype=np.int64)])
    return query_order(pattern, g, temporal_permute)


def tile_row(pattern: int, g: Geometry, pp: PatternParams, temporal_permute: bool,
             BM: int, BN: int, a: int) -> List[int]:
    """Ascending list of non-empty KV tiles of query tile `a`, PARTIAL entries carrying bit 31.

    Tile (a, b) covers query slots [a*BM, min((a+1)*BM, N)) and key slots
    [b*BN, min((b+1)*BN, Lkv)).  It is non-empty iff some pair in it is kept, FULL iff every
    pair is kept and the tile holds BN real key slots, PARTIAL otherwise."""
    pq = query_order(pattern, g, temporal_permute)
    pk = key_order(pattern, g, pp, temporal_permute)
    Lkv = pk.shape[0]
    rows = pq[a * BM: min((a + 1) * BM, g.N)]
    kept = keep_mask(pattern, rows, pk, g, pp)
    out: List[int] = []
    for b in range((Lkv + BN - 1) // BN):
        sub = kept[:, b * BN: min((b + 1) * BN, Lkv)]
        if not sub.any():
            continue
        full = bool(sub.all()) and (b + 1) * BN <= Lkv
        out.append(b if full else (b | PARTIAL_BIT))
    return out


def kv_len(pattern: int, g: Geometry, pp: PatternParams) -> int:
    return int(key_order(pattern, g, pp, False).shape[0])


# ----------------------------------------------------------------------------------------
# Masked softmax attention (Eq. 1-2 with the pattern's mask)
# ----------------------------------------------------------------------------------------

def masked_attention(q_bits: np.ndarray, k_bits: np.ndarray, v_bits: np.ndarray, pattern: int,
                     g: Geometry, pp: PatternParams, rows: Optional[Sequence[int]] = None,
                     chunk: int = 256) -> Tuple[np.ndarray, np.ndarray]:
    """O_i = sum_j softmax_j(<q_i, k_j>/sqrt(d) + M_ij) v_j for one head, M = 0 where kept, -inf elsewhere.
    q_bits, k_bits, v_bits: [N, D] bf16 bit patterns.  rows: query tokens to compute (default all).
    Returns (O [R, D] fp64, lse [R] fp64, natural log of the row's sum of exp(score))."""
    N, D = q_bits.shape
    rows = np.arange(N, dtype=np.int64) if rows is None else np.asarray(rows, dtype=np.int64)
    K = bf16_to_f64(k_bits)
    V = bf16_to_f64(v_bits)
    cols = np.arange(N, dtype=np.int64)
    O = np.empty((rows.shape[0], V.shape[1]), dtype=np.float64)
    lse = np.empty(rows.shape[0], dtype=np.float64)
    for c0 in range(0, rows.shape[0], chunk):
        r = rows[c0: c0 + chunk]
        s = bf16_to_f64(q_bits[r]) @ K.T / math.sqrt(D)
        s = np.where(keep_mask(pattern, r, cols, g, pp), s, -np.inf)
        mx = s.max(axis=1, keepdims=True)
        e = np.exp(s - mx)
        l = e.sum(axis=1, keepdims=True)
        O[c0: c0 + chunk] = (e / l) @ V
        lse[c0: c0 + chunk] = (mx + np.log(l))[:, 0]
    return O, lse
