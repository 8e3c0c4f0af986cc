"""Float64 CPU oracle for declared-reference ("fold") softmax attention decode.

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain statement of what the
decode path computes.  It shares no code with the CUDA library and must never be
imported by it; only the tests, the smoke check and the benchmark's CPU-baseline
leg call it.  Everything is numpy float64; inputs are BF16 values that the caller
has already widened exactly (see ``widen_bf16``).

Conventions (Section 2, "Online softmax and its merge"):
  * scores are base-2:  s_j = log2(e) * c * <q, k_j>,  c the softmax scale
    (1/sqrt(D) by default);
  * Z, T and every log-sum-exp are in binades (base-2 units).

What is here, with the passage each function restates:
  scores                Section 2 definition of s_ij
  dense_row             Section 2: o = sum_j 2^s_j v_j / sum_j 2^s_j (max-subtracted)
  fold_partial          Eq. 2: F(I) = (A, L) for one key set, plus the depth-T cut
                        of Section 4 "Depth as a dial" (cut keys keep their mass)
  draft_visible /
  mask_draft_scores     Section 4 "Value product" (drafts and verification trees are extra query
                        rows masked to their ancestors): which of the last m keys a row sees
  block_means           Section 4 "Depth as a dial": the mean value of each 64-key block
                        (the block model without its fitted rank-16 map), stored as BF16
  fold_row              Eq. 2 + Prop. 1(i): partials over key ranges, added
  merge_partials        Prop. 1(i): partials add; o = A/L, lse = Z + log2 L
  online_softmax_bf16   Section 2 online softmax with a running maximum; the
                        "plain BF16 kernel" error yardstick
  lse_merge             Eq. 1: the max-compare/rescale merge fold replaces
  estimator_indices /
  estimate_z            Section 3 "Choosing the reference": 192-key estimate.
                        PARITY UNPINNED by the paper beyond its one-sentence
                        description; the reading taken is written out below.
  grid_sum              Eq. 3 / Prop. 2 applied to the forward partial add:
                        order-free integer-grid summation (Python ints, exact)
  decode_batch          GQA / batch / paged plumbing around the row functions
"""
from __future__ import annotations

import math
from typing import Iterable, Optional, Sequence

import numpy as np

LOG2E = 1.4426950408889634  # log2(e)

# Estimator constants (Section 3, "Choosing the reference": sink + 63 most recent
# keys scored exactly, 128 stratum centres over the rest, trimmed).
EST_RECENT = 63
EST_STRATA = 128
EST_TRIM = 8          # reading: the 8 largest centre weights are dropped
EST_EXACT_MAX_N = 192  # rows with at most this many keys use their exact lse


# --------------------------------------------------------------------------- inputs
def widen_bf16(bits: np.ndarray) -> np.ndarray:
    """Exact BF16 -> float64 from the 16-bit patterns (uint16 / int16 array)."""
    b = np.ascontiguousarray(bits).view(np.uint16).astype(np.uint32) << np.uint32(16)
    return b.view(np.float32).astype(np.float64)


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """float -> nearest BF16 (ties to even), returned as float64.  Used only by the
    BF16 yardstick and to model the BF16 output rounding."""
    f = np.asarray(x, dtype=np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    rounded = ((u + 0x7FFF + ((u >> 16) & 1)) >> 16) << 16
    out = rounded.astype(np.uint32).view(np.float32).astype(np.float64)
    nan = np.isnan(f)
    if nan.any():
        out = np.where(nan, np.nan, out)
    return out


# --------------------------------------------------------------------------- scores
def scores(q: np.ndarray, K: np.ndarray, scale: Optional[float] = None) -> np.ndarray:
    """Base-2 scores s_j = log2(e) * c * <q, k_j> for one query row.  q [D], K [n, D]."""
    q = np.asarray(q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    if scale is None:
        scale = 1.0 / math.sqrt(q.shape[-1])
    return (K @ q) * (LOG2E * scale)


# --------------------------------------------------------------------------- dense
def draft_visible(n: int, m: int, mask: int) -> np.ndarray:
    """Keys a draft / tree-verification row sees (Section 4 "Value product"; Appendix "Cascades and
    drafts").  The last m keys of the sequence are the draft tokens, already appended to the cache;
    key n - m + t is visible iff bit t of `mask` is set (the row's ancestors and itself); every
    earlier key is visible to every row.  If n < m only bits m - n .. m - 1 have a key.  Returns bool [n]."""
    vis = np.ones(n, dtype=bool)
    for t in range(m):
        j = n - m + t
        if j >= 0 and not (mask >> t) & 1:
            vis[j] = False
    return vis


def mask_draft_scores(s: np.ndarray, m: int, mask: int) -> np.ndarray:
    """Scores with the keys the row may not see set to -inf: their weight is exactly 0 in every
    function of this module (dense, declared-reference, estimator)."""
    s = np.array(s, dtype=np.float64)
    s[~draft_visible(s.size, m, mask)] = -np.inf
    return s


def dense_row(s: np.ndarray, V: np.ndarray):
    """Textbook softmax attention of one row from base-2 scores: returns (o [D], lse2).
    The maximum is subtracted only to stay in range (Section 2)."""
    s = np.asarray(s, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    if s.size == 0:
        return np.zeros(V.shape[-1]), -np.inf
    m = s.max()
    w = np.exp2(s - m)
    L = w.sum()
    o = (w[:, None] * V).sum(axis=0) / L
    return o, m + math.log2(L)


# --------------------------------------------------------------------------- fold
def live_mask(s: np.ndarray, Z: float, T: float) -> np.ndarray:
    """Depth gate of Section 4: key j is live iff s_j >= Z - T.  T = inf keeps all."""
    if math.isinf(T):
        return np.ones(s.shape, dtype=bool)
    return (s - Z) >= -T


BLOCK_KEYS = 64  # keys per block of the block model (Section 4, "Depth as a dial")


def block_means(V: np.ndarray, block: int = BLOCK_KEYS) -> np.ndarray:
    """Mean value row of each block of `block` consecutive keys (the last block may be
    short: the mean is over the keys it has), rounded to BF16 as the cache stores it.
    Section 4 "Depth as a dial": the block model's mean; its rank-16 key-to-deviation map
    needs a fit on the prompt and is not part of this reading.  Returns [ceil(n/block), D]."""
    V = np.asarray(V, dtype=np.float64)
    n = V.shape[0]
    nb = (n + block - 1) // block
    out = np.zeros((nb, V.shape[1]))
    for b in range(nb):
        rows = V[b * block:min((b + 1) * block, n)]
        out[b] = rows.sum(axis=0) / rows.shape[0]
    return round_to_bf16(out)


def fold_partial(s: np.ndarray, V: np.ndarray, Z: float, T: float = math.inf, tail=None):
    """F(I) of Eq. 2 over the keys given, with the depth-T cut: every key adds its
    weight 2^(s-Z) to L; only live keys add weight*value to A.  Returns (A [D], L).

    tail = (v_mean [num_blocks, D], block_of [len(s)]) switches the block tail on
    (Section 4 "Depth as a dial"; Algorithm 1, the step that gives the cut keys' weights to the
    tile's virtual row): a cut key j adds weight * v_mean[block_of[j]] to A instead of nothing."""
    s = np.asarray(s, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    p = np.exp2(s - Z)
    L = p.sum()
    live = live_mask(s, Z, T)
    A = (p[live, None] * V[live]).sum(axis=0)
    if tail is not None:
        v_mean, block_of = tail
        v_mean = np.asarray(v_mean, dtype=np.float64)
        block_of = np.asarray(block_of)
        cut = ~live
        for b in np.unique(block_of[cut]):
            A = A + p[cut & (block_of == b)].sum() * v_mean[b]
    return A, L


def merge_partials(partials: Iterable, Z: float):
    """Prop. 1(i): partial pairs add.  Returns (o, lse2, A, L)."""
    A = None
    L = 0.0
    for (a, l) in partials:
        A = np.array(a, dtype=np.float64) if A is None else A + a
        L = L + l
    if A is None:
        raise ValueError("no partials")
    with np.errstate(divide="ignore", invalid="ignore"):
        o = A / L
        lse = Z + (math.log2(L) if L > 0 else -np.inf)
    return o, lse, A, L


def fold_row(s, V, Z: float, T: float = math.inf, ranges: Optional[Sequence] = None, v_mean=None):
    """Declared-reference attention of one row.  `ranges` is a list of index arrays /
    slices that partition the keys (default: one range); each range's (A, L) is
    formed on its own and the pairs are added.  `v_mean` [ceil(n/64), D] switches the
    block tail on (key j belongs to block j // 64).  Returns (o, lse2, A, L)."""
    s = np.asarray(s, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    if s.size == 0:
        return np.zeros(V.shape[-1]), -np.inf, np.zeros(V.shape[-1]), 0.0
    if ranges is None:
        ranges = [slice(None)]
    block_of = np.arange(s.size) // BLOCK_KEYS
    return merge_partials((fold_partial(s[r], V[r], Z, T, None if v_mean is None else (v_mean, block_of[r]))
                           for r in ranges), Z)


def cut_report(s, V, Z: float, T: float, band: float = 2.0 ** -10):
    """Diagnostics for a finite depth: live fraction, cut-mass fraction sum_cut p / L,
    and the threshold slack  sum_{|s-Z+T|<=band} p*|v|_inf / L : the largest change of
    any output element if every key within `band` binades of the threshold flipped
    (fp32 scores on the GPU against fp64 scores here can disagree on those)."""
    s = np.asarray(s, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    p = np.exp2(s - Z)
    L = p.sum()
    live = live_mask(s, Z, T)
    near = np.abs(s - Z + T) <= band if not math.isinf(T) else np.zeros(s.shape, bool)
    slack = float((p[near] * np.abs(V[near]).max(axis=1)).sum() / L) if near.any() else 0.0
    return {"live_frac": float(live.mean()), "cut_mass": float(p[~live].sum() / L), "slack": slack}


# --------------------------------------------------------------------------- baselines
def lse_merge(o1, l1, o2, l2):
    """Eq. 1 in base 2: merge two (o, lse) states by comparing and rescaling."""
    m = max(l1, l2)
    w1, w2 = 2.0 ** (l1 - m), 2.0 ** (l2 - m)
    return (w1 * np.asarray(o1) + w2 * np.asarray(o2)) / (w1 + w2), m + math.log2(w1 + w2)


def _f32(x):
    return np.asarray(x, dtype=np.float32)


def online_softmax_bf16(q, K, V, scale: Optional[float] = None, tile: int = 64):
    """Emulation of a plain BF16 online-softmax decode kernel (Section 2): walk the keys
    in tiles, FP32 scores from the BF16 inputs, running maximum with rescale of (A, L),
    weights rounded to BF16 for the value product, FP32 accumulation, BF16 output.
    Returns o as float64 holding BF16 values.  This is the error yardstick only."""
    q = np.asarray(q, dtype=np.float64)
    if scale is None:
        scale = 1.0 / math.sqrt(q.shape[-1])
    n, D = K.shape
    m = np.float32(-np.inf)
    A = np.zeros(D, dtype=np.float32)
    L = np.float32(0.0)
    for t0 in range(0, n, tile):
        Kt = np.asarray(K[t0:t0 + tile], dtype=np.float64)
        Vt = _f32(V[t0:t0 + tile])
        st = _f32((Kt @ q) * (LOG2E * scale))      # fp32 score (products of BF16 are exact)
        m_new = np.float32(max(m, st.max()))
        r = np.float32(0.0) if np.isinf(m) else np.exp2(np.float32(m - m_new))
        p = np.exp2(st - m_new).astype(np.float32)
        pb = _f32(round_to_bf16(p))
        A = (A * r + (pb[:, None] * Vt).sum(axis=0, dtype=np.float32)).astype(np.float32)
        L = np.float32(L * r + p.sum(dtype=np.float32))
        m = m_new
    return round_to_bf16(A / L)


# --------------------------------------------------------------------------- estimator
def estimator_indices(n: int):
    """Which keys the 192-key reference estimate reads for a row of n keys.
    Returns (sink, recent [63], centres [128], n_mid) for n > 192, or None when the row
    is short enough to score in full.

    Reading of the one-sentence description in Section 3: key 0 is the sink; the last
    63 keys are the recent window; the n_mid = n - 64 keys between them are cut into
    128 equal contiguous strata with edges 1 + floor(k * n_mid / 128) and the key in
    the middle of each stratum, floor((edge_k + edge_{k+1}) / 2), stands for it."""
    if n <= EST_EXACT_MAX_N:
        return None
    n_mid = n - 1 - EST_RECENT
    edges = [1 + (k * n_mid) // EST_STRATA for k in range(EST_STRATA + 1)]
    centres = np.array([(edges[k] + edges[k + 1]) // 2 for k in range(EST_STRATA)], dtype=np.int64)
    recent = np.arange(n - EST_RECENT, n, dtype=np.int64)
    return 0, recent, centres, n_mid


def estimate_z(score_of, n: int) -> float:
    """Reference estimate Z (binades) for one row of n keys.  `score_of(idx)` returns the
    base-2 scores of the keys in the integer array idx.

    n <= 192: the exact log-sum-exp of all keys.  Otherwise the mass of the sink and the
    63 recent keys is exact, and the middle's mass is n_mid times the mean weight of the
    128 stratum centres after dropping the 8 largest (the trim keeps one heavy centre
    from being multiplied by its whole stratum, and biases Z low, where the paper's
    estimate sits).  PARITY UNPINNED: the paper gives no formula for this estimate."""
    if n <= 0:
        return -np.inf
    idx = estimator_indices(n)
    if idx is None:
        s = np.asarray(score_of(np.arange(n, dtype=np.int64)), dtype=np.float64)
        m = s.max()
        return float(m + math.log2(np.exp2(s - m).sum()))
    sink, recent, centres, n_mid = idx
    s_sink = float(np.asarray(score_of(np.array([sink], dtype=np.int64)), dtype=np.float64)[0])
    s_rec = np.asarray(score_of(recent), dtype=np.float64)
    s_cen = np.asarray(score_of(centres), dtype=np.float64)
    m = max(s_sink, s_rec.max(), s_cen.max())
    w_cen = np.sort(np.exp2(s_cen - m))           # ascending
    kept = w_cen[: EST_STRATA - EST_TRIM]
    mid = n_mid * kept.mean()
    total = 2.0 ** (s_sink - m) + np.exp2(s_rec - m).sum() + mid
    return float(m + math.log2(total))


# --------------------------------------------------------------------------- order-free add
def grid_sum(values: Sequence[float], b: int = 61):
    """Eq. 3 with the bound taken from the terms themselves: B = C * 2^(e_max+1) where
    2^e_max <= max|g_c| < 2^(e_max+1), alpha = 2^(b - ceil(log2 B)); the terms are
    rounded to nearest-even on that grid and added as exact integers.  Returns
    (sum as float, integer sum, log2(alpha)).  Any order or grouping of `values` gives
    the same integers (Prop. 2)."""
    vals = [float(v) for v in values]
    C = len(vals)
    mx = max((abs(v) for v in vals), default=0.0)
    if C == 0 or mx == 0.0:
        return 0.0, 0, 0
    e_max = math.frexp(mx)[1] - 1                 # mx in [2^e_max, 2^(e_max+1))
    ceil_log2_C = (C - 1).bit_length()
    shift = b - (ceil_log2_C + e_max + 1)         # log2(alpha)
    total = 0
    for v in vals:
        mant, ex = math.frexp(v)                  # v = mant * 2^ex, exact
        num = int(mant * (1 << 53))               # exact integer
        e = ex - 53 + shift
        if e >= 0:
            g = num << e
        else:                                      # round half to even at 2^-e
            d = 1 << (-e)
            qv, r = divmod(num, d)
            if 2 * r > d or (2 * r == d and (qv & 1)):
                qv += 1
            g = qv
        total += g
    return math.ldexp(total, -shift) if abs(total) < (1 << 1000) else float("inf"), total, shift


# --------------------------------------------------------------------------- batch plumbing
def gather_paged(pool: np.ndarray, page_row: np.ndarray, n: int, page_size: int) -> np.ndarray:
    """Logical rows 0..n-1 of one request from a page pool [num_pages, page_size, ...]:
    logical key j lives in page page_row[j // page_size], row j % page_size."""
    j = np.arange(n)
    return pool[page_row[j // page_size], j % page_size]


def decode_batch(q, k_rows, v_rows, seqlens, scale=None, Z=None, T=math.inf, rows=None):
    """Decode a batch, one row (request b, query head h) at a time.

    q [B, Hq, D] float64.  k_rows(b, kvh) / v_rows(b, kvh) return that request's logical
    [n_b, D] float64 key / value rows of one KV head (the caller hides contiguous vs
    paged layout there).  GQA: query head h reads KV head h // (Hq / Hkv), given through
    `rows` = iterable of (b, h, kvh); default: all rows with Hkv = Hq.
    Z: None -> dense reference; else array [B, Hq] of references (binades).
    Returns dict {(b, h): (o, lse2)}."""
    B, Hq, D = q.shape
    if rows is None:
        rows = [(b, h, h) for b in range(B) for h in range(Hq)]
    out = {}
    cache = {}
    for (b, h, kvh) in rows:
        key = (b, kvh)
        if key not in cache:
            cache.clear()
            cache[key] = (np.asarray(k_rows(b, kvh), dtype=np.float64),
                          np.asarray(v_rows(b, kvh), dtype=np.float64))
        Kb, Vb = cache[key]
        n = int(seqlens[b])
        s = scores(q[b, h], Kb[:n], scale)
        if Z is None:
            out[(b, h)] = dense_row(s, Vb[:n])
        else:
            o, lse, _, _ = fold_row(s, Vb[:n], float(Z[b, h]), T)
            out[(b, h)] = (o, lse)
    return out
