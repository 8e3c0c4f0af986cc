"""CPU oracle for the two-plane INT8 key cache of fold decode.

TEST INFRASTRUCTURE ONLY, like ``fold_oracle``: the slow, plain statement of what the
two-plane path computes.  It shares no code with the CUDA library; only the tests, the smoke
check and the benchmark's CPU-baseline leg call it.

What is here, with the passage each function restates (Section 4, "Cache format" and
"Weight-gated reads"; Algorithm 1):
  hadamard            the orthonormal (Sylvester) Hadamard matrix, float64: the definition the
                      fast transform below is pinned against
  rotate_f32          the same rotation as the cache writer performs it: FP32 butterflies in a
                      fixed order, then one multiply by fp32(1/sqrt(D))
  split_planes        k = e (a + b/256): BF16 scale rounded up so plane A never saturates, two
                      INT8 planes.  The codes are integers decided by FP32 arithmetic, so this
                      function works in FP32, operation by operation, as the writer does
  quantize_rows       rotate_f32 + split_planes for an array of rows (keys at cache write, the
                      query rows at every step, which Section 4 splits like the keys)
  dequantize          e (a + b/256) in float64
  plane_products      the four integer products c^aa, c^ab, c^ba, c^bb (exact)
  coarse_scores /
  refined_scores      Algorithm 1: eta e (c^aa + c^ab/256) and the plane-B correction, float64
  auto_refine_tau     the refine gate when the caller gives none.  PARITY UNPINNED by the paper (it
                      gives no formula); the reading taken is in the docstring
  e4m3_values / round_e4m3 / quantize_values / widen_values
                      Section 4 "Cache format": values as two E4M3 planes under a power-of-two scale,
                      v ~ 2^k (v1 + v2), the second plane read only for keys whose weight matters
                      ("refine V"); E4M3 = 1-4-3 bits, bias 7, no infinities, largest value 448
  running_mean        Section 4 "Depth as a dial": the cut model of the 8-bit value format, the mean value row of
                      the sequence (BF16)
  fold_group_planes   Algorithm 1 for one (sequence, kv head): verdict bits ORed over the
                      group's rows, final weights, (A, L) per row; also counts the bytes the
                      gates ask for (130 + 128 r_K + 256 lambda per key at D = 128)
  fold_levels_planes  a cascade over two-plane levels for one kv head (Appendix "Cascades and drafts";
                      Prop. 1(i)): every level's sequence is Algorithm 1 over the rows of the requests
                      stacked on it, in blocks of 16 rows with their own verdicts; the levels' (A, L) add
"""
from __future__ import annotations

import math
from typing import Optional

import numpy as np

from . import fold_oracle as O

F32 = np.float32


# --------------------------------------------------------------------------- rotation
def hadamard(D: int) -> np.ndarray:
    """Orthonormal Sylvester-Hadamard matrix H_D (D a power of two), float64: H H^T = I."""
    assert D >= 1 and D & (D - 1) == 0
    H = np.ones((1, 1))
    while H.shape[0] < D:
        H = np.block([[H, H], [H, -H]])
    return H / math.sqrt(D)


def rotate_f32(x: np.ndarray) -> np.ndarray:
    """Rows of x [.., D] (values exactly representable in FP32) times H_D, computed as the cache
    writer computes it: log2(D) butterfly stages with strides 1, 2, 4, ..., each an FP32 add and
    an FP32 subtract ((lo, hi) -> (lo + hi, lo - hi)), then one FP32 multiply by fp32(1/sqrt(D))."""
    y = np.array(x, dtype=F32)
    D = y.shape[-1]
    assert D & (D - 1) == 0
    h = 1
    while h < D:
        y = y.reshape(y.shape[:-1] + (D // (2 * h), 2, h))
        lo, hi = y[..., 0, :], y[..., 1, :]
        y = np.stack([(lo + hi).astype(F32), (lo - hi).astype(F32)], axis=-2).reshape(y.shape[:-3] + (D,))
        h *= 2
    return (y * F32(1.0 / math.sqrt(D))).astype(F32)


# --------------------------------------------------------------------------- planes
def bf16_round_up(x: np.ndarray) -> np.ndarray:
    """Smallest BF16 value >= x, for x >= 0 finite FP32; returned as FP32."""
    u = np.asarray(x, dtype=F32).view(np.uint32)
    up = np.where((u & np.uint32(0xFFFF)) != 0, (u >> np.uint32(16)) + np.uint32(1), u >> np.uint32(16))
    return (up.astype(np.uint32) << np.uint32(16)).view(F32)


def split_planes(y: np.ndarray):
    """y [.., D] FP32 -> (a int8, b int8, e FP32 holding a BF16 value) with y ~ e (a + b/256).
    Section 4 "Cache format": a scale per row, rounded UP so plane A never saturates; a row's code
    depends on that row alone.  Every step is one FP32 operation (the reading of how the codes are
    decided):  e = bf16_up(max|y| / 127)  (1 when the row is all zero);  t = y / e;
    a = rint(t) kept within +-127;  b = rint((t - a) * 256) kept within [-128, 127]."""
    y = np.asarray(y, dtype=F32)
    m = np.abs(y).max(axis=-1)
    e = np.where(m > 0, bf16_round_up((m / F32(127.0)).astype(F32)), F32(1.0)).astype(F32)
    t = (y / e[..., None]).astype(F32)
    a = np.clip(np.rint(t), -127, 127).astype(F32)
    r = (t - a).astype(F32)                                   # exact: t minus its nearest integer
    b = np.clip(np.rint((r * F32(256.0)).astype(F32)), -128, 127)
    return a.astype(np.int8), b.astype(np.int8), e


def quantize_rows(x: np.ndarray):
    """Rotate and split rows x [.., D] (FP32-representable values): returns (a, b, e)."""
    return split_planes(rotate_f32(x))


def dequantize(a, b, e) -> np.ndarray:
    return np.asarray(e, dtype=np.float64)[..., None] * (np.asarray(a, dtype=np.float64) + np.asarray(b, dtype=np.float64) / 256.0)


# --------------------------------------------------------------------------- scores
def plane_products(ka, kb, qa, qb):
    """The four integer products of Algorithm 1 for one query row: keys [n, D] int8, query [D] int8.
    Returns (c_aa, c_ab, c_ba, c_bb), int64 [n] each, exact."""
    ka = np.asarray(ka, dtype=np.int64); kb = np.asarray(kb, dtype=np.int64)
    qa = np.asarray(qa, dtype=np.int64); qb = np.asarray(qb, dtype=np.int64)
    return ka @ qa, ka @ qb, kb @ qa, kb @ qb


def coarse_scores(ka, ke, qa, qb, eta: float) -> np.ndarray:
    """Algorithm 1, coarse score (before the reference is subtracted): eta e_j (c^aa_j + c^ab_j / 256).
    `eta` is the query row's scale times log2(e) times the softmax scale, so the result is in binades."""
    ka = np.asarray(ka, dtype=np.int64)
    c_aa = ka @ np.asarray(qa, dtype=np.int64)
    c_ab = ka @ np.asarray(qb, dtype=np.int64)
    return float(eta) * np.asarray(ke, dtype=np.float64) * (c_aa + c_ab / 256.0)


def refine_terms(kb, ke, qa, qb, eta: float) -> np.ndarray:
    """Algorithm 1, the plane-B correction: eta e_j (c^ba_j + c^bb_j / 256) / 256."""
    kb = np.asarray(kb, dtype=np.int64)
    c_ba = kb @ np.asarray(qa, dtype=np.int64)
    c_bb = kb @ np.asarray(qb, dtype=np.int64)
    return float(eta) * np.asarray(ke, dtype=np.float64) * (c_ba + c_bb / 256.0) / 256.0


def refined_scores(ka, kb, ke, qa, qb, eta: float) -> np.ndarray:
    return coarse_scores(ka, ke, qa, qb, eta) + refine_terms(kb, ke, qa, qb, eta)


# --------------------------------------------------------------------------- E4M3 value planes
def e4m3_values() -> np.ndarray:
    """The 256 E4M3 codes as float64: sign, 4 exponent bits (bias 7), 3 mantissa bits; exponent 0 is
    subnormal (m/8 * 2^-6), there are no infinities, 0x7f / 0xff are NaN, the largest value is 448."""
    v = np.empty(256)
    for b in range(256):
        sgn = -1.0 if b & 0x80 else 1.0
        e, m = (b >> 3) & 0xF, b & 7
        if e == 15 and m == 7:
            v[b] = np.nan
        elif e == 0:
            v[b] = sgn * (m / 8.0) * 2.0 ** -6
        else:
            v[b] = sgn * (1.0 + m / 8.0) * 2.0 ** (e - 7)
    return v


_E4M3 = e4m3_values()
_E4M3_POS = _E4M3[:0x7f]                                     # codes 0x00 .. 0x7e ascend from 0 to 448


def round_e4m3(x: np.ndarray) -> np.ndarray:
    """x -> the E4M3 code (uint8) nearest to x, ties to the even code, magnitudes beyond 448 saturate
    to 448 (the "satfinite" conversion)."""
    x = np.asarray(x, dtype=np.float64)
    a = np.minimum(np.abs(x), 448.0)
    hi = np.clip(np.searchsorted(_E4M3_POS, a, side="left"), 1, 0x7e)
    lo = hi - 1
    dlo, dhi = a - _E4M3_POS[lo], _E4M3_POS[hi] - a
    code = np.where((dhi < dlo) | ((dhi == dlo) & (hi % 2 == 0)), hi, lo).astype(np.uint8)
    return np.where(np.signbit(x), code | np.uint8(0x80), code).astype(np.uint8)


def quantize_values(V: np.ndarray, scale_log2: int):
    """Value rows -> two E4M3 planes under the scale 2^scale_log2 (a power of two per layer, given by the
    caller): p1 = e4m3(v / 2^k), p2 = e4m3(v / 2^k - p1).  Both subtractions and the scaling are exact for
    BF16 inputs, so the codes depend on nothing but the rounding rule.  Returns (p1, p2) uint8."""
    x = np.asarray(V, dtype=np.float64) * 2.0 ** (-scale_log2)
    p1 = round_e4m3(x)
    p2 = round_e4m3(x - _E4M3[p1])
    return p1, p2


def widen_values(p1, p2, scale_log2: int, refined) -> np.ndarray:
    """What the scan multiplies: 2^k * v1 for a key read from plane 1 alone, 2^k * bf16(v1 + v2) for a key
    whose second plane is read (`refined` bool [n]).  v1 and v2 widen to BF16 exactly; their sum can need
    nine significant bits and is rounded to BF16 once (the reading taken: the value product runs in BF16)."""
    v1 = _E4M3[np.asarray(p1)]
    v2 = _E4M3[np.asarray(p2)]
    both = O.round_to_bf16(v1 + v2)
    return np.where(np.asarray(refined, dtype=bool)[:, None], both, v1) * 2.0 ** scale_log2


def running_mean(V: np.ndarray) -> np.ndarray:
    """The cut model of the 8-bit value format (Section 4, "Depth as a dial": with 8-bit values the
    model is a mean kept per request and needs no fitting): the mean of all the value rows the sequence holds so far (for one
    kv head), rounded to BF16 as the cache stores it.  V [n, D] -> [D]."""
    V = np.asarray(V, dtype=np.float64)
    return O.round_to_bf16(V.sum(axis=0) / V.shape[0])


def auto_refine_tau_v(n: int) -> float:
    """The refine-V gate when the caller gives none.  Reading (PARITY UNPINNED, like auto_refine_tau): a key's
    second value plane is read when some row of its group gives it at least 1/(2n) of the row's mass,
    tau_V = max(log2(n) + 1, 4).  On the synthetic rows plane 1 alone leaves the dense output at 13 x the BF16
    online-softmax error, tau_V = log2 n at 0.6-1.6 x, log2 n + 2 at 0.1-0.3 x."""
    return max(math.log2(max(n, 1)) + 1.0, 4.0)


def auto_refine_tau(n: int) -> float:
    """The refine gate tau_K used when the caller gives none.  The paper says only that the
    thresholds depend on the request's length and are placed where plane B begins to affect the error.  Reading:  tau_K = max(log2(n) - 2, 4): a key reads plane B when some row of its
    group gives it at least four times the uniform share 1/n of the row's mass (every key of a short row).
    On the synthetic rows of this build that refines about a quarter of the keys at 4K-32K context and
    leaves the dense output within 0.7 x the BF16 online-softmax error of exact attention (plane A alone:
    3 x that error; every key refined: 0.03 x)."""
    return max(math.log2(max(n, 1)) - 2.0, 4.0)


def fold_group_planes(ka, kb, ke, V, qa, qb, eta, Z, T: float = math.inf, tau: Optional[float] = None, visible=None,
                      v_mean=None, value_planes=None, tau_v: Optional[float] = None, v_run_mean=None):
    """Algorithm 1 for the rows of one (sequence, kv head) group over all its keys.
    ka, kb [n, D] int8; ke [n]; V [n, D]; qa, qb [R, D] int8; eta [R]; Z [R] (binades).
    tau: refine gate in binades (None: auto_refine_tau(n); inf: refine every live key; negative:
    never).  Per key j:  live_j = OR_i [coarse_ij - Z_i >= -T];  refine_j = live_j AND
    OR_i [coarse_ij - Z_i >= -tau];  s_ij = coarse_ij (+ correction_ij if refine_j);  the weight
    2^(s_ij - Z_i) always adds to L_i and adds weight x value to A_i iff live_j and s_ij - Z_i >= -T.
    visible [R, n] bool (drafts and verification trees, Section 4 "Value product": extra query rows masked to
    their ancestors): a key a row does not see has coarse score -inf for that row -- weight exactly 0, and no
    say in the verdicts.
    v_mean [ceil(n/64), D] switches the block tail on (``fold_oracle.block_means``; Algorithm 1, the step that gives
    the cut keys' weights to the tile's virtual row): a key whose weight row i does not keep in A adds weight x the mean value row
    of its 64-key block to A_i instead of nothing.
    value_planes = (p1, p2, scale_log2) replaces V by two E4M3 planes: refine_v_j = live_j AND
    OR_i [coarse_ij - Z_i >= -tau_v] (tau_v None: auto_refine_tau_v(n); inf: every live key; negative: none), and
    key j's value row is widen_values(...) with that mask (`V` is then ignored).
    v_run_mean [D] (with value_planes; `running_mean`): the 8-bit format's cut model -- a key whose weight row i does
    not keep in A adds weight x the sequence's mean value row to A_i.
    Returns (A [R, D], L [R], info) with info = live / refine masks and the bytes-per-key count."""
    ka = np.asarray(ka); kb = np.asarray(kb)
    V = np.asarray(V, dtype=np.float64) if value_planes is None else None
    n, D = ka.shape
    R = len(eta)
    if tau is None:
        tau = auto_refine_tau(n)
    coarse = np.stack([coarse_scores(ka, ke, qa[i], qb[i], eta[i]) - Z[i] for i in range(R)])      # [R, n]
    if visible is not None:
        coarse = np.where(np.asarray(visible, dtype=bool), coarse, -np.inf)
    live = np.isfinite(coarse).any(axis=0) if math.isinf(T) else (coarse >= -T).any(axis=0)
    refine = live & ((coarse >= -tau).any(axis=0) if tau >= 0 else np.zeros(n, dtype=bool))
    refine_v = np.zeros(n, dtype=bool)
    if value_planes is not None:
        if tau_v is None:
            tau_v = auto_refine_tau_v(n)
        refine_v = live & ((coarse >= -tau_v).any(axis=0) if tau_v >= 0 else np.zeros(n, dtype=bool))
        V = widen_values(value_planes[0], value_planes[1], value_planes[2], refine_v)
    A = np.zeros((R, D)); L = np.zeros(R)
    for i in range(R):
        s = coarse[i] + np.where(refine, refine_terms(kb, ke, qa[i], qb[i], eta[i]), 0.0)
        p = np.exp2(s)
        keep = live if math.isinf(T) else (live & (s >= -T))
        L[i] = p.sum()
        A[i] = (p[keep, None] * V[keep]).sum(axis=0)
        if v_mean is not None:
            vm = np.asarray(v_mean, dtype=np.float64)
            block_of = np.arange(n) // O.BLOCK_KEYS
            for b in np.unique(block_of[~keep]):
                A[i] = A[i] + p[~keep & (block_of == b)].sum() * vm[b]
        if v_run_mean is not None:
            A[i] = A[i] + p[~keep].sum() * np.asarray(v_run_mean, dtype=np.float64)
    lam, rk, rv = (float(m.mean()) if n else 0.0 for m in (live, refine, refine_v))
    v_bytes = 2 * D * lam if value_planes is None else D * lam + D * rv          # (Section 4: the 256 value bytes become 128 + 128 r_V)
    info = dict(live=live, refine=refine, refine_v=refine_v, coarse=coarse, bytes_per_key=(D + 2) + D * rk + v_bytes)
    return A, L, info


def fold_levels_planes(levels, qa, qb, eta, Z, T: float = math.inf, tau: Optional[float] = None, block_rows: int = 16):
    """A cascade on two-plane keys, one kv head.  `levels` = [(stack, [(ka, kb, ke, V), ...]), ...]: level l holds one
    key sequence per `stack` consecutive requests (request b reads sequence b // stack; a shared prefix is stack =
    all requests, a private suffix stack = 1).  qa, qb [B, G, D] int8; eta, Z [B, G].
    Readings (the paper states Algorithm 1 for one group and says a cascade level stacks the rows of the requests
    that hold it): a sequence's rows -- request-major, the group's rows within a request -- are cut into blocks of
    `block_rows`, each block is `fold_group_planes` over its own rows (its verdicts ORed over the block), and
    tau = None takes `auto_refine_tau` of the LEVEL's own sequence length.  Partials of one row under one reference
    add (Prop. 1(i)).  A sequence may carry a fifth entry, a dict of `fold_group_planes`' optional arguments for it
    (`v_mean`: its block means; `value_planes`, `tau_v`: its E4M3 value planes and their gate, tau_v None = the
    level's own `auto_refine_tau_v`; `v_run_mean`: its mean value row).  Returns (A [B, G, D], L [B, G], infos) with
    infos = [(level, sequence, rows of the block as (b, g) pairs, info of fold_group_planes)]."""
    qa = np.asarray(qa); qb = np.asarray(qb)
    B, G, D = qa.shape
    A = np.zeros((B, G, D)); L = np.zeros((B, G))
    infos = []
    for li, (stack, seqs) in enumerate(levels):
        assert B % stack == 0 and len(seqs) == B // stack
        for j, entry in enumerate(seqs):
            ka, kb, ke, V = entry[:4]
            extra = dict(entry[4]) if len(entry) > 4 else {}
            n = np.asarray(ka).shape[0]
            if n == 0:
                continue
            rows = [(b, g) for b in range(j * stack, (j + 1) * stack) for g in range(G)]
            for r0 in range(0, len(rows), block_rows):
                blk = rows[r0:r0 + block_rows]
                a, l, info = fold_group_planes(ka, kb, ke, V, np.stack([qa[b, g] for b, g in blk]), np.stack([qb[b, g] for b, g in blk]),
                                               np.array([eta[b][g] for b, g in blk], dtype=np.float64),
                                               np.array([Z[b][g] for b, g in blk], dtype=np.float64), T,
                                               auto_refine_tau(n) if tau is None else tau, **extra)
                for i, (b, g) in enumerate(blk):
                    A[b, g] += a[i]; L[b, g] += l[i]
                infos.append((li, j, blk, info))
    return A, L, infos


def estimate_z_planes(ka, kb, ke, qa, qb, eta: float) -> float:
    """The 192-key reference estimate (``fold_oracle.estimate_z``) on two-plane scores: the sampled keys
    are scored with both planes."""
    n = ka.shape[0]
    return O.estimate_z(lambda idx: refined_scores(ka[idx], kb[idx], np.asarray(ke)[idx], qa, qb, eta), n)
