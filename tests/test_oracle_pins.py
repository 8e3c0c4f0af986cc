"""Pins for the float64 oracle: each test ties one oracle function to something other
than itself -- a library routine, exact rational arithmetic, a closed form, a theorem of
the paper (Prop. 1, Prop. 2), or a hand-computed example."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import fold_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rng(seed):
    return np.random.default_rng(seed)


def _bf16ish(x):
    """Random data rounded to BF16 so products are realistic cache contents."""
    return O.round_to_bf16(x)


def _row(seed, n=300, D=32, sink=True):
    r = _rng(seed)
    q = _bf16ish(r.standard_normal(D))
    K = _bf16ish(r.standard_normal((n, D)))
    V = _bf16ish(r.standard_normal((n, D)))
    if sink:
        K[0] = _bf16ish(K[0] * 8)
    return q, K, V


# ------------------------------------------------------------------ O-1 dense
def test_dense_matches_torch_sdpa_float64():
    # library routine: torch scaled_dot_product_attention on CPU in float64
    for seed, (n, D) in enumerate([(1, 16), (7, 64), (513, 128)]):
        q, K, V = _row(seed, n, D)
        o, lse = O.dense_row(O.scores(q, K), V)
        tq = torch.from_numpy(q).view(1, 1, 1, D)
        tk = torch.from_numpy(K).view(1, 1, n, D)
        tv = torch.from_numpy(V).view(1, 1, n, D)
        ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv).view(D).numpy()
        assert np.abs(o - ref).max() < 1e-13
        nat = torch.logsumexp((tk.view(n, D) @ tq.view(D)) / math.sqrt(D), 0).item()
        assert abs(lse - nat * O.LOG2E) < 1e-12


def test_dense_exact_rationals_on_integer_scores():
    # integer base-2 scores make every weight a power of two: the quotient is an exact rational
    s = np.array([3, -2, 0, 5, 5, 1, -7], dtype=np.float64)
    V = np.array([[1, -2], [3, 4], [-5, 6], [7, 8], [-9, 10], [11, -12], [13, 14]], dtype=np.float64)
    w = [Fraction(2) ** int(x) for x in s]
    Lr = sum(w)
    for d in range(2):
        exact = sum(wi * Fraction(int(v)) for wi, v in zip(w, V[:, d])) / Lr
        o, lse = O.dense_row(s, V)
        assert abs(o[d] - float(exact)) < 1e-15
    assert abs(lse - math.log2(float(Lr))) < 1e-14


def test_scores_base2_and_scale():
    q, K, _ = _row(3, 10, 64)
    s = O.scores(q, K)
    nat = (K @ q) / 8.0
    assert np.allclose(np.exp2(s), np.exp(nat), rtol=1e-13)
    assert np.allclose(O.scores(q, K, 0.5), 0.5 * O.LOG2E * (K @ q))


def test_closed_forms():
    q, K, V = _row(4, 1, 16, sink=False)
    o, lse = O.dense_row(O.scores(q, K), V)
    assert np.array_equal(o, V[0]) and lse == O.scores(q, K)[0]
    # q = 0: uniform weights -> mean of V, lse = log2 n
    _, K, V = _row(5, 37, 16)
    s = O.scores(np.zeros(16), K)
    o, lse = O.dense_row(s, V)
    assert np.allclose(o, V.mean(0), atol=1e-15) and abs(lse - math.log2(37)) < 1e-15
    o2, lse2, _, _ = O.fold_row(s, V, Z=3.0)
    assert np.allclose(o2, V.mean(0), atol=1e-15) and abs(lse2 - math.log2(37)) < 1e-14


# ------------------------------------------------------------------ O-2 declared reference
def test_prop1_ii_shift_invariance():
    # Prop. 1(ii): A/L equals softmax attention for every finite Z; range from Section 3 (80 binades)
    for seed in range(4):
        q, K, V = _row(10 + seed, 400, 64)
        s = O.scores(q, K)
        o_ref, lse_ref = O.dense_row(s, V)
        for dz in (-80, -30, 0, 30, 80):
            o, lse, A, L = O.fold_row(s, V, Z=lse_ref + dz)
            assert np.abs(o - o_ref).max() <= 1e-12
            assert abs(lse - lse_ref) <= 1e-12
            assert abs(math.log2(L) + dz) < 1e-9      # L = 2^(lse - Z)


def test_prop1_i_additivity_permutation_and_partition():
    q, K, V = _row(20, 1000, 32)
    s = O.scores(q, K)
    Z = 2.5
    o1, l1, A1, L1 = O.fold_row(s, V, Z, T=16.0)
    r = _rng(0)
    perm = r.permutation(1000)
    cuts = np.sort(r.choice(np.arange(1, 1000), 9, replace=False))
    ranges = np.split(perm, cuts)
    o2, l2, A2, L2 = O.fold_row(s, V, Z, T=16.0, ranges=ranges)
    assert np.abs(o1 - o2).max() <= 1e-12 and abs(l1 - l2) <= 1e-12
    # interleaved by 64-key tile over 8 splits, as the decode kernel assigns tiles
    tiles = [np.arange(t, min(t + 64, 1000)) for t in range(0, 1000, 64)]
    ranges = [np.concatenate(tiles[k::8]) for k in range(8)]
    o3, l3, _, _ = O.fold_row(s, V, Z, T=16.0, ranges=ranges[::-1])
    assert np.abs(o1 - o3).max() <= 1e-12 and abs(l1 - l3) <= 1e-12


def test_additivity_exact_on_dyadic_inputs():
    # every term dyadic -> every ordering and split gives identical bits
    s = np.array([2, 5, 3, 6, 1, 4, 0, 7], dtype=np.float64)
    V = np.arange(16, dtype=np.float64).reshape(8, 2)
    base = O.fold_row(s, V, Z=4.0)
    for ranges in ([slice(0, 3), slice(3, 8)], [np.array([7, 0, 3]), np.array([1, 2]), np.array([6, 5, 4])]):
        got = O.fold_row(s, V, Z=4.0, ranges=ranges)
        assert np.array_equal(base[0], got[0]) and base[1] == got[1] and base[3] == got[3]


def test_worked_example_z4_golden():
    rows, kv = [], {}
    for line in open(os.path.join(GOLDEN, "worked_example_z4.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        parts = line.split()
        if parts[0][0].isdigit():
            rows.append([float(x) for x in parts])
        else:
            kv[parts[0]] = float(parts[1])
    rows = np.array(rows)
    s, v, w = rows[:, 1], rows[:, 2:3], rows[:, 3]
    Z = kv["Z"]
    assert np.array_equal(np.exp2(s - Z), w)
    o, lse, A, L = O.fold_row(s, v, Z)
    assert L == kv["L"] and A[0] == kv["A"]
    assert Fraction(A[0]) / Fraction(L) == Fraction(int(kv["o_num"]), int(kv["o_den"]))
    # the online-softmax stream ends at the stated (A, L, m) and the same quotient
    m = max(s)
    assert m == kv["online_m"]
    wm = np.exp2(s - m)
    assert wm.sum() == kv["online_L"] and (wm * v[:, 0]).sum() == kv["online_A"]
    od, _ = O.dense_row(s, v)
    assert od[0] == o[0] == kv["A"] / kv["L"]
    # Eq. 1 merge of two halves reaches the same value
    oa, la = O.dense_row(s[:2], v[:2]); ob, lb = O.dense_row(s[2:], v[2:])
    om, lm = O.lse_merge(oa, la, ob, lb)
    assert abs(om[0] - o[0]) < 1e-15 and abs(lm - lse) < 1e-15
    # ... in either order and for an uneven cut (the two log-sum-exps differ, whichever is larger)
    for cut in (1, 4):
        oa, la = O.dense_row(s[:cut], v[:cut]); ob, lb = O.dense_row(s[cut:], v[cut:])
        assert la != lb
        for (x, lx, y, ly) in ((oa, la, ob, lb), (ob, lb, oa, la)):
            om, lm = O.lse_merge(x, lx, y, ly)
            assert abs(om[0] - o[0]) < 1e-15 and abs(lm - lse) < 1e-15


def test_bf16_online_softmax_two_key_example():
    # the yardstick's defining choices on two keys, by hand: P is rounded to BF16 for the value product, L sums the
    # unrounded FP32 weights, the output is rounded to BF16.  Scores 0 and -0.5 binades: p = (1, 2^-0.5 = 0.70710677),
    # bf16(p_2) = 0.70703125; values (0, 12.5625): A = 0.70703125 * 12.5625 = 8.88208, L = 1.70710677 -> 5.203002,
    # just below the BF16 tie 5.203125 -> 5.1875.  With P left unrounded it would be 5.203558 -> 5.21875.
    D = 4
    q = np.zeros(D); q[0] = 1.0
    K = np.zeros((2, D)); K[1, 0] = -0.5 / (O.LOG2E / math.sqrt(D))
    V = np.zeros((2, D)); V[1, 0] = 12.5625
    got = O.online_softmax_bf16(q, K, V)
    assert got[0] == 5.1875 and not got[1:].any()
    # the other way round, one key per tile: the first key's weight is 1 when it is multiplied, and the maximum found
    # afterwards rescales A and L by the FP32 factor 2^-0.5, which is never rounded to BF16: the other side of the tie
    assert O.online_softmax_bf16(q, K[::-1], V[::-1], tile=1)[0] == 5.21875


def test_cut_report_by_hand():
    # Z = 0, T = 4: keys at 0, -3, -4 (on the threshold: live), -4.0005 (just cut), -9 binades; band 2^-10 holds keys 2, 3
    s = np.array([0.0, -3.0, -4.0, -4.0005, -9.0])
    V = np.array([[1.0, -2.0], [0.5, 0.25], [3.0, -7.0], [-5.0, 4.0], [100.0, 100.0]])
    p = 2.0 ** s
    rep = O.cut_report(s, V, 0.0, 4.0)
    assert rep["live_frac"] == 3 / 5
    assert abs(rep["cut_mass"] - (p[3] + p[4]) / p.sum()) < 1e-15
    assert abs(rep["slack"] - (p[2] * 7.0 + p[3] * 5.0) / p.sum()) < 1e-15      # weight x the row's largest |value|
    assert O.cut_report(s, V, 0.0, math.inf) == {"live_frac": 1.0, "cut_mass": 0.0, "slack": 0.0}


def test_mass_is_kept_for_every_depth():
    # cut keys add weight to L and nothing to A ("Depth as a dial")
    q, K, V = _row(30, 2000, 64)
    s = O.scores(q, K)
    _, lse = O.dense_row(s, V)
    Z = lse - 0.7
    ref = O.fold_row(s, V, Z)
    for T in (0.0, 4.0, 8.0, 16.0, 40.0):
        o, l, A, L = O.fold_row(s, V, Z, T)
        assert L == ref[3] and l == ref[1]
    # constant values: o_inf = c, o_T = c * (1 - cut mass): separates "mass kept" from "mass dropped"
    Vc = np.full_like(V, 3.25)
    for T in (2.0, 6.0):
        o, _, _, L = O.fold_row(s, Vc, Z, T)
        rep = O.cut_report(s, Vc, Z, T)
        assert rep["cut_mass"] > 0.01
        assert np.allclose(o, 3.25 * (1 - rep["cut_mass"]), rtol=1e-12)
    o, _, _, _ = O.fold_row(s, Vc, Z)
    assert np.allclose(o, 3.25, rtol=1e-13)


def test_truncation_identity_bound_and_monotone_live_set():
    q, K, V = _row(31, 3000, 64)
    s = O.scores(q, K)
    _, lse = O.dense_row(s, V)
    Z = lse - 1.0
    o_inf, _, _, L = O.fold_row(s, V, Z)
    p = np.exp2(s - Z)
    prev_live = None
    for T in (1.0, 3.0, 6.0, 9.0):
        o_T, _, _, _ = O.fold_row(s, V, Z, T)
        cut = (s - Z) < -T
        assert np.allclose(o_inf - o_T, (p[cut, None] * V[cut]).sum(0) / L, atol=1e-14)
        assert np.abs(o_inf - o_T).max() <= cut.sum() * 2.0 ** -T * np.abs(V).max() / L + 1e-15
        live = O.live_mask(s, Z, T)
        assert np.array_equal(live, ~cut)
        if prev_live is not None:
            assert np.all(live[prev_live])           # live set grows with T
        prev_live = live
    # T >= Z - min s reproduces dense exactly; threshold is inclusive (s >= Z - T)
    T_all = Z - s.min()
    assert np.array_equal(O.fold_row(s, V, Z, T_all)[0], o_inf)
    assert O.live_mask(np.array([1.0]), 5.0, 4.0)[0] and not O.live_mask(np.array([0.999]), 5.0, 4.0)[0]


def test_fold_partial_brute_force_loop():
    # brute force on a tiny input: explicit Python loop over keys and channels
    q, K, V = _row(32, 9, 4)
    s = O.scores(q, K)
    Z, T = 1.0, 2.0
    A = [0.0] * 4
    L = 0.0
    for j in range(9):
        w = 2.0 ** (s[j] - Z)
        L += w
        if s[j] >= Z - T:
            for d in range(4):
                A[d] += w * V[j, d]
    a, l = O.fold_partial(s, V, Z, T)
    assert np.allclose(a, A, rtol=1e-14) and abs(l - L) < 1e-14
    assert 0 < O.cut_report(s, V, Z, T)["live_frac"] < 1


def test_gqa_row_independent_of_its_group_and_paged_equals_contiguous():
    r = _rng(40)
    B, Hq, Hkv, D, n, ps = 2, 4, 2, 16, 150, 16
    q = _bf16ish(r.standard_normal((B, Hq, D)))
    K = _bf16ish(r.standard_normal((B, n, Hkv, D)))
    V = _bf16ish(r.standard_normal((B, n, Hkv, D)))
    rows = [(b, h, h // 2) for b in range(B) for h in range(Hq)]
    full = O.decode_batch(q, lambda b, k: K[b, :, k], lambda b, k: V[b, :, k], [n, n - 31], rows=rows)
    # each row alone, as MHA over a duplicated KV head
    for (b, h, kvh) in rows:
        nb = [n, n - 31][b]
        o, lse = O.dense_row(O.scores(q[b, h], K[b, :nb, kvh]), V[b, :nb, kvh])
        assert np.array_equal(o, full[(b, h)][0]) and lse == full[(b, h)][1]
    # paged: scatter rows into a permuted pool and read them back through the page table
    npg = (n + ps - 1) // ps
    perm = r.permutation(B * npg)
    table = perm.reshape(B, npg)
    kpool = np.full((B * npg, ps, Hkv, D), np.nan); vpool = np.full_like(kpool, np.nan)
    for b in range(B):
        for j in range(n):
            kpool[table[b, j // ps], j % ps] = K[b, j]; vpool[table[b, j // ps], j % ps] = V[b, j]
    paged = O.decode_batch(q, lambda b, k: O.gather_paged(kpool, table[b], n, ps)[:, k],
                           lambda b, k: O.gather_paged(vpool, table[b], n, ps)[:, k], [n, n - 31], rows=rows)
    for key in full:
        assert np.array_equal(full[key][0], paged[key][0]) and full[key][1] == paged[key][1]


def test_empty_row():
    o, lse, A, L = O.fold_row(np.zeros(0), np.zeros((0, 8)), 0.0)
    assert not o.any() and lse == -np.inf and L == 0.0


# ------------------------------------------------------------------ O-4 yardstick
def test_bf16_online_softmax_error_band():
    # Table 1 puts BF16 kernels at 1.66e-3..3.13e-3 FP32-relative l2 error on real rows;
    # on peaked synthetic rows the emulation must land in the same decade.
    errs = []
    for seed in range(3):
        r = _rng(50 + seed)
        D, n = 128, 4096
        q = _bf16ish(r.standard_normal(D)); K = _bf16ish(r.standard_normal((n, D)))
        V = _bf16ish(r.standard_normal((n, D))); K[0] = _bf16ish(K[0] * 8)
        ref, _ = O.dense_row(O.scores(q, K), V)
        got = O.online_softmax_bf16(q, K, V)
        assert np.array_equal(O.round_to_bf16(got), got)          # a BF16 kernel writes BF16
        errs.append(np.linalg.norm(got - ref) / np.linalg.norm(ref))
    assert 5e-4 < np.mean(errs) < 6e-3, errs


def test_round_to_bf16_ties_to_even():
    x = np.array([1.0, 1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8, 1.0 + 2 ** -7, -(1.0 + 2 ** -8) - 2 ** -20])
    assert np.array_equal(O.round_to_bf16(x), [1.0, 1.0, 1.0 + 2 ** -6, 1.0 + 2 ** -7, -(1.0 + 2 ** -7)])
    t = torch.randn(1000, dtype=torch.float32)
    assert np.array_equal(O.round_to_bf16(t.numpy()), t.to(torch.bfloat16).to(torch.float64).numpy())
    bits = t.to(torch.bfloat16).view(torch.int16).numpy()
    assert np.array_equal(O.widen_bf16(bits), t.to(torch.bfloat16).to(torch.float64).numpy())


# ------------------------------------------------------------------ O-3 estimator (reading; parity unpinned)
def test_estimator_index_structure():
    for n in (193, 200, 256, 1000, 4096, 32768, 131072):
        sink, recent, centres, n_mid = O.estimator_indices(n)
        assert sink == 0 and n_mid == n - 64
        assert np.array_equal(recent, np.arange(n - 63, n))
        assert len(centres) == 128 and len(np.unique(centres)) == 128
        assert centres.min() >= 1 and centres.max() < n - 63
        edges = [1 + (k * n_mid) // 128 for k in range(129)]
        assert all(edges[k] <= centres[k] < edges[k + 1] for k in range(128))
        assert edges[0] == 1 and edges[-1] == n - 63
        # the key in the MIDDLE of each stratum stands for it (not its first key)
        assert all(centres[k] - edges[k] == (edges[k + 1] - edges[k]) // 2 for k in range(128))
    # strata of exactly 10 keys: 1..10, 11..20, ...: centres 6, 16, 26, ...
    assert np.array_equal(O.estimator_indices(64 + 1280)[2], 6 + 10 * np.arange(128))
    assert O.estimator_indices(192) is None and O.estimator_indices(1) is None


def test_estimator_closed_forms():
    # short rows: the exact log-sum-exp
    r = _rng(60)
    s = r.standard_normal(150) * 3
    m = s.max()
    assert abs(O.estimate_z(lambda i: s[i], 150) - (m + math.log2(np.exp2(s - m).sum()))) < 1e-13
    # constant scores: every sampled weight equal -> the estimate is exact: c + log2 n
    for n in (193, 777, 40000):
        assert abs(O.estimate_z(lambda i: np.full(len(i), 2.5), n) - (2.5 + math.log2(n))) < 1e-12
    # a row owned by its sink: Z ~ s_0
    n = 5000
    s = np.zeros(n); s[0] = 60.0
    assert abs(O.estimate_z(lambda i: s[i], n) - 60.0) < 1e-9
    # up to 8 heavy stratum centres are trimmed away entirely
    s = np.zeros(n)
    _, _, centres, _ = O.estimator_indices(n)
    base = O.estimate_z(lambda i: s[i], n)
    s[centres[[3, 17, 40, 41, 90, 100, 120, 127]]] = 30.0
    assert abs(O.estimate_z(lambda i: s[i], n) - base) < 1e-12
    s[centres[5]] = 30.0                      # a ninth one is not
    assert O.estimate_z(lambda i: s[i], n) > base + 10


def test_estimator_lands_just_below_lse_on_iid_rows():
    # The paper reports the true lse 1.0 binade above Z at the median, never more than 0.9 below.
    gaps = []
    for seed in range(6):
        q, K, V = _row(70 + seed, 8192, 64)
        s = O.scores(q, K)
        _, lse = O.dense_row(s, V)
        Z = O.estimate_z(lambda i: s[i], len(s))
        assert math.isfinite(Z) and abs(s.max() - Z) < 80
        gaps.append(lse - Z)
    assert -0.9 < min(gaps) and max(gaps) < 3.0, gaps


# ------------------------------------------------------------------ order-free add (Eq. 3, Prop. 2)
def test_grid_sum_order_free_and_within_prop2_bound():
    r = _rng(80)
    for C in (1, 2, 7, 512, 2048):
        g = (r.standard_normal(C) * np.exp2(r.integers(-30, 30, C))).astype(np.float32).astype(np.float64)
        val, total, shift = O.grid_sum(g)
        for _ in range(3):
            v2, t2, s2 = O.grid_sum(r.permutation(g))
            assert t2 == total and s2 == shift and v2 == val
        exact = sum(Fraction(x) for x in g)
        B = C * 2.0 ** (math.frexp(np.abs(g).max())[1])
        assert abs(Fraction(val) - exact) <= Fraction(C * B) * Fraction(2) ** -61 + Fraction(abs(val)) * Fraction(2) ** -52
        assert abs(total) < 2 ** 62                 # fits the (b+2)-bit accumulator
    assert O.grid_sum([]) == (0.0, 0, 0) and O.grid_sum([0.0, 0.0])[0] == 0.0
    # Eq. 3 by hand on a coarse grid (b = 4): C = 2 terms, largest 1.0 -> B = 2 * 2^1, alpha = 2^(4 - 2) = 4;
    # 4 * 0.625 = 2.5 -> 2 and 4 * 0.375 = 1.5 -> 2 (ties to even), 4 * 0.875 = 3.5 -> 4, 4 * 0.3 = 1.2 -> 1
    assert O.grid_sum([1.0, 0.625], b=4) == (1.5, 6, 2)
    assert O.grid_sum([1.0, 0.375], b=4) == (1.5, 6, 2)
    assert O.grid_sum([1.0, 0.875], b=4) == (2.0, 8, 2)
    assert O.grid_sum([1.0, -0.3], b=4) == (0.75, 3, 2)
    # C = 5 terms: ceil(log2 5) = 3 -> alpha = 2^(6 - 3 - 1) = 4 for a largest term in [1, 2)
    assert O.grid_sum([1.5, 0.25, 0.25, 0.25, 0.25], b=6) == (2.5, 10, 2)
    # FP32 partials that need no rounding on the grid add exactly
    g = [1.5, 2.0 ** -20, -0.75, 3.0]
    assert O.grid_sum(g)[0] == sum(g)


# ------------------------------------------------------------------ block tail (Section 4, "Depth as a dial")
def test_block_means_brute_force_and_short_last_block():
    r = _rng(40)
    V = _bf16ish(r.standard_normal((150, 8)))                 # blocks of 64, 64 and 22 keys
    m = O.block_means(V)
    assert m.shape == (3, 8)
    for b, (lo, hi) in enumerate([(0, 64), (64, 128), (128, 150)]):
        for d in range(8):
            exact = Fraction(0)
            for j in range(lo, hi):
                exact += Fraction(float(V[j, d]))
            exact /= (hi - lo)
            # stored as BF16: within half a BF16 ulp of the exact rational mean
            assert abs(Fraction(float(m[b, d])) - exact) <= abs(exact) * Fraction(1, 256) + Fraction(1, 2 ** 130)
    # dyadic values with an exactly representable mean come back exactly
    Vd = np.tile(np.array([[1.0, -2.0], [3.0, 6.0]]), (32, 1))           # 64 rows: mean (2, 2)
    assert np.array_equal(O.block_means(Vd), np.array([[2.0, 2.0]]))


def test_block_tail_is_exact_when_values_are_constant_within_blocks():
    # if every key of a block holds the block's mean, replacing cut values by the mean changes nothing:
    # the finite-depth result with the tail must equal dense attention, whatever T cuts
    r = _rng(41)
    n, D = 300, 16
    q = _bf16ish(r.standard_normal(D)); K = _bf16ish(r.standard_normal((n, D)))
    vb = _bf16ish(r.standard_normal(((n + 63) // 64, D)))
    V = vb[np.arange(n) // 64]
    s = O.scores(q, K)
    o_dense, lse_dense = O.dense_row(s, V)
    m = O.block_means(V)
    assert np.array_equal(m, vb)
    for Z in (lse_dense, lse_dense - 3.0):
        for T in (0.5, 2.0, 6.0, 16.0):
            assert (~O.live_mask(s, Z, T)).any() or T == 16.0
            o, lse, _, _ = O.fold_row(s, V, Z, T, v_mean=m)
            assert np.allclose(o, o_dense, rtol=1e-12, atol=1e-13) and abs(lse - lse_dense) < 1e-12
            o_plain, _, _, _ = O.fold_row(s, V, Z, T)
            if (~O.live_mask(s, Z, T)).any():
                assert not np.allclose(o_plain, o_dense, rtol=1e-6)      # without the tail the cut shows


def test_block_tail_identity_brute_force_and_partition_invariance():
    q, K, V = _row(42, n=200, D=8)
    s = O.scores(q, K)
    _, lse = O.dense_row(s, V)
    Z, T = lse - 1.0, 3.0
    m = O.block_means(V)
    o_tail, _, A_tail, L = O.fold_row(s, V, Z, T, v_mean=m)
    o_plain, _, A_plain, L2 = O.fold_row(s, V, Z, T)
    assert L == L2                                                       # the mass is the same either way
    # brute force: A_tail - A_plain = sum over cut keys of p_j * mean of j's block
    extra = np.zeros(8)
    for j in range(200):
        if s[j] - Z < -T:
            extra += 2.0 ** (s[j] - Z) * m[j // 64]
    assert np.allclose(A_tail - A_plain, extra, rtol=1e-12, atol=1e-15)
    # T = inf: nothing is cut, the tail adds nothing
    assert np.array_equal(O.fold_row(s, V, Z, math.inf, v_mean=m)[2], O.fold_row(s, V, Z, math.inf)[2])
    # any partition of the keys, also one that splits blocks, adds up to the same pair
    perm = _rng(43).permutation(200)
    ranges = [perm[:37], perm[37:120], perm[120:]]
    o_parts, _, A_parts, _ = O.fold_row(s, V, Z, T, ranges=ranges, v_mean=m)
    assert np.allclose(A_parts, A_tail, rtol=1e-12, atol=1e-15)


def test_block_tail_reduces_the_truncation_error_on_smooth_values():
    # values that drift slowly along the sequence are well described by their block means
    r = _rng(44)
    n, D = 2000, 16
    q = _bf16ish(r.standard_normal(D)); K = _bf16ish(r.standard_normal((n, D)))
    t = np.arange(n)[:, None] / n
    V = _bf16ish(np.sin(2 * np.pi * (t + np.arange(D)[None, :] / D)) + 0.01 * r.standard_normal((n, D)))
    s = O.scores(q, K)
    o_dense, lse = O.dense_row(s, V)
    T = 11.0                                                             # weights sit near 2^-11: about half are cut
    cut = ~O.live_mask(s, lse, T)
    assert 0.2 < cut.mean() < 0.8
    e_plain = np.linalg.norm(O.fold_row(s, V, lse, T)[0] - o_dense)
    e_tail = np.linalg.norm(O.fold_row(s, V, lse, T, v_mean=O.block_means(V))[0] - o_dense)
    assert e_tail < 0.3 * e_plain


# ------------------------------------------------------------------ drafts (Section 4 "Value product", Appendix "Cascades and drafts")
def test_draft_chain_row_equals_attention_over_its_prefix():
    # draft row r of a chain of m sees the committed keys and drafts 0..r: plain attention over a prefix of the keys
    q, K, V = _row(50, n=300, D=16)
    m = 5
    s = O.scores(q, K)
    for r in range(m):
        sm = O.mask_draft_scores(s, m, (1 << (r + 1)) - 1)
        o, lse = O.dense_row(sm, V)
        keep = 300 - m + r + 1
        ref = torch.nn.functional.scaled_dot_product_attention(
            torch.from_numpy(q)[None, None, None, :], torch.from_numpy(K[:keep])[None, None], torch.from_numpy(V[:keep])[None, None])
        assert np.allclose(o, ref[0, 0, 0].numpy(), rtol=1e-12, atol=1e-14)
        o2, lse2 = O.dense_row(s[:keep], V[:keep])
        assert np.allclose(o, o2, rtol=1e-13) and abs(lse - lse2) < 1e-12


def test_draft_mask_conventions_and_tree_brute_force():
    n, m = 40, 6
    assert O.draft_visible(n, m, (1 << m) - 1).all()                     # every draft visible: no mask at all
    assert O.draft_visible(n, 0, 0).all()
    vis = O.draft_visible(n, m, 0b100101)                                # a tree row: drafts 0, 2 and 5 (itself)
    assert vis[:n - m].all() and list(vis[n - m:]) == [True, False, True, False, False, True]
    # fewer keys than drafts: only the bits that have a key count (key j = n - m + t >= 0)
    assert list(O.draft_visible(2, 4, 0b0100)) == [True, False] and list(O.draft_visible(2, 4, 0b1000)) == [False, True]
    # declared-reference attention over masked scores = the same over the visible keys alone, for every depth
    q, K, V = _row(51, n=n, D=8)
    s = O.scores(q, K)
    sm = O.mask_draft_scores(s, m, 0b100101)
    _, lse = O.dense_row(s[vis], V[vis])
    for T in (math.inf, 6.0, 1.0):
        a = O.fold_row(sm, V, lse - 0.5, T)
        b = O.fold_row(s[vis], V[vis], lse - 0.5, T)
        assert np.allclose(a[0], b[0], rtol=1e-13) and abs(a[1] - b[1]) < 1e-12 and abs(a[3] - b[3]) <= 1e-13 * b[3]
    # the estimator sees the same mask (n <= 192: the exact log-sum-exp of the visible keys)
    assert abs(O.estimate_z(lambda i: sm[i], n) - lse) < 1e-12
