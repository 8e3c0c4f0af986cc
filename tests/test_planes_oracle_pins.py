"""Pins of the two-plane INT8 key oracle (Section 4 "Cache format", "Weight-gated reads"; Algorithm 1)
to things other than itself: the matrix definition of the rotation, hand-worked codes, closed-form
bounds, special cases that reduce to the plain declared-reference functions, and a per-key
brute-force restatement of Algorithm 1."""
import math

import numpy as np
import pytest

from oracle import fold_oracle as O
from oracle import fold_planes_oracle as P


def rng_rows(seed, n, D, spread=1.0):
    r = np.random.default_rng(seed)
    x = r.standard_normal((n, D)) * spread
    x[:, 3] *= 9.0                                          # an outlier channel, as real keys have
    return O.round_to_bf16(x)


@pytest.mark.parametrize("D", [64, 128])
def test_rotation_is_the_orthonormal_hadamard_matrix(D):
    H = P.hadamard(D)
    assert np.allclose(H @ H.T, np.eye(D), atol=1e-14)
    assert np.allclose(np.abs(H), 1 / math.sqrt(D))
    x = rng_rows(1, 17, D)
    y = P.rotate_f32(x).astype(np.float64)
    assert np.abs(y - x @ H).max() <= 2e-6 * np.abs(x).max() * math.sqrt(D)      # fp32 butterflies vs the definition
    # a unit vector picks out one row of H: pins the butterfly indexing element by element
    for j in (0, 1, 5, D - 1):
        e = np.zeros((1, D)); e[0, j] = 1.0
        assert np.array_equal(P.rotate_f32(e)[0].astype(np.float64), np.float32(1 / math.sqrt(D)).astype(np.float64) * np.sign(H[j]))


@pytest.mark.parametrize("D", [64, 128])
def test_rotation_keeps_every_inner_product(D):
    k = rng_rows(2, 50, D); q = rng_rows(3, 4, D)
    exact = q @ k.T
    rot = P.rotate_f32(q).astype(np.float64) @ P.rotate_f32(k).astype(np.float64).T
    assert np.abs(rot - exact).max() <= 1e-5 * np.abs(exact).max()


def test_bf16_round_up_values():
    x = np.array([1.0, 1.0 + 2.0 ** -10, 0.3, 3.0e-5, 127.0], dtype=np.float32)
    up = P.bf16_round_up(x)
    assert up[0] == 1.0 and up[1] == 1.0078125 and up[4] == 127.0
    assert np.all(up >= x)
    assert np.all((up.view(np.uint32) & 0xFFFF) == 0)                            # BF16 values
    below = ((up.view(np.uint32) >> 16) - 1).astype(np.uint32) << 16             # the BF16 just below
    assert np.all((below.view(np.float32) < x) | (up == x))


def test_split_planes_hand_worked_row():
    # max = 127 -> e = 1; t = y.  rint(-63.5) = -64 (ties to even), remainder +0.5 -> 128 -> kept at 127;
    # 0.25 -> a = 0, b = 64;  100.75 -> a = 101, b = -64
    y = np.array([[127.0, -63.5, 0.25, 0.0, 100.75, -0.001953125]], dtype=np.float32)
    a, b, e = P.split_planes(y)
    assert e[0] == 1.0
    assert a[0].tolist() == [127, -64, 0, 0, 101, 0]
    assert b[0].tolist() == [0, 127, 64, 0, -64, 0]            # -0.001953125 * 256 = -0.5 -> rint -> -0 (ties to even)
    # a scale that is not a power of two: max = 100 -> 100/127 = 0.78740156 -> BF16 up = 0.7890625
    a, b, e = P.split_planes(np.array([[100.0, 50.0]], dtype=np.float32))
    assert e[0] == 0.7890625
    assert a[0].tolist() == [127, 63] and b[0].tolist() == [-68, 94]   # 100/e = 126.7327 (-0.2673 * 256 = -68.4), 50/e = 63.3663 (0.3663 * 256 = 93.8)
    # the other end of plane B: t = 3.5 -> a = 4 (ties to even), remainder -0.5 -> -128, which an int8 holds
    a, b, e = P.split_planes(np.array([[127.0, 3.5, -2.5]], dtype=np.float32))
    assert e[0] == 1.0 and a[0].tolist() == [127, 4, -2] and b[0].tolist() == [0, -128, -128]
    # an all-zero row
    a, b, e = P.split_planes(np.zeros((1, 8), dtype=np.float32))
    assert e[0] == 1.0 and not a.any() and not b.any()


@pytest.mark.parametrize("D", [64, 128])
def test_codes_never_saturate_and_reconstruct_within_half_a_step(D):
    x = rng_rows(4, 400, D, spread=3.0)
    y = P.rotate_f32(x)
    a, b, e = P.split_planes(y)
    t = y.astype(np.float64) / e[:, None].astype(np.float64)
    assert np.abs(np.rint(t)).max() <= 127                                      # the clip on plane A never acts
    assert np.abs(a.astype(int)).max() <= 127 and b.min() >= -128 and b.max() <= 127
    assert np.all(e.astype(np.float64) >= np.abs(y).max(axis=1) / 127.0 * (1 - 2.0 ** -23))   # scale rounded up
    assert np.all(e.astype(np.float64) <= np.abs(y).max(axis=1) / 127.0 * (1 + 2.0 ** -7))    # by less than a BF16 step
    err = np.abs(P.dequantize(a, b, e) - y.astype(np.float64))
    # half a plane-B step (e/512), one whole step where +128 was kept at 127, plus the fp32 division's rounding
    assert np.all(err <= e[:, None].astype(np.float64) * (1.0 / 256 + 1e-5))
    assert np.mean(err <= e[:, None].astype(np.float64) * (1.0 / 512 + 1e-5)) > 0.99
    # plane A alone is within half a coarse step
    assert np.all(np.abs(P.dequantize(a, 0 * b, e) - y.astype(np.float64)) <= e[:, None] * (0.5 + 1e-5))


def test_scores_are_the_product_of_the_dequantized_codes():
    D = 128
    ka, kb, ke = P.quantize_rows(rng_rows(5, 60, D))
    qa, qb, qe = P.quantize_rows(rng_rows(6, 1, D))
    eta = float(qe[0]) * 0.1275
    kd = P.dequantize(ka, kb, ke); qd = P.dequantize(qa, qb, qe)[0]
    assert np.allclose(P.refined_scores(ka, kb, ke, qa[0], qb[0], eta), 0.1275 * kd @ qd, rtol=1e-12, atol=1e-12)
    # coarse = plane A of the key against BOTH planes of the query
    ka_only = P.dequantize(ka, 0 * kb, ke)
    assert np.allclose(P.coarse_scores(ka, ke, qa[0], qb[0], eta), 0.1275 * ka_only @ qd, rtol=1e-12, atol=1e-12)
    c = P.plane_products(ka, kb, qa[0], qb[0])
    assert all(v.dtype == np.int64 for v in c)
    j = 7
    assert c[1][j] == sum(int(ka[j, d]) * int(qb[0, d]) for d in range(D))      # c^ab: key plane A, query plane B
    assert c[2][j] == sum(int(kb[j, d]) * int(qa[0, d]) for d in range(D))      # c^ba: key plane B, query plane A


@pytest.mark.parametrize("D", [64, 128])
def test_two_plane_scores_sit_within_the_quantisation_bound_of_the_exact_scores(D):
    k = rng_rows(7, 300, D); q = rng_rows(8, 3, D)
    ka, kb, ke = P.quantize_rows(k); qa, qb, qe = P.quantize_rows(q)
    c = O.LOG2E / math.sqrt(D)
    for i in range(3):
        exact = O.scores(q[i], k)
        two = P.refined_scores(ka, kb, ke, qa[i], qb[i], float(qe[i]) * c)
        one = P.coarse_scores(ka, ke, qa[i], qb[i], float(qe[i]) * c)
        kn = np.linalg.norm(k, axis=1); qn = np.linalg.norm(q[i])
        # Cauchy-Schwarz with per-channel code errors e/256 (both planes) and e/2 (plane A only)
        b2 = c * (ke * math.sqrt(D) / 256 * qn + float(qe[i]) * math.sqrt(D) / 256 * kn) * 1.01 + 1e-4
        b1 = c * (ke * math.sqrt(D) / 2 * qn) * 1.01 + b2
        assert np.all(np.abs(two - exact) <= b2)
        assert np.all(np.abs(one - exact) <= b1)
        assert np.abs(two - exact).max() < 0.02 and np.abs(one - exact).max() > np.abs(two - exact).max()


def brute_force_algorithm_1(ka, kb, ke, V, qa, qb, eta, Z, T, tau):
    """Algorithm 1, key by key, in plain Python."""
    n, D = ka.shape
    R = len(eta)
    A = [[0.0] * D for _ in range(R)]; L = [0.0] * R
    n_live = n_ref = 0
    for j in range(n):
        co = []
        for i in range(R):
            caa = sum(int(ka[j, d]) * int(qa[i][d]) for d in range(D))
            cab = sum(int(ka[j, d]) * int(qb[i][d]) for d in range(D))
            co.append(float(eta[i]) * float(ke[j]) * (caa + cab / 256.0) - Z[i])
        live = any(x >= -T for x in co)
        refine = live and tau >= 0 and any(x >= -tau for x in co)
        n_live += live; n_ref += refine
        for i in range(R):
            s = co[i]
            if refine:
                cba = sum(int(kb[j, d]) * int(qa[i][d]) for d in range(D))
                cbb = sum(int(kb[j, d]) * int(qb[i][d]) for d in range(D))
                s += float(eta[i]) * float(ke[j]) * (cba + cbb / 256.0) / 256.0
            p = 2.0 ** s
            L[i] += p
            if live and s >= -T:
                for d in range(D):
                    A[i][d] += p * V[j, d]
    return np.array(A), np.array(L), n_live, n_ref


@pytest.mark.parametrize("T,tau", [(math.inf, math.inf), (math.inf, 3.0), (6.0, 2.0), (4.0, -1.0), (5.0, math.inf)])
def test_group_fold_matches_a_key_by_key_restatement_of_algorithm_1(T, tau):
    D, n, R = 64, 90, 3
    k = rng_rows(9, n, D); q = rng_rows(10, R, D); V = rng_rows(11, n, D)
    ka, kb, ke = P.quantize_rows(k); qa, qb, qe = P.quantize_rows(q)
    eta = qe.astype(np.float64) * (O.LOG2E / math.sqrt(D))
    Z = np.array([P.coarse_scores(ka, ke, qa[i], qb[i], eta[i]).max() for i in range(R)]) + np.array([0.0, -0.5, 0.25])
    A, L, info = P.fold_group_planes(ka, kb, ke, V, qa, qb, eta, Z, T, tau)
    A2, L2, n_live, n_ref = brute_force_algorithm_1(ka, kb, ke, V, qa, qb, eta, Z, T, tau)
    assert np.allclose(A, A2, rtol=1e-12, atol=1e-300) and np.allclose(L, L2, rtol=1e-12)
    assert info["live"].sum() == n_live and info["refine"].sum() == n_ref
    if not math.isinf(T):
        assert 0 < n_live < n                                 # the case exercises the gate
    if 0 <= tau < 10:
        assert 0 < n_ref < n_live


def test_special_cases_reduce_to_the_plain_declared_reference_functions():
    D, n, R = 128, 500, 4
    k = rng_rows(12, n, D); q = rng_rows(13, R, D); V = rng_rows(14, n, D)
    ka, kb, ke = P.quantize_rows(k); qa, qb, qe = P.quantize_rows(q)
    eta = qe.astype(np.float64) * (O.LOG2E / math.sqrt(D))
    Z = np.zeros(R)
    # dense, every key refined: plain softmax attention on the two-plane scores
    A, L, info = P.fold_group_planes(ka, kb, ke, V, qa, qb, eta, Z, math.inf, math.inf)
    for i in range(R):
        s = P.refined_scores(ka, kb, ke, qa[i], qb[i], eta[i])
        o, lse = O.dense_row(s, V)
        assert np.allclose(A[i] / L[i], o, rtol=1e-12) and abs(math.log2(L[i]) - lse) < 1e-12
    assert info["bytes_per_key"] == 514.0                      # 130 + 128 + 256: both planes, the scale, a BF16 value row
    # never refined, finite depth, ONE row: the plain depth-T fold on the coarse scores
    for i in range(R):
        s = P.coarse_scores(ka, ke, qa[i], qb[i], eta[i])
        Zi = O.dense_row(s, V)[1]
        A1, L1, info1 = P.fold_group_planes(ka, kb, ke, V, qa[i:i + 1], qb[i:i + 1], eta[i:i + 1], [Zi], 8.0, -1.0)
        o, lse, A0, L0 = O.fold_row(s, V, Zi, 8.0)
        assert np.allclose(A1[0], A0, rtol=1e-12) and np.isclose(L1[0], L0, rtol=1e-12)
        assert info1["bytes_per_key"] == 130.0 + 256.0 * info1["live"].mean()
    # without refinement L does not depend on the depth
    La = P.fold_group_planes(ka, kb, ke, V, qa, qb, eta, Z, 3.0, -1.0)[1]
    Lb = P.fold_group_planes(ka, kb, ke, V, qa, qb, eta, Z, math.inf, -1.0)[1]
    assert np.array_equal(La, Lb)


def test_verdicts_are_ored_over_the_group_but_weights_are_cut_per_row():
    D = 64
    k = rng_rows(15, 200, D); V = np.ones((200, D)); q = rng_rows(16, 2, D)
    ka, kb, ke = P.quantize_rows(k); qa, qb, qe = P.quantize_rows(q)
    eta = qe.astype(np.float64) * (O.LOG2E / math.sqrt(D))
    Z = np.array([P.coarse_scores(ka, ke, qa[i], qb[i], eta[i]).max() for i in range(2)])
    T = 3.0
    A, L, info = P.fold_group_planes(ka, kb, ke, V, qa, qb, eta, Z, T, -1.0)
    own = [(info["coarse"][i] >= -T) for i in range(2)]
    assert np.array_equal(info["live"], own[0] | own[1])
    assert (own[0] & ~own[1]).any()                            # keys fetched for row 0 alone ...
    for i in range(2):                                         # ... add nothing to row 1's A (V = 1: A counts kept mass)
        assert np.isclose(A[i][0], np.exp2(info["coarse"][i][own[i]]).sum(), rtol=1e-12)


def test_auto_refine_gate_follows_the_request_length_only():
    assert P.auto_refine_tau(1024) == 8.0 and P.auto_refine_tau(32768) == 13.0 and P.auto_refine_tau(16) == 4.0
    assert P.auto_refine_tau(2048) - P.auto_refine_tau(1024) == 1.0


def test_estimate_on_planes_is_the_plain_estimate_of_the_two_plane_scores():
    D, n = 128, 1000
    k = rng_rows(17, n, D); q = rng_rows(18, 1, D)
    ka, kb, ke = P.quantize_rows(k); qa, qb, qe = P.quantize_rows(q)
    eta = float(qe[0]) * O.LOG2E / math.sqrt(D)
    s = P.refined_scores(ka, kb, ke, qa[0], qb[0], eta)
    assert P.estimate_z_planes(ka, kb, ke, qa[0], qb[0], eta) == O.estimate_z(lambda i: s[i], n)
    short = P.estimate_z_planes(ka[:100], kb[:100], ke[:100], qa[0], qb[0], eta)
    assert abs(short - O.dense_row(s[:100], np.zeros((100, 1)))[1]) < 1e-12


def test_rows_that_do_not_see_a_key_give_it_no_weight_and_no_vote():
    # drafts / verification trees: a masked key is as good as absent for that row, and cannot make the key live
    D, n = 64, 120
    k = rng_rows(19, n, D); V = rng_rows(20, n, D); q = rng_rows(21, 2, D)
    ka, kb, ke = P.quantize_rows(k); qa, qb, qe = P.quantize_rows(q)
    eta = qe.astype(np.float64) * (O.LOG2E / math.sqrt(D))
    Z = np.array([P.coarse_scores(ka, ke, qa[i], qb[i], eta[i]).max() for i in range(2)])
    vis = np.ones((2, n), dtype=bool); vis[1, -7:] = False; vis[1, 3] = False
    A, L, info = P.fold_group_planes(ka, kb, ke, V, qa, qb, eta, Z, math.inf, -1.0, visible=vis)
    sub = vis[1]
    A1, L1, _ = P.fold_group_planes(ka[sub], kb[sub], ke[sub], V[sub], qa[1:], qb[1:], eta[1:], Z[1:], math.inf, -1.0)
    assert np.allclose(A[1], A1[0], rtol=1e-12) and np.isclose(L[1], L1[0], rtol=1e-12)
    A0, L0, _ = P.fold_group_planes(ka, kb, ke, V, qa[:1], qb[:1], eta[:1], Z[:1], math.inf, -1.0)
    assert np.allclose(A[0], A0[0], rtol=1e-12) and np.isclose(L[0], L0[0], rtol=1e-12)
    # a key nobody sees is not live even in dense decode (its value row is never asked for)
    vis[0, 5] = vis[1, 5] = False
    info = P.fold_group_planes(ka, kb, ke, V, qa, qb, eta, Z, math.inf, -1.0, visible=vis)[2]
    assert not info["live"][5] and info["live"].sum() == n - 1
    # at finite depth a masked row has no vote: the key is live only through the rows that see it
    T = 3.0
    info = P.fold_group_planes(ka, kb, ke, V, qa, qb, eta, Z, T, -1.0, visible=vis)[2]
    own0 = np.where(vis[0], info["coarse"][0] >= -T, False); own1 = np.where(vis[1], info["coarse"][1] >= -T, False)
    assert np.array_equal(info["live"], own0 | own1)


def test_block_tail_on_planes_reduces_to_the_plain_block_tail():
    # one row, no refinement: the two-plane fold with a mean table is the plain depth-T fold with that table on the
    # coarse scores; with constant values the tail restores exactly what the cut took away
    D, n = 64, 300
    k = rng_rows(22, n, D); V = rng_rows(23, n, D); q = rng_rows(24, 1, D)
    ka, kb, ke = P.quantize_rows(k); qa, qb, qe = P.quantize_rows(q)
    eta = qe.astype(np.float64) * (O.LOG2E / math.sqrt(D))
    s = P.coarse_scores(ka, ke, qa[0], qb[0], eta[0])
    Z = float(s.max()) - 1.0
    vm = O.block_means(V)
    A, L, info = P.fold_group_planes(ka, kb, ke, V, qa, qb, eta, [Z], 4.0, -1.0, v_mean=vm)
    o, lse, A0, L0 = O.fold_row(s, V, Z, 4.0, v_mean=vm)
    assert 0 < info["live"].sum() < n
    assert np.allclose(A[0], A0, rtol=1e-12) and np.isclose(L[0], L0, rtol=1e-12)
    Vc = np.full((n, D), 1.5)
    A, L, _ = P.fold_group_planes(ka, kb, ke, Vc, qa, qb, eta, [Z], 4.0, -1.0, v_mean=O.block_means(Vc))
    assert np.allclose(A[0] / L[0], 1.5, rtol=1e-12)


def test_block_tail_on_planes_counts_what_each_row_cuts():
    # several rows: a key another row keeps live (so it is fetched) is still cut for a row whose own final score is
    # below the depth, and that row's weight goes to the block's mean.  Brute force, key by key.
    D, n, R, T = 64, 200, 3, 5.0
    k = rng_rows(32, n, D); V = rng_rows(33, n, D); q = rng_rows(34, R, D, spread=2.0)
    ka, kb, ke = P.quantize_rows(k); qa, qb, qe = P.quantize_rows(q)
    eta = qe.astype(np.float64) * (O.LOG2E / math.sqrt(D))
    Z = np.array([P.coarse_scores(ka, ke, qa[i], qb[i], eta[i]).max() for i in range(R)]) - 1.0
    vm = O.block_means(V)
    A, L, info = P.fold_group_planes(ka, kb, ke, V, qa, qb, eta, Z, T, 2.0, v_mean=vm)
    A0, L0, _ = P.fold_group_planes(ka, kb, ke, V, qa, qb, eta, Z, T, 2.0)
    assert np.array_equal(L, L0)
    shared = 0
    for i in range(R):
        extra = np.zeros(D)
        for j in range(n):
            s = info["coarse"][i, j] + (P.refine_terms(kb[j:j + 1], ke[j:j + 1], qa[i], qb[i], eta[i])[0] if info["refine"][j] else 0.0)
            kept = info["live"][j] and s >= -T
            if not kept:
                extra += 2.0 ** s * vm[j // 64]
            shared += int(info["live"][j] and not kept)
        assert np.allclose(A[i] - A0[i], extra, rtol=1e-9, atol=1e-12)
    assert shared > 0                                             # the case the test is about does occur


def test_e4m3_grid_and_rounding_hand_values():
    v = P.e4m3_values()
    # 1-4-3 bits, bias 7: 0x38 = 1.0, 0x7e = 448 (largest), 0x01 = 2^-9 (smallest subnormal), 0x08 = 2^-6 (smallest normal)
    assert v[0x38] == 1.0 and v[0x7e] == 448.0 and v[0x01] == 2.0 ** -9 and v[0x08] == 2.0 ** -6 and v[0xb8] == -1.0
    assert np.isnan(v[0x7f]) and np.isnan(v[0xff]) and np.all(np.diff(v[:0x7f]) > 0)
    x = np.array([1.0, 1.0625, 1.1875, 17.0, 448.0, 1000.0, -464.0, 2.0 ** -10, 3 * 2.0 ** -10, 0.3])
    want = [0x38, 0x38, 0x3a, 0x58, 0x7e, 0x7e, 0xfe, 0x00, 0x02, 0x2a]       # ties to the even code; beyond 448 saturates
    assert P.round_e4m3(x).tolist() == want
    # nearest: no other code is closer, for a dense sample of the range
    xs = np.linspace(-460, 460, 20011)
    c = P.round_e4m3(xs)
    d = np.abs(np.minimum(np.abs(xs), 448.0)[:, None] - v[None, :0x7f])
    assert np.all(np.abs(np.abs(v[c]) - np.minimum(np.abs(xs), 448.0)) <= d.min(axis=1) + 1e-15)


def test_value_planes_reconstruct_within_their_steps():
    V = rng_rows(25, 300, 128, spread=2.0)
    k = int(math.ceil(math.log2(np.abs(V).max() / 448.0)))
    p1, p2 = P.quantize_values(V, k)
    one = P.widen_values(p1, p2, k, np.zeros(300, bool)); two = P.widen_values(p1, p2, k, np.ones(300, bool))
    nz = np.abs(V) >= 2.0 ** (k - 6)                            # normal range of plane 1: 3 mantissa bits, then 3 more + BF16
    assert np.all(np.abs(one - V)[nz] <= np.abs(V)[nz] * 2.0 ** -4)
    assert np.all(np.abs(two - V)[nz] <= np.abs(V)[nz] * 2.0 ** -8 * 1.01 + 2.0 ** (k - 10))   # (the residual's code may be subnormal)
    assert np.mean(np.abs(two - V)[nz] <= np.abs(V)[nz] * 2.0 ** -8 * 1.01) > 0.95
    assert np.all(np.abs(one - V) <= 2.0 ** (k - 10) + np.abs(V) * 2.0 ** -4)    # subnormal plane-1 codes: absolute step 2^-9
    assert np.array_equal(O.round_to_bf16(two), two) and np.array_equal(O.round_to_bf16(one), one)   # both are BF16 values
    # v1 + v2 can need nine significant bits; it is rounded to BF16 once, ties to even: 1 + 2^-5 + 2^-8 -> 1 + 2^-5
    # (codes 0x38 = 1, 0x11 = 1.125 * 2^-5) and 1 + 2^-5 + 2^-7 + 2^-8 -> 1 + 2^-5 + 2^-6 (0x13 = 1.375 * 2^-5)
    w = P.widen_values(np.array([[0x38, 0x38]], dtype=np.uint8), np.array([[0x11, 0x13]], dtype=np.uint8), 3, np.ones(1, bool))
    assert w[0].tolist() == [8.0 * (1 + 2.0 ** -5), 8.0 * (1 + 2.0 ** -5 + 2.0 ** -6)]
    # values that are not BF16 themselves (the writer takes any float): the widened rows still are, and for BF16
    # inputs the sum of the planes never needs the rounding at all
    Vf = np.random.default_rng(31).standard_normal((200, 64)) * 2.0
    f1, f2 = P.quantize_values(Vf, k)
    twof = P.widen_values(f1, f2, k, np.ones(200, bool))
    assert np.array_equal(O.round_to_bf16(twof), twof)
    assert not np.array_equal(P.e4m3_values()[f1] + P.e4m3_values()[f2], twof * 2.0 ** -k)
    assert np.array_equal((P.e4m3_values()[p1] + P.e4m3_values()[p2]) * 2.0 ** k, two)
    mixed = P.widen_values(p1, p2, k, np.arange(300) % 2 == 0)
    assert np.array_equal(mixed[0::2], two[0::2]) and np.array_equal(mixed[1::2], one[1::2])


def test_group_fold_with_value_planes_special_cases_and_bytes():
    D, n, R = 128, 400, 4
    k_ = rng_rows(26, n, D); q = rng_rows(27, R, D); V = rng_rows(28, n, D)
    ka, kb, ke = P.quantize_rows(k_); qa, qb, qe = P.quantize_rows(q)
    eta = qe.astype(np.float64) * (O.LOG2E / math.sqrt(D))
    Z = np.array([P.coarse_scores(ka, ke, qa[i], qb[i], eta[i]).max() for i in range(R)]) - 2.0
    sl = int(math.ceil(math.log2(np.abs(V).max() / 448.0)))
    p1, p2 = P.quantize_values(V, sl)
    # every live key refined (keys and values), dense: the plain fold on the fully widened values; 514 - 256 + 256 bytes
    A, L, info = P.fold_group_planes(ka, kb, ke, None, qa, qb, eta, Z, math.inf, math.inf, value_planes=(p1, p2, sl), tau_v=math.inf)
    A0, L0, _ = P.fold_group_planes(ka, kb, ke, P.widen_values(p1, p2, sl, np.ones(n, bool)), qa, qb, eta, Z, math.inf, math.inf)
    assert np.array_equal(A, A0) and np.array_equal(L, L0) and info["bytes_per_key"] == 130 + 128 + 128 + 128
    # no second plane at all: plane-1 values; the 256 value bytes become 128 + 128 r_V (Section 4)
    A, L, info = P.fold_group_planes(ka, kb, ke, None, qa, qb, eta, Z, 6.0, -1.0, value_planes=(p1, p2, sl), tau_v=-1.0)
    A0, L0, i0 = P.fold_group_planes(ka, kb, ke, P.widen_values(p1, p2, sl, np.zeros(n, bool)), qa, qb, eta, Z, 6.0, -1.0)
    assert np.array_equal(A, A0) and info["bytes_per_key"] == 130 + 128 * i0["live"].mean()
    # the refine-V verdict is ORed over the group like the others, and only live keys can carry it
    A, L, info = P.fold_group_planes(ka, kb, ke, None, qa, qb, eta, Z, 6.0, -1.0, value_planes=(p1, p2, sl), tau_v=3.0)
    assert np.array_equal(info["refine_v"], info["live"] & (info["coarse"] >= -3.0).any(axis=0))
    assert 0 < info["refine_v"].sum() < info["live"].sum()
    assert P.auto_refine_tau_v(32768) == 16.0 and P.auto_refine_tau_v(4) == 4.0


def test_running_mean_cut_model_of_the_value_planes():
    # Section 4, "Depth as a dial": with 8-bit values a cut key's weight goes to the sequence's mean value row
    D, n, R, T = 64, 300, 3, 5.0
    k = rng_rows(40, n, D); V = rng_rows(41, n, D); q = rng_rows(42, R, D, spread=2.0)
    ka, kb, ke = P.quantize_rows(k); qa, qb, qe = P.quantize_rows(q)
    eta = qe.astype(np.float64) * (O.LOG2E / math.sqrt(D))
    Z = np.array([P.coarse_scores(ka, ke, qa[i], qb[i], eta[i]).max() for i in range(R)]) - 1.0
    sl = int(math.ceil(math.log2(np.abs(V).max() / 448.0)))
    vp = P.quantize_values(V, sl) + (sl,)
    # the mean by hand: exact rationals on small integers, then the BF16 rounding (257 / 3 = 85.67 -> 85.5)
    assert P.running_mean(np.array([[1.0, 2.0], [2.0, 255.0], [6.0, 0.0]])).tolist() == [3.0, 85.5]
    m = P.running_mean(V)
    assert np.array_equal(O.round_to_bf16(m), m) and np.allclose(m, V.mean(axis=0), rtol=2.0 ** -8, atol=1e-12)
    A, L, info = P.fold_group_planes(ka, kb, ke, None, qa, qb, eta, Z, T, 2.0, value_planes=vp, tau_v=3.0, v_run_mean=m)
    A0, L0, i0 = P.fold_group_planes(ka, kb, ke, None, qa, qb, eta, Z, T, 2.0, value_planes=vp, tau_v=3.0)
    assert np.array_equal(L, L0) and np.array_equal(info["refine_v"], i0["refine_v"])
    # brute force, key by key: what a row does not keep adds weight x mean
    for i in range(R):
        cut = 0.0
        for j in range(n):
            s = info["coarse"][i, j] + (P.refine_terms(kb[j:j + 1], ke[j:j + 1], qa[i], qb[i], eta[i])[0] if info["refine"][j] else 0.0)
            if not (info["live"][j] and s >= -T):
                cut += 2.0 ** s
        assert cut > 0 and np.allclose(A[i] - A0[i], cut * m, rtol=1e-9, atol=1e-12)
    # dense decode cuts nothing: no effect
    Ai, Li, _ = P.fold_group_planes(ka, kb, ke, None, qa, qb, eta, Z, math.inf, 2.0, value_planes=vp, tau_v=3.0, v_run_mean=m)
    Aj, Lj, _ = P.fold_group_planes(ka, kb, ke, None, qa, qb, eta, Z, math.inf, 2.0, value_planes=vp, tau_v=3.0)
    assert np.array_equal(Ai, Aj)
    # constant values that the planes hold exactly: the model restores exactly what the cut took, at any depth
    Vc = np.full((n, D), 1.5)
    vc = P.quantize_values(Vc, 0) + (0,)
    A, L, _ = P.fold_group_planes(ka, kb, ke, None, qa, qb, eta, Z, 3.0, -1.0, value_planes=vc, tau_v=-1.0, v_run_mean=P.running_mean(Vc))
    assert np.allclose(A / L[:, None], 1.5, rtol=1e-12)
    # a sequence of at most 64 keys is one block: the running mean is the block model's mean, and the two tails agree
    ks, Vs = k[:50], V[:50]
    a2, b2, e2 = P.quantize_rows(ks)
    vs = P.quantize_values(Vs, sl) + (sl,)
    Z2 = np.array([P.coarse_scores(a2, e2, qa[i], qb[i], eta[i]).max() for i in range(R)]) - 1.0
    assert np.array_equal(P.running_mean(Vs), O.block_means(Vs)[0])
    Ar, Lr, _ = P.fold_group_planes(a2, b2, e2, None, qa, qb, eta, Z2, 3.0, 1.0, value_planes=vs, tau_v=2.0, v_run_mean=P.running_mean(Vs))
    Ab, Lb, _ = P.fold_group_planes(a2, b2, e2, None, qa, qb, eta, Z2, 3.0, 1.0, value_planes=vs, tau_v=2.0, v_mean=O.block_means(Vs))
    assert np.allclose(Ar, Ab, rtol=1e-12) and np.array_equal(Lr, Lb)


# --------------------------------------------------------------------------- cascades on two-plane keys
def _cascade_inputs(B=6, G=2, D=64, n_prefix=150, suffixes=(40, 0, 7, 64, 1, 90)):
    q = rng_rows(31, B * G, D).reshape(B, G, D)
    qa, qb, qe = P.quantize_rows(q.reshape(B * G, D))
    qa = qa.reshape(B, G, D); qb = qb.reshape(B, G, D)
    eta = qe.reshape(B, G).astype(np.float64) * (O.LOG2E / math.sqrt(D))
    kp = rng_rows(32, n_prefix, D); vp = rng_rows(33, n_prefix, D)
    pre = P.quantize_rows(kp) + (vp,)
    sufs = []
    for b, n in enumerate(suffixes):
        ks = rng_rows(40 + b, n, D) if n else np.zeros((0, D)); vs = rng_rows(60 + b, n, D) if n else np.zeros((0, D))
        sufs.append((P.quantize_rows(ks) + (vs,)) if n else (np.zeros((0, D), np.int8), np.zeros((0, D), np.int8), np.zeros(0), vs))
    return qa, qb, eta, pre, sufs


def test_cascade_levels_add_up_to_the_flat_decode_when_no_gate_couples_the_rows():
    """Prop. 1(i): partials of one row under one reference add.  Without refinement (tau < 0) no verdict couples a row's
    scores to the other rows of its block, so the cascade -- any block size -- equals each request's flat decode over
    prefix ++ suffix, at any depth."""
    qa, qb, eta, pre, sufs = _cascade_inputs()
    B, G, D = qa.shape
    Z = np.array([[5.0 + 0.25 * b - 0.5 * g for g in range(G)] for b in range(B)])
    for T in (math.inf, 6.0):
        for block_rows in (16, 4, 1):
            A, L, infos = P.fold_levels_planes([(B, [pre]), (1, sufs)], qa, qb, eta, Z, T, -1.0, block_rows)
            for b in range(B):
                ka = np.concatenate([pre[0], sufs[b][0]]); kb = np.concatenate([pre[1], sufs[b][1]])
                ke = np.concatenate([pre[2], sufs[b][2]]); V = np.concatenate([pre[3], sufs[b][3]])
                A1, L1, _ = P.fold_group_planes(ka, kb, ke, V, qa[b], qb[b], eta[b], Z[b], T, -1.0)
                # (two orders of one sum: equal to rounding, measured against the row's largest entry)
                assert np.abs(A[b] - A1).max() <= 1e-12 * np.abs(A1).max() and np.allclose(L[b], L1, rtol=1e-12)
    # and with one level, one request per sequence, it IS fold_group_planes (any gate)
    A, L, infos = P.fold_levels_planes([(1, sufs)], qa, qb, eta, Z, 5.0, 3.0)
    for b in range(B):
        if sufs[b][0].shape[0]:
            A1, L1, _ = P.fold_group_planes(sufs[b][0], sufs[b][1], sufs[b][2], sufs[b][3], qa[b], qb[b], eta[b], Z[b], 5.0, 3.0)
            assert np.array_equal(A[b], A1) and np.array_equal(L[b], L1)
        else:
            assert not A[b].any() and not L[b].any()


def test_cascade_levels_carry_their_own_cut_models_and_value_planes():
    """A sequence's optional arguments reach `fold_group_planes` unchanged: one level of unstacked requests with block
    means / E4M3 value planes / a mean value row equals the direct call, and with constant values the block tail gives
    a cascade's rows back exactly what its levels cut (A / L = the constant, Section 4 "Depth as a dial")."""
    qa, qb, eta, pre, sufs = _cascade_inputs()
    B, G, D = qa.shape
    Z = np.array([[P.coarse_scores(pre[0], pre[2], qa[b, g], qb[b, g], eta[b, g]).max() for g in range(G)] for b in range(B)])
    b0 = 3                                                      # a request with a 64-key suffix
    ka, kb, ke, V = sufs[b0]
    vm = O.block_means(V)
    p1, p2 = P.quantize_values(V, -2)
    for extra in (dict(v_mean=vm), dict(value_planes=(p1, p2, -2), tau_v=3.0), dict(value_planes=(p1, p2, -2), tau_v=None, v_run_mean=P.running_mean(V))):
        seqs = [s if i != b0 else s + (extra,) for i, s in enumerate(sufs)]
        A, L, _ = P.fold_levels_planes([(1, seqs)], qa, qb, eta, Z, 4.0, 2.0)
        kw = dict(extra)
        if "tau_v" in kw and kw["tau_v"] is None:
            kw["tau_v"] = P.auto_refine_tau_v(ka.shape[0])
        A1, L1, _ = P.fold_group_planes(ka, kb, ke, V, qa[b0], qb[b0], eta[b0], Z[b0], 4.0, 2.0, **kw)
        assert np.array_equal(A[b0], A1) and np.array_equal(L[b0], L1)
    const = lambda n: np.full((n, D), 1.5)
    pre_c = pre[:3] + (const(pre[0].shape[0]), dict(v_mean=O.block_means(const(pre[0].shape[0]))))
    sufs_c = [s[:3] + (const(s[0].shape[0]), dict(v_mean=O.block_means(const(s[0].shape[0])))) if s[0].shape[0] else s for s in sufs]
    A, L, _ = P.fold_levels_planes([(B, [pre_c]), (1, sufs_c)], qa, qb, eta, Z, 3.0, -1.0)
    assert np.allclose(A / L[..., None], 1.5, rtol=1e-12)


def test_cascade_blocks_keep_their_verdicts_to_themselves_and_levels_take_their_own_gate():
    qa, qb, eta, pre, sufs = _cascade_inputs(B=5, G=4, suffixes=(40, 0, 7, 64, 90))   # 20 stacked rows on the prefix: blocks of 16 and 4
    B, G, D = qa.shape
    Z = np.zeros((B, G))
    for b in range(B):
        for g in range(G):
            Z[b, g] = P.coarse_scores(pre[0], pre[2], qa[b, g], qb[b, g], eta[b, g]).max() - 1.0
    A, L, infos = P.fold_levels_planes([(B, [pre])], qa, qb, eta, Z, 6.0, 2.0)
    assert [len(blk) for (_, _, blk, _) in infos] == [16, 4]
    rows = [(b, g) for b in range(B) for g in range(G)]
    assert infos[0][2] == rows[:16] and infos[1][2] == rows[16:]
    # a block's refine verdicts are the OR over ITS rows only: recompute them from the coarse scores it reports
    differ = False
    for (_, _, blk, info) in infos:
        own = (info["coarse"] >= -2.0).any(axis=0) & (info["coarse"] >= -6.0).any(axis=0)
        assert np.array_equal(info["refine"], own)
    differ = not np.array_equal(infos[0][3]["refine"], infos[1][3]["refine"])
    assert differ                                               # the case tells blocks apart
    # the automatic gate is the level's own: a 150-key prefix and a 90-key suffix both take max(log2 n - 2, 4) = 4 ... 5.2
    A2, L2, infos2 = P.fold_levels_planes([(B, [pre]), (1, sufs)], qa, qb, eta, Z, math.inf, None)
    for (li, j, blk, info) in infos2:
        n = pre[0].shape[0] if li == 0 else sufs[j][0].shape[0]
        tau = P.auto_refine_tau(n)
        assert np.array_equal(info["refine"], (info["coarse"] >= -tau).any(axis=0) & info["live"])
