"""Two-plane INT8 keys on the GPU against the oracle: the cache writer and the query split bit for bit
(integer codes decided by FP32 arithmetic both sides perform identically), the decode within the build's
tolerances of Algorithm 1 evaluated in float64 at the GPU's own references."""
import math

import numpy as np
import pytest
import torch

import paper_2609_33410_b200 as F
from oracle import fold_oracle as O
from oracle import fold_planes_oracle as P
from paper_2609_33410_b200.workloads import make_decode_workload, bf16_bits
from helpers import cache_of, oracle_block_means, same_bits, DENSE_MAX_ABS, DENSE_MEAN_REL, FINITE_T_FACTOR, LSE_TOL, ROW_FACTOR, Z_TOL

pytestmark = pytest.mark.gpu
DEV = "cuda"
BAND = 2.0 ** -10          # binades around a gate within which fp32 and fp64 scores may decide differently


def scale_log2_f32(w):
    return np.float32(np.float64(np.float32(w.scale)) * 1.4426950408889634)


def plane_cache(w):
    cache = cache_of(w)
    F.fold_quantize_keys(cache)
    torch.cuda.synchronize()
    return cache


def cache_after(w, cache):
    """The same planes over the workload's (modified) BF16 tensors."""
    return F.KVCache(w.k, w.v, w.seqlens, w.max_seqlen, w.page_table, None, cache.k_plane_a, cache.k_plane_b, cache.k_scale)


def logical_planes(w, cache, seq, kvh):
    """(a, b, e) of the logical keys of one (sequence, kv head), read back from the device planes."""
    n = int(w.seqlens[seq])
    j = torch.arange(n, device=cache.k.device)
    if w.paged:
        ps = cache.k.shape[1]
        pg = w.page_table[seq].long()[j // ps]
        a = cache.k_plane_a[pg, j % ps, kvh]; b = cache.k_plane_b[pg, j % ps, kvh]; e = cache.k_scale[pg, kvh, j % ps]
    else:
        a = cache.k_plane_a[seq, :n, kvh]; b = cache.k_plane_b[seq, :n, kvh]; e = cache.k_scale[seq, kvh, :n]
    return a.cpu().numpy(), b.cpu().numpy(), e.float().cpu().numpy()


def split_queries(w, bufs):
    """The split query rows the front kernel left in the workspace: (qa, qb [B, Hq, D] int8, eta [B, Hq] fp32)."""
    B, Hq, D = w.q.shape
    probe = F.make_args(w.q, cache_of(w), stack=w.stack)
    q_off = (F.fold_workspace_bytes(probe) + 255) // 256 * 256
    codes = bufs.workspace[q_off: q_off + B * Hq * 2 * D].view(torch.int8).view(B, Hq, 2, D).cpu().numpy()
    e_off = q_off + (B * Hq * 2 * D + 255) // 256 * 256
    eta = bufs.workspace[e_off: e_off + B * Hq * 4].view(torch.float32).view(B, Hq).cpu().numpy()
    return codes[:, :, 0], codes[:, :, 1], eta


def with_means(cache, vm):
    return F.KVCache(cache.k, cache.v, cache.seqlens, cache.max_seqlen, cache.page_table, vm, cache.k_plane_a,
                     cache.k_plane_b, cache.k_scale)


def value_planes_of(w, cache):
    """Quantize the values into two E4M3 planes under the smallest power-of-two scale that keeps plane 1 unsaturated."""
    vmax = float(torch.nan_to_num(w.v.float(), nan=0.0).abs().max())          # (padding rows may be poisoned with NaN)
    k = int(math.ceil(math.log2(max(vmax, 1e-30) / 448.0)))
    F.fold_quantize_values(cache, k)
    torch.cuda.synchronize()
    return cache


def logical_value_planes(w, cache, seq, kvh):
    n = int(w.seqlens[seq])
    j = torch.arange(n, device=cache.k.device)
    if w.paged:
        ps = cache.k.shape[1]
        pg = w.page_table[seq].long()[j // ps]
        return cache.v_plane_1[pg, j % ps, kvh].cpu().numpy(), cache.v_plane_2[pg, j % ps, kvh].cpu().numpy()
    return cache.v_plane_1[seq, :n, kvh].cpu().numpy(), cache.v_plane_2[seq, :n, kvh].cpu().numpy()


def run_planes(w, cache, T=math.inf, tau=0.0, z_mode=F.Z_ESTIMATE, num_splits=0, z=None, draft=None, tau_v=0.0):
    """`draft` = (masks int32 [batch], draft_len): draft / tree-verification rows."""
    bufs = F.alloc_buffers(w.q, cache, w.stack)
    if z is not None:
        bufs.z.copy_(z)
    F.decode(w.q, cache, bufs, depth_T=T, z_mode=z_mode, num_splits=num_splits, stack=w.stack, scale=w.scale, refine_tau=tau,
             refine_tau_v=tau_v, draft_mask=None if draft is None else draft[0], draft_len=0 if draft is None else draft[1])
    torch.cuda.synchronize()
    assert bufs.header().wait_timeouts == 0
    return bufs


def compare_planes(w, cache, bufs, T=math.inf, tau=0.0, units=None, check_estimate=False, check_counts=True, draft=None,
                   v_block_mean=None, tau_v=0.0, v_run_mean=None):
    """`v_block_mean`: the table the GPU was given (block tail); a key that flips at a gate then moves between its value
    and its block's mean, so the threshold slack counts twice."""
    vmt = None if v_block_mean is None else v_block_mean.float().cpu().numpy().astype(np.float64)
    vrt = None if v_run_mean is None else v_run_mean.float().cpu().numpy().astype(np.float64)     # [seqs, 1, Hkv, D]
    dmask = None if draft is None else [int(x) & 0xffffffff for x in draft[0].cpu().tolist()]
    G = w.num_q_heads // w.num_kv_heads
    R = w.stack * G
    out = bufs.out.float().cpu().numpy().astype(np.float64)
    lse = bufs.lse.cpu().numpy().astype(np.float64)
    z = bufs.z.cpu().numpy().astype(np.float64)
    status = bufs.row_status.cpu().numpy()
    qa, qb, eta = split_queries(w, bufs)
    units = units if units is not None else [(s, h) for s in range(w.num_seqs) for h in range(w.num_kv_heads)]
    num = den = ynum = slack2 = 0.0
    max_abs = vmax = dz = 0.0
    rel_rows = []
    per_row = []                                             # (b, h, |d|_2, |d|_inf, |ref|_2, slack, max|V|): judged row by row below
    n_live = n_ref = n_keys = n_refv = 0
    vfp8 = cache.v_plane_1 is not None
    for (seq, kvh) in units:
        n = int(w.seqlens[seq])
        rows = [(seq * w.stack + r // G, kvh * G + r % G) for r in range(R)]
        if n == 0:
            for (b, h) in rows:
                assert not out[b, h].any() and lse[b, h] == -np.inf and status[b, h] == F.ROW_EMPTY
            continue
        ka, kb, ke = logical_planes(w, cache, seq, kvh)
        V = O.widen_bf16(bf16_bits(w.logical_rows("v", seq, kvh)))
        Kx = O.widen_bf16(bf16_bits(w.logical_rows("k", seq, kvh)))
        # more than 16 rows per (sequence, kv head): blocks of 16 rows in row order, each Algorithm 1 over its own rows
        all_rows = rows
        for blk0 in range(0, R, 16):
            rows_blk = all_rows[blk0:blk0 + 16]
            rqa = np.stack([qa[b, h] for (b, h) in rows_blk]); rqb = np.stack([qb[b, h] for (b, h) in rows_blk])
            reta = np.array([eta[b, h] for (b, h) in rows_blk], dtype=np.float64)
            rz = np.array([z[b, h] for (b, h) in rows_blk])
            tau_eff = P.auto_refine_tau(n) if tau == 0.0 else tau
            vis = None if draft is None else np.stack([O.draft_visible(n, draft[1], dmask[b]) for (b, h) in rows_blk])
            vm = None if vmt is None else vmt[seq, :(n + 63) // 64, kvh]
            vpl, tau_v_eff = None, None
            if vfp8:
                p1, p2 = logical_value_planes(w, cache, seq, kvh)
                vpl = (p1, p2, cache.v_scale_log2)
                tau_v_eff = P.auto_refine_tau_v(n) if tau_v == 0.0 else tau_v
            A, L, info = P.fold_group_planes(ka, kb, ke, V, rqa, rqb, reta, rz, T, tau_eff, visible=vis, v_mean=vm,
                                             value_planes=vpl, tau_v=tau_v_eff,
                                             v_run_mean=None if vrt is None else vrt[seq, 0, kvh])
            n_refv += int(info["refine_v"].sum())
            n_live += int(info["live"].sum()); n_ref += int(info["refine"].sum()); n_keys += n
            vinf = np.abs(V).max(axis=1)
            near_T = np.zeros(n, bool) if math.isinf(T) else (np.abs(info["coarse"] + T) <= BAND).any(axis=0)
            near_tau = (np.abs(info["coarse"] + tau_eff) <= BAND).any(axis=0) if 0 <= tau_eff < math.inf else np.zeros(n, bool)
            for i, (b, h) in enumerate(rows_blk):
                o_ref = A[i] / L[i]
                d = out[b, h] - o_ref
                num += float(d @ d); den += float(o_ref @ o_ref)
                max_abs = max(max_abs, float(np.abs(d).max())); vmax = max(vmax, float(vinf.max()))
                rel_rows.append(np.linalg.norm(d) / max(np.linalg.norm(o_ref), 1e-300))
                assert abs(lse[b, h] - (rz[i] + math.log2(L[i]))) <= LSE_TOL, (b, h)
                if 0.5 <= L[i] <= 2.0 ** 100:
                    assert status[b, h] == 0, (b, h, status[b, h], L[i])
                corr = P.refine_terms(kb, ke, rqa[i], rqb[i], reta[i])
                s_fin = info["coarse"][i] + np.where(info["refine"], corr, 0.0)
                p = np.exp2(s_fin)
                if check_estimate:
                    s_all = P.refined_scores(ka, kb, ke, rqa[i], rqb[i], reta[i])
                    if vis is not None:
                        s_all = np.where(vis[i], s_all, -np.inf)
                    dz = max(dz, abs(O.estimate_z(lambda idx: s_all[idx], n) - z[b, h]))
                if not math.isinf(T):
                    near = near_T | (np.abs(s_fin + T) <= BAND)
                    sl = (2.0 if (vmt is not None or vrt is not None) else 1.0) * float((p[near] * vinf[near]).sum() / L[i])
                    sl += float((p[near_tau] * (np.exp2(np.abs(corr[near_tau])) - 1.0) * vinf[near_tau]).sum() / L[i])
                    slack2 += sl ** 2 * V.shape[1]
                    keep = slice(None) if vis is None else vis[i]
                    o_dense = O.dense_row(O.scores(O.widen_bf16(bf16_bits(w.q[b, h])), Kx[keep], w.scale), V[keep])[0]
                    y = O.online_softmax_bf16(O.widen_bf16(bf16_bits(w.q[b, h])), Kx[keep], V[keep], w.scale) - o_dense
                    ynum += float(y @ y)
                    per_row.append((b, h, float(np.linalg.norm(d)), float(np.abs(d).max()), float(np.linalg.norm(o_ref)), sl,
                                    float(vinf.max()), float(np.linalg.norm(y))))
    res = dict(rel_l2=math.sqrt(num / max(den, 1e-300)), max_abs=max_abs, vmax=vmax,
               mean_rel=float(np.mean(rel_rows)) if rel_rows else 0.0, dz=dz,
               live_frac=n_live / max(n_keys, 1), refine_frac=n_ref / max(n_keys, 1))
    if math.isinf(T):
        assert max_abs <= DENSE_MAX_ABS * vmax, res
        assert res["mean_rel"] <= DENSE_MEAN_REL, res
    else:
        res["yard"] = math.sqrt(ynum / max(den, 1e-300)); res["slack"] = math.sqrt(slack2 / max(den, 1e-300))
        assert res["rel_l2"] <= FINITE_T_FACTOR * res["yard"] + res["slack"] + 1e-12, res
        # and every row by itself (a pooled norm cannot see one bad row or channel among dozens)
        for (b, h, d2, dinf, r2, sl, row_vmax, yard_row) in per_row:
            assert dinf <= DENSE_MAX_ABS * row_vmax + sl + 1e-30, (b, h, dinf, row_vmax, sl)
            assert d2 <= ROW_FACTOR * yard_row + math.sqrt(w.head_dim) * sl + 1e-12, (b, h, d2, r2, yard_row, sl)
    if check_estimate:
        assert dz <= Z_TOL, res
    if check_counts and len(units) == w.num_seqs * w.num_kv_heads:
        h = bufs.header()
        assert h.v_rows_total == n_keys
        assert abs(h.v_rows_fetched - n_live) <= max(2, 2e-3 * n_keys), (h.v_rows_fetched, n_live)
        assert abs(h.k_rows_refined - n_ref) <= max(2, 2e-3 * n_keys), (h.k_rows_refined, n_ref)
        if vfp8:
            assert abs(h.v2_rows_refined - n_refv) <= max(2, 2e-3 * n_keys), (h.v2_rows_refined, n_refv)
    return res


@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("paged", [False, True])
def test_cache_writer_and_query_split_match_the_oracle_bit_for_bit(D, paged):
    w = make_decode_workload(3, 8, 2, D, [700, 64, 333], seed=41, device=DEV, paged=paged, page_size=32,
                             poison_padding=True)
    cache = plane_cache(w)
    for seq in range(3):
        for kvh in range(2):
            a, b, e = logical_planes(w, cache, seq, kvh)
            K = O.widen_bf16(bf16_bits(w.logical_rows("k", seq, kvh)))
            ra, rb, re = P.quantize_rows(K)
            assert np.array_equal(a, ra) and np.array_equal(b, rb) and np.array_equal(e, re)
    bufs = run_planes(w, cache)
    qa, qb, eta = split_queries(w, bufs)
    q = O.widen_bf16(bf16_bits(w.q.reshape(-1, D))).reshape(3, 8, D)
    ra, rb, re = P.quantize_rows(q)
    assert np.array_equal(qa, ra) and np.array_equal(qb, rb)
    assert np.array_equal(eta, (re * scale_log2_f32(w)).astype(np.float32))


@pytest.mark.parametrize("D", [64, 128])
def test_device_key_codes_against_the_hadamard_matrix_in_float64(D):
    # The bit-for-bit test above compares two copies of one FP32 procedure.  This one compares the codes the DEVICE
    # wrote with the DEFINITION, independently of any operation order: H the orthonormal Hadamard matrix (Sylvester's
    # construction, built here by Kronecker products), y = H k in float64, and the format's claim
    # |e (a + b / 256) - y| <= one plane-B step e / 256 (half a step of rounding, the +128 clamp, FP32 rotation error),
    # with plane A never saturated and e the smallest BF16 >= max|y| / 127 up to the FP32 rotation error.
    w = make_decode_workload(2, 4, 2, D, [900, 257], seed=43, device=DEV)
    cache = plane_cache(w)
    H = np.array([[1.0]])
    while H.shape[0] < D:
        H = np.kron(H, np.array([[1.0, 1.0], [1.0, -1.0]]))
    H /= math.sqrt(D)
    assert np.allclose(H @ H.T, np.eye(D), atol=1e-12)
    for seq in range(2):
        for kvh in range(2):
            a, b, e = logical_planes(w, cache, seq, kvh)
            K = O.widen_bf16(bf16_bits(w.logical_rows("k", seq, kvh)))
            Y = K @ H.T                                        # float64, matrix definition
            e64 = e.astype(np.float64)[:, None]
            rec = e64 * (a.astype(np.float64) + b.astype(np.float64) / 256.0)
            ymax = np.abs(Y).max(axis=1, keepdims=True)
            assert np.all(np.abs(rec - Y) <= e64 / 256.0 + 4e-6 * ymax)
            assert np.abs(a.astype(np.int32)).max() <= 127
            # the scale: at least max|y| / 127 (no saturation), and no more than one BF16 step above it
            assert np.all(e64 >= ymax / 127.0 * (1 - 1e-5)) and np.all(e64 <= ymax / 127.0 * (1 + 2.0 ** -7) + 1e-30)


def test_appending_tokens_quantizes_only_the_new_rows():
    w = make_decode_workload(2, 4, 2, 128, [500, 200], seed=43, device=DEV, capacity=640)
    cache = plane_cache(w)
    a0, b0, s0 = cache.k_plane_a.clone(), cache.k_plane_b.clone(), cache.k_scale.clone()
    old = w.seqlens.clone()
    w.seqlens += torch.tensor([3, 40], dtype=torch.int32, device=DEV)
    w.max_seqlen = int(w.seqlens.max())
    cache2 = F.KVCache(w.k, w.v, w.seqlens, w.max_seqlen, None, None, cache.k_plane_a, cache.k_plane_b, cache.k_scale)
    cache.k_plane_a[0, :500].fill_(77)                         # rows below first_token must not be rewritten
    F.fold_quantize_keys(cache2, first_token=old)
    torch.cuda.synchronize()
    assert bool((cache.k_plane_a[0, :500] == 77).all())
    cache.k_plane_a[0, :500] = a0[0, :500]
    full = cache_of(w); F.fold_quantize_keys(full); torch.cuda.synchronize()
    for seq, n in enumerate(w.seqlens.tolist()):
        assert torch.equal(cache.k_plane_a[seq, :n], full.k_plane_a[seq, :n])
        assert torch.equal(cache.k_plane_b[seq, :n], full.k_plane_b[seq, :n])
        assert torch.equal(cache.k_scale[seq, :, :n], full.k_scale[seq, :, :n])


@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("n", [1, 15, 16, 17, 127, 128, 129, 255, 257, 1000])
def test_edge_lengths(D, n):
    w = make_decode_workload(2, 4, 2, D, [n, max(1, n - 17)], seed=200 + n, device=DEV, poison_padding=True,
                             capacity=n + 70)
    cache = plane_cache(w)
    compare_planes(w, cache, run_planes(w, cache), check_estimate=True)
    compare_planes(w, cache, run_planes(w, cache, T=16.0), T=16.0)
    compare_planes(w, cache, run_planes(w, cache, T=4.0, tau=2.0), T=4.0, tau=2.0)


@pytest.mark.parametrize("Hq,Hkv,stack", [(1, 1, 1), (8, 8, 1), (4, 2, 1), (8, 1, 1), (8, 2, 2), (2, 2, 4), (3, 1, 2),
                                          # 9 to 16 rows per (sequence, kv head): two 8-row tiles, verdicts over all of them
                                          (16, 1, 1), (9, 1, 1), (24, 2, 1), (8, 2, 4), (3, 1, 5), (4, 2, 7), (13, 1, 1),
                                          # more than 16 stacked rows: blocks of 16 rows, each with its own verdicts
                                          (8, 2, 5), (4, 1, 20), (16, 2, 3), (3, 1, 11)])
def test_group_and_stack_shapes(Hq, Hkv, stack):
    w = make_decode_workload(2 * stack, Hq, Hkv, 128, [700, 300], seed=47, device=DEV, stack=stack)
    cache = plane_cache(w)
    compare_planes(w, cache, run_planes(w, cache))
    compare_planes(w, cache, run_planes(w, cache, T=12.0), T=12.0)
    if stack * (Hq // Hkv) > 16:                                # the wide forms with the block tail and with E4M3 values too
        vm = oracle_block_means(w)
        ct = with_means(cache, vm)
        compare_planes(w, ct, run_planes(w, ct, T=10.0), T=10.0, v_block_mean=vm)
        value_planes_of(w, cache)
        compare_planes(w, cache, run_planes(w, cache, T=12.0), T=12.0)


@pytest.mark.parametrize("page_size", [16, 32, 64, 128, 256])
@pytest.mark.parametrize("D", [64, 128])
def test_paged_layout_and_poisoned_tails(page_size, D):
    w = make_decode_workload(3, 8, 2, D, [1500, 64, 333], seed=53, device=DEV, paged=True, page_size=page_size,
                             poison_padding=True)
    cache = plane_cache(w)
    compare_planes(w, cache, run_planes(w, cache), check_estimate=True)
    compare_planes(w, cache, run_planes(w, cache, T=16.0), T=16.0)


@pytest.mark.parametrize("tau", [-1.0, 3.0, 12.0, math.inf])
def test_refine_gate_settings(tau):
    w = make_decode_workload(2, 8, 2, 128, [3000, 1111], seed=59, device=DEV)
    cache = plane_cache(w)
    r = compare_planes(w, cache, run_planes(w, cache, tau=tau), tau=tau)
    if tau < 0:
        assert r["refine_frac"] == 0.0
    if math.isinf(tau):
        assert r["refine_frac"] == 1.0
    if tau == 3.0:
        assert 0.0 < r["refine_frac"] < 0.5
    r = compare_planes(w, cache, run_planes(w, cache, T=10.0, tau=tau), T=10.0, tau=tau)
    assert r["refine_frac"] <= r["live_frac"] < 1.0


def test_long_context_several_chunks_and_two_plane_accuracy():
    # > 8192 keys: 1024-key chunks; the two-plane dense result is also within the BF16 tolerances of EXACT attention
    w = make_decode_workload(2, 8, 2, 128, [20000, 9001], seed=61, device=DEV)
    cache = plane_cache(w)
    units = [(0, 0), (1, 1)]
    b = run_planes(w, cache, tau=math.inf)
    compare_planes(w, cache, b, tau=math.inf, units=units, check_estimate=True)
    out = b.out.float().cpu().numpy().astype(np.float64)
    for (seq, kvh) in units:
        K = O.widen_bf16(bf16_bits(w.logical_rows("k", seq, kvh))); V = O.widen_bf16(bf16_bits(w.logical_rows("v", seq, kvh)))
        for g in range(4):
            h = kvh * 4 + g
            o = O.dense_row(O.scores(O.widen_bf16(bf16_bits(w.q[seq, h])), K, w.scale), V)[0]
            assert np.linalg.norm(out[seq, h] - o) <= 1e-2 * np.linalg.norm(o)
    compare_planes(w, cache, run_planes(w, cache, T=16.0), T=16.0, units=units)


def test_split_count_and_reference_modes():
    w = make_decode_workload(2, 8, 2, 128, [9000, 2500], seed=67, device=DEV)
    cache = plane_cache(w)
    base = run_planes(w, cache, T=14.0)
    for s in (1, 3, 9):
        other = run_planes(w, cache, T=14.0, num_splits=s)
        assert same_bits(base.out, other.out) and same_bits(base.lse, other.lse) and same_bits(base.z, other.z)
    given = run_planes(w, cache, T=14.0, z_mode=F.Z_GIVEN, z=base.z)
    assert same_bits(base.out, given.out) and same_bits(base.lse, given.lse)
    compare_planes(w, cache, run_planes(w, cache, z_mode=F.Z_ZERO))
    compare_planes(w, cache, run_planes(w, cache, z_mode=F.Z_GIVEN, z=base.lse + 30.0), check_counts=False)


def test_empty_sequences_and_unsupported_shapes():
    w = make_decode_workload(3, 4, 2, 128, [0, 500, 0], seed=71, device=DEV, capacity=512)
    cache = plane_cache(w)
    compare_planes(w, cache, run_planes(w, cache))
    compare_planes(w, cache, run_planes(w, cache, T=16.0), T=16.0)
    wide = make_decode_workload(5, 4, 1, 128, [300], seed=73, device=DEV, stack=5)      # 20 rows: two blocks -- not with draft rows,
    c2 = plane_cache(wide)                                                              # which share their sequence's verdicts
    bufs = F.alloc_buffers(wide.q, c2, 5)
    masks = torch.full((5,), 1, dtype=torch.int32, device=DEV)
    a = F.make_args(wide.q, c2, z=bufs.z, workspace=bufs.workspace, out=bufs.out, lse=bufs.lse, stack=5, draft_mask=masks, draft_len=5)
    assert F.lib().fold_decode(a, None) == F.FOLD_EUNSUPPORTED
    a = F.make_args(w.q, cache, z=bufs.z, workspace=bufs.workspace, out=bufs.out, lse=bufs.lse, z_mode=F.Z_EXACT_MAX)
    assert F.lib().fold_decode(a, None) == F.FOLD_EUNSUPPORTED
    torch.cuda.synchronize()


def test_decode_without_the_bf16_keys_and_graph_replay():
    w = make_decode_workload(2, 8, 2, 128, [4000, 1000], seed=79, device=DEV)
    cache = plane_cache(w)
    ref = run_planes(w, cache, T=16.0)
    nok = F.KVCache(w.k, w.v, w.seqlens, w.max_seqlen, None, None, cache.k_plane_a, cache.k_plane_b, cache.k_scale)
    bufs = F.alloc_buffers(w.q, nok)
    args = F.make_args(w.q, nok, depth_T=16.0, z=bufs.z, workspace=bufs.workspace, out=bufs.out, lse=bufs.lse,
                       row_status=bufs.row_status)
    args.kv.k = None                                            # the planes are all the decode reads of the keys
    F.fold_decode(args)
    torch.cuda.synchronize()
    assert same_bits(bufs.out, ref.out) and same_bits(bufs.lse, ref.lse)
    g = torch.cuda.CUDAGraph()
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        F.fold_decode(args, s)
        s.synchronize()
        bufs.out.zero_()
        with torch.cuda.graph(g, stream=s):
            F.fold_decode(args, s)
    g.replay()
    torch.cuda.synchronize()
    assert same_bits(bufs.out, ref.out) and same_bits(bufs.lse, ref.lse)


def test_config2_full_size_two_plane_keys_sampled_units():
    # the benchmark's workload (16 x 8 kv heads x 32768 keys, group 4) in the launch configuration bench.py --planes times
    free, _ = torch.cuda.mem_get_info()
    if free / 2 ** 30 < 14:
        pytest.skip("not enough free device memory")
    w = make_decode_workload(16, 32, 8, 128, 32768, seed=1, device=DEV)
    cache = plane_cache(w)
    units = [(0, 0), (7, 5), (15, 7)]
    for seq, kvh in units[:2]:                                  # the writer at full size, bit for bit
        a, b, e = logical_planes(w, cache, seq, kvh)
        ra, rb, re = P.quantize_rows(O.widen_bf16(bf16_bits(w.logical_rows("k", seq, kvh))))
        assert np.array_equal(a, ra) and np.array_equal(b, rb) and np.array_equal(e, re)
    b16 = run_planes(w, cache, T=16.0)
    r = compare_planes(w, cache, b16, T=16.0, units=units, check_estimate=True)
    assert 0.1 < r["refine_frac"] < 0.3 and r["live_frac"] > 0.9
    assert same_bits(run_planes(w, cache, T=16.0, num_splits=8).out, b16.out)
    compare_planes(w, cache, run_planes(w, cache), units=units)
    # the same cache with its values in two E4M3 planes (bench.py --planes --fp8v): writer bit for bit on one unit,
    # gated decode at the automatic gates on the sampled units
    cache = value_planes_of(w, cache)
    p1, p2 = logical_value_planes(w, cache, 7, 5)
    r1, r2 = P.quantize_values(O.widen_bf16(bf16_bits(w.logical_rows("v", 7, 5))), cache.v_scale_log2)
    assert np.array_equal(p1, r1) and np.array_equal(p2, r2)
    v16 = run_planes(w, cache, T=16.0)
    compare_planes(w, cache, v16, T=16.0, units=units[1:], check_estimate=True)
    assert same_bits(run_planes(w, cache, T=16.0, num_splits=8).out, v16.out)
    del w, cache
    torch.cuda.empty_cache()


def test_head_dim_64_mha_long_rows_sampled_units():
    w = make_decode_workload(4, 16, 16, 64, 32768, seed=83, device=DEV, paged=True, page_size=64)
    cache = plane_cache(w)
    units = [(0, 0), (3, 15)]
    compare_planes(w, cache, run_planes(w, cache, T=16.0), T=16.0, units=units, check_estimate=True)
    compare_planes(w, cache, run_planes(w, cache, T=8.0), T=8.0, units=units)
    compare_planes(w, cache, run_planes(w, cache), units=units)


PLANE_LENGTHS = [0, 1, 15, 16, 17, 63, 64, 65, 127, 128, 129, 191, 192, 193, 255, 256, 257, 1000, 2047, 5000, 9000]


@pytest.mark.parametrize("seed", range(5))
def test_random_shapes_match_the_oracle(seed):
    """Seeded random shapes of the two-plane path: head dimension, rows per kv head (1..33: up to three 16-row blocks), lengths around every tile /
    chunk / estimator boundary, paged or contiguous, depth, refine gates, block tail, draft masks and E4M3 value planes drawn together."""
    import random
    rnd = random.Random(7300 + seed)
    for i in range(8):
        D = rnd.choice([64, 128])
        G, stack = rnd.choice([(1, 1), (2, 1), (3, 1), (4, 1), (8, 1), (5, 1), (1, 3), (2, 4), (4, 2), (1, 8), (2, 2),
                               (16, 1), (9, 1), (4, 4), (2, 7), (3, 5), (1, 13), (12, 1), (4, 5), (2, 12), (8, 3), (1, 33)])
        Hkv = rnd.choice([1, 2, 3])
        nseq = rnd.choice([1, 2, 3])
        lens = [rnd.choice(PLANE_LENGTHS) for _ in range(nseq)]
        if max(lens) == 0:
            lens[0] = 33
        T = rnd.choice([math.inf, 16.0, 12.0, 8.0])
        tau = rnd.choice([0.0, 0.0, -1.0, 3.0, 9.0, math.inf])
        kw = dict(device=DEV, poison_padding=True)
        if rnd.random() < 0.4:
            kw.update(paged=True, page_size=rnd.choice([16, 32, 64, 128]))
        else:
            kw.update(capacity=max(lens) + rnd.choice([0, 5, 100]))
        tail = (not math.isinf(T)) and rnd.random() < 0.4
        drafts = stack > 1 and G * stack <= 16 and rnd.random() < 0.5        # (draft rows stay within one 16-row block)
        vfp8 = rnd.random() < 0.4                                # (with the tail: the format's own cut model, the mean row)
        tau_v = rnd.choice([0.0, 0.0, -1.0, 5.0, math.inf])
        case = dict(D=D, G=G, stack=stack, Hkv=Hkv, lens=lens, T=T, tau=tau, kw=kw, tail=tail, drafts=drafts, vfp8=vfp8, tau_v=tau_v)
        draft = None
        if drafts:
            from paper_2609_33410_b200.workloads import make_draft_workload
            kw.pop("capacity", None)
            w, masks, m = make_draft_workload(nseq, stack, G * Hkv, Hkv, D, [max(n, 1) for n in lens], seed=seed * 100 + i,
                                              tree=rnd.random() < 0.5, **kw)
            draft = (masks, m)
        else:
            w = make_decode_workload(nseq * stack, G * Hkv, Hkv, D, lens, seed=seed * 100 + i, stack=stack, **kw)
        cache = plane_cache(w)
        vm = oracle_block_means(w) if tail and not vfp8 else None
        if vm is not None:
            cache = with_means(cache, vm)
        if vfp8:
            value_planes_of(w, cache)
        vr = F.fold_running_means(cache) if tail and vfp8 else None
        try:
            b = run_planes(w, cache, T=T, tau=tau, draft=draft, tau_v=tau_v)
            compare_planes(w, cache, b, T=T, tau=tau, check_estimate=True, draft=draft, v_block_mean=vm, tau_v=tau_v,
                           v_run_mean=vr)
            s = run_planes(w, cache, T=T, tau=tau, num_splits=rnd.choice([1, 2, 5]), draft=draft, tau_v=tau_v)
            assert same_bits(s.out, b.out) and same_bits(s.lse, b.lse), "split count changed a bit"
        except AssertionError as e:
            raise AssertionError(f"case {case}: {e}") from e


def test_static_scratch_entry_point_takes_two_plane_keys():
    w = make_decode_workload(2, 8, 2, 128, [3000, 900], seed=89, device=DEV, paged=True, page_size=64)
    cache = plane_cache(w)
    ref = run_planes(w, cache, T=16.0)
    out = torch.zeros_like(ref.out); lse = torch.zeros_like(ref.lse); z = torch.zeros_like(ref.z)
    st = torch.zeros_like(ref.row_status)
    args = F.make_args(w.q, cache, depth_T=16.0, z=z, out=out, lse=lse, row_status=st)       # no workspace
    F.fold_decode_static(args)
    torch.cuda.synchronize()
    assert same_bits(out, ref.out) and same_bits(lse, ref.lse) and same_bits(z, ref.z) and not st.any()


@pytest.mark.parametrize("Hq,Hkv,m,tree", [(8, 2, 2, False), (4, 2, 4, True), (2, 2, 8, False), (3, 1, 2, True),
                                           (8, 2, 4, True), (2, 1, 7, False)])          # 16 and 14 rows: two row tiles
def test_draft_rows_on_two_plane_keys(Hq, Hkv, m, tree):
    from paper_2609_33410_b200.workloads import make_draft_workload
    w, masks, m = make_draft_workload(2, m, Hq, Hkv, 128, [700, 190], seed=97, device=DEV, tree=tree, poison_padding=True)
    cache = plane_cache(w)
    d = (masks, m)
    b = run_planes(w, cache, draft=d)
    compare_planes(w, cache, b, check_estimate=True, draft=d)
    compare_planes(w, cache, run_planes(w, cache, T=12.0, draft=d), T=12.0, draft=d)
    s = run_planes(w, cache, num_splits=1, draft=d)
    assert same_bits(s.out, b.out) and same_bits(s.lse, b.lse)
    # a row's masked-out draft keys change nothing: flipping their value rows leaves that row's output bit-identical
    keep = b.out.clone()
    n0 = int(w.seqlens[0])
    w.v[0, n0 - 1] = -w.v[0, n0 - 1]                            # the LAST draft key: row 0 of a chain / tree never uses it
    again = run_planes(w, cache_after(w, cache), draft=d)
    assert same_bits(again.out[0], keep[0])


@pytest.mark.parametrize("Hq,Hkv,D,paged", [(8, 2, 128, False), (8, 8, 64, True), (4, 1, 128, True), (2, 2, 64, False)])
def test_block_tail_on_two_plane_keys(Hq, Hkv, D, paged):
    kw = dict(paged=True, page_size=32) if paged else dict(capacity=3100)
    w = make_decode_workload(2, Hq, Hkv, D, [3000, 733], seed=101, device=DEV, poison_padding=True, **kw)
    vm = oracle_block_means(w)
    cache = with_means(plane_cache(w), vm)
    plain = plane_cache(w)
    for T in (6.0, 12.0, 16.0):
        b = run_planes(w, cache, T=T)
        r = compare_planes(w, cache, b, T=T, v_block_mean=vm)
        s = run_planes(w, cache, T=T, num_splits=1)
        assert same_bits(s.out, b.out) and same_bits(s.lse, b.lse)
        assert same_bits(b.lse, run_planes(w, plain, T=T).lse)          # the tail moves A only: L and lse are untouched
    assert same_bits(run_planes(w, cache).out, run_planes(w, plain).out)  # nothing is cut in dense decode
    # constant values: the tail gives back what the cut took away
    w.v.fill_(1.5)
    vm2 = oracle_block_means(w)
    t = run_planes(w, with_means(plain, vm2), T=6.0)
    ok = t.row_status.cpu().numpy() == 0
    assert np.allclose(t.out.float().cpu().numpy()[ok], 1.5, rtol=1e-2)


@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("paged", [False, True])
def test_value_plane_writer_matches_the_oracle_bit_for_bit(D, paged):
    w = make_decode_workload(3, 8, 2, D, [700, 64, 333], seed=103, device=DEV, paged=paged, page_size=32, poison_padding=True)
    w.v[..., 5] *= 300.0                                         # a wide range: saturating and subnormal codes both occur
    cache = plane_cache(w)
    for k in (0, -3):
        F.fold_quantize_values(cache, k)
        torch.cuda.synchronize()
        for seq in range(3):
            for kvh in range(2):
                p1, p2 = logical_value_planes(w, cache, seq, kvh)
                r1, r2 = P.quantize_values(O.widen_bf16(bf16_bits(w.logical_rows("v", seq, kvh))), k)
                assert np.array_equal(p1, r1) and np.array_equal(p2, r2), (k, seq, kvh)
    assert (p1 & 0x7f).max() == 0x7e and ((p1 & 0x78) == 0).any()


@pytest.mark.parametrize("Hq,Hkv,D,paged", [(8, 2, 128, False), (8, 8, 64, True), (4, 1, 128, True), (1, 1, 64, False)])
def test_decode_on_e4m3_value_planes(Hq, Hkv, D, paged):
    kw = dict(paged=True, page_size=32) if paged else dict(capacity=3100)
    w = make_decode_workload(2, Hq, Hkv, D, [3000, 733], seed=107, device=DEV, poison_padding=True, **kw)
    cache = value_planes_of(w, plane_cache(w))
    for T, tau_v in ((math.inf, 0.0), (math.inf, math.inf), (16.0, 0.0), (12.0, -1.0), (6.0, 3.0)):
        b = run_planes(w, cache, T=T, tau_v=tau_v)
        r = compare_planes(w, cache, b, T=T, tau_v=tau_v, check_estimate=True)
        s = run_planes(w, cache, T=T, tau_v=tau_v, num_splits=1)
        assert same_bits(s.out, b.out) and same_bits(s.lse, b.lse)
    # the decode reads no BF16 value: the same bits with v taken away
    nov = F.KVCache(w.k, w.v, w.seqlens, w.max_seqlen, w.page_table, None, cache.k_plane_a, cache.k_plane_b, cache.k_scale,
                    cache.v_plane_1, cache.v_plane_2, cache.v_scale_log2)
    bufs = F.alloc_buffers(w.q, nov)
    args = F.make_args(w.q, nov, depth_T=16.0, z=bufs.z, workspace=bufs.workspace, out=bufs.out, lse=bufs.lse, row_status=bufs.row_status)
    args.kv.v = None; args.kv.k = None
    F.fold_decode(args)
    torch.cuda.synchronize()
    ref = run_planes(w, cache, T=16.0)
    assert same_bits(bufs.out, ref.out) and same_bits(bufs.lse, ref.lse)
    # with every second plane read, the dense result is the BF16 result up to the planes' own step (2^-8 per value)
    full = run_planes(w, cache, tau_v=math.inf)
    plain = run_planes(w, plane_cache(w))
    d = (full.out.float() - plain.out.float()).norm() / plain.out.float().norm()
    assert float(d) < 5e-3


@pytest.mark.parametrize("Hq,Hkv,m,tree", [(4, 1, 2, False), (2, 2, 4, True), (1, 1, 8, False)])
def test_draft_rows_on_e4m3_value_planes(Hq, Hkv, m, tree):
    from paper_2609_33410_b200.workloads import make_draft_workload
    w, masks, m = make_draft_workload(2, m, Hq, Hkv, 128, [700, 190], seed=109, device=DEV, tree=tree, poison_padding=True)
    cache = value_planes_of(w, plane_cache(w))
    d = (masks, m)
    for T, tau_v in ((math.inf, 0.0), (12.0, 0.0), (12.0, 4.0)):
        b = run_planes(w, cache, T=T, draft=d, tau_v=tau_v)
        compare_planes(w, cache, b, T=T, check_estimate=True, draft=d, tau_v=tau_v)
        s = run_planes(w, cache, T=T, num_splits=1, draft=d, tau_v=tau_v)
        assert same_bits(s.out, b.out) and same_bits(s.lse, b.lse)


@pytest.mark.parametrize("vfp8", [False, True])
def test_head_major_plane_strides(vfp8):
    # planes stored [seq, head, token, D] and viewed as [seq, token, head, D]: only the strides differ, not a bit of the result
    w = make_decode_workload(2, 8, 4, 128, [900, 400], seed=113, device=DEV)
    cache = plane_cache(w)
    if vfp8:
        cache = value_planes_of(w, cache)
    hm = lambda t: None if t is None else t.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    other = F.KVCache(hm(w.k), hm(w.v), w.seqlens, w.max_seqlen, None, None, hm(cache.k_plane_a), hm(cache.k_plane_b),
                      cache.k_scale, hm(cache.v_plane_1), hm(cache.v_plane_2), cache.v_scale_log2)
    assert other.k_plane_a.stride() != cache.k_plane_a.stride()
    for T in (math.inf, 16.0, 8.0):
        a = run_planes(w, cache, T=T)
        b = run_planes(w, other, T=T)
        assert same_bits(a.out, b.out) and same_bits(a.lse, b.lse)
    # the writers into head-major planes: the same codes
    fresh = F.KVCache(hm(w.k), hm(w.v), w.seqlens, w.max_seqlen, None, None, torch.zeros_like(other.k_plane_a),
                      torch.zeros_like(other.k_plane_b), torch.zeros_like(cache.k_scale),
                      torch.zeros_like(other.k_plane_a).view(torch.uint8) if vfp8 else None,
                      torch.zeros_like(other.k_plane_a).view(torch.uint8) if vfp8 else None, cache.v_scale_log2)
    F.fold_quantize_keys(fresh)
    if vfp8:
        F.fold_quantize_values(fresh, cache.v_scale_log2)
    torch.cuda.synchronize()
    for s, n in enumerate([900, 400]):
        assert torch.equal(fresh.k_plane_a[s, :n], cache.k_plane_a[s, :n]) and torch.equal(fresh.k_plane_b[s, :n], cache.k_plane_b[s, :n])
        assert torch.equal(fresh.k_scale[s, :, :n], cache.k_scale[s, :, :n])
        if vfp8:
            assert torch.equal(fresh.v_plane_1[s, :n], cache.v_plane_1[s, :n]) and torch.equal(fresh.v_plane_2[s, :n], cache.v_plane_2[s, :n])


@pytest.mark.parametrize("Hq,Hkv,D,paged", [(8, 2, 128, False), (8, 8, 64, True), (4, 1, 128, True)])
def test_running_mean_cut_model_on_e4m3_value_planes(Hq, Hkv, D, paged):
    # Section 4, "Depth as a dial": with 8-bit values the cut keys' weight goes to the sequence's mean value row
    kw = dict(paged=True, page_size=32) if paged else dict(capacity=3100)
    w = make_decode_workload(3, Hq, Hkv, D, [3000, 733, 0], seed=127, device=DEV, poison_padding=True, **kw)
    cache = value_planes_of(w, plane_cache(w))
    vm = F.fold_running_means(cache)
    torch.cuda.synchronize()
    for seq, n in enumerate([3000, 733]):                       # the builder against the oracle, bit for bit
        for kvh in range(Hkv):
            ref = P.running_mean(O.widen_bf16(bf16_bits(w.logical_rows("v", seq, kvh))))
            assert np.array_equal(vm[seq, 0, kvh].float().cpu().numpy().astype(np.float64), ref), (seq, kvh)
    assert not vm[2].any()                                      # an empty sequence: zeros
    plain = value_planes_of(w, plane_cache(w))
    for T, tau_v in ((6.0, 0.0), (12.0, 0.0), (16.0, 3.0), (8.0, -1.0)):
        b = run_planes(w, cache, T=T, tau_v=tau_v)
        compare_planes(w, cache, b, T=T, tau_v=tau_v, v_run_mean=vm)
        s = run_planes(w, cache, T=T, tau_v=tau_v, num_splits=1)
        assert same_bits(s.out, b.out) and same_bits(s.lse, b.lse)
        p0 = run_planes(w, plain, T=T, tau_v=tau_v)
        assert same_bits(b.lse, p0.lse)                         # the model moves A only
        assert not same_bits(b.out, p0.out)
    # dense decode cuts nothing: the table is not read
    assert same_bits(run_planes(w, cache).out, run_planes(w, plain).out)


def test_running_mean_cut_model_with_draft_rows():
    from paper_2609_33410_b200.workloads import make_draft_workload
    w, masks, m = make_draft_workload(2, 2, 4, 1, 128, [700, 190], seed=131, device=DEV, poison_padding=True)
    cache = value_planes_of(w, plane_cache(w))
    vm = F.fold_running_means(cache)
    d = (masks, m)
    b = run_planes(w, cache, T=10.0, draft=d)
    compare_planes(w, cache, b, T=10.0, draft=d, v_run_mean=vm, check_estimate=True)


def test_million_key_sequence_on_planes_and_value_planes():
    # a thousand canonical chunks per row, plane offsets past 2^31 bytes across the tensor
    free, _ = torch.cuda.mem_get_info()
    if free / 2 ** 30 < 6:
        pytest.skip("not enough free device memory")
    w = make_decode_workload(1, 8, 4, 128, 1_100_003, seed=9, device=DEV)
    cache = value_planes_of(w, plane_cache(w))
    for T in (math.inf, 16.0):
        b = run_planes(w, cache, T=T)
        compare_planes(w, cache, b, T=T, units=[(0, 3)], check_estimate=True)
        assert same_bits(run_planes(w, cache, T=T, num_splits=3).out, b.out)
    del w, cache
    torch.cuda.empty_cache()


# ------------------------------------------------------------------ shared-prefix cascades on two-plane keys
def _planes_cascade(B, Hq, Hkv, D, n_prefix, suffixes, seed, T, tau, z_mode=F.Z_ESTIMATE, z=None, paged=False, side=None,
                    separate_calls=False, tail=False, vfp8=False):
    """tail: every level carries its block means (the block tail); vfp8: every level's values are two E4M3 planes, and
    with `tail` their cut model is the level sequences' mean value rows."""
    from paper_2609_33410_b200.workloads import make_cascade_workload
    kw = dict(paged=True, page_size=32) if paged else {}
    pre, suf = make_cascade_workload(B, Hq, Hkv, D, n_prefix, suffixes, seed=seed, device=DEV, poison_padding=True, **kw)
    cp, cs = plane_cache(pre), plane_cache(suf)
    if vfp8:
        value_planes_of(pre, cp); value_planes_of(suf, cs)
        if tail:
            F.fold_running_means(cp); F.fold_running_means(cs)
    elif tail:
        cp, cs = with_means(cp, oracle_block_means(pre)), with_means(cs, oracle_block_means(suf))
    bp, bs = F.alloc_buffers(pre.q, cp, stack=B), F.alloc_buffers(pre.q, cs)
    if z is not None:
        bs.z.copy_(z)
    common = dict(z=bs.z, depth_T=T, out=bs.out, lse=bs.lse, row_status=bs.row_status, refine_tau=tau, z_mode=z_mode)
    levels = [F.make_args(pre.q, cp, stack=B, workspace=bp.workspace, side=side, **common),
              F.make_args(pre.q, cs, workspace=bs.workspace, **common)]
    if separate_calls:                                         # the cascade spelled out: estimate, two scans, one add
        if z_mode == F.Z_ESTIMATE:
            F.fold_estimate_z(levels)
        given = [F.make_args(pre.q, cp, stack=B, workspace=bp.workspace, **{**common, "z_mode": F.Z_GIVEN}),
                 F.make_args(pre.q, cs, workspace=bs.workspace, **{**common, "z_mode": F.Z_GIVEN})]
        parts = [F.fold_decode_split(a) for a in given]
        F.fold_cascade_merge(parts, bs.out, bs.lse, bs.row_status)
    else:
        F.fold_decode_cascade(levels, torch.cuda.current_stream())
    torch.cuda.synchronize()
    assert bp.header().wait_timeouts == 0 and bs.header().wait_timeouts == 0
    return pre, suf, cp, cs, bp, bs


def _compare_planes_cascade(pre, suf, cp, cs, bp, bs, T, tau, check_estimate, tail=False, vfp8=False):
    """The oracle's cascade (`fold_levels_planes`: each level Algorithm 1 over its own rows in blocks of 16, the levels'
    (A, L) added, Eq. 3) at the GPU's own references and split query rows."""
    B, Hq, D = pre.q.shape
    Hkv = pre.num_kv_heads
    G = Hq // Hkv
    out = bs.out.float().cpu().numpy().astype(np.float64)
    lse = bs.lse.cpu().numpy().astype(np.float64)
    z = bs.z.cpu().numpy().astype(np.float64)
    qa, qb, eta = split_queries(suf, bs)
    qa2, qb2, eta2 = split_queries(pre, bp)                    # every level's workspace holds the same split rows
    assert np.array_equal(qa, qa2) and np.array_equal(qb, qb2) and np.array_equal(eta, eta2)
    dz = 0.0
    rels = []
    for kvh in range(Hkv):
        hs = slice(kvh * G, (kvh + 1) * G)

        def seq_of(w, cache, seq):
            n = int(w.seqlens[seq])
            if n == 0:
                return (np.zeros((0, D), np.int8), np.zeros((0, D), np.int8), np.zeros(0), np.zeros((0, D)))
            extra = {}
            if vfp8:
                p1, p2 = logical_value_planes(w, cache, seq, kvh)
                extra = dict(value_planes=(p1, p2, cache.v_scale_log2), tau_v=None)
                if tail:
                    extra["v_run_mean"] = cache.v_block_mean[seq, 0, kvh].float().cpu().numpy().astype(np.float64)
            elif tail:
                extra = dict(v_mean=cache.v_block_mean[seq, :(n + 63) // 64, kvh].float().cpu().numpy().astype(np.float64))
            return logical_planes(w, cache, seq, kvh) + (O.widen_bf16(bf16_bits(w.logical_rows("v", seq, kvh))), extra)

        levels = [(B, [seq_of(pre, cp, 0)]), (1, [seq_of(suf, cs, b) for b in range(B)])]
        A, L, infos = P.fold_levels_planes(levels, qa[:, hs], qb[:, hs], eta[:, hs].astype(np.float64), z[:, hs], T,
                                           None if tau == 0.0 else tau)
        # what a key next to a gate may cost (fp32 against fp64 decisions), and the rows' full two-plane scores
        slack = np.zeros((B, G)); vmax = np.zeros((B, G))
        s_all = [[[] for _ in range(G)] for _ in range(B)]
        for (li, j, blk, info) in infos:
            ka, kb, ke, V = levels[li][1][j][:4]
            n = ka.shape[0]
            tau_eff = P.auto_refine_tau(n) if tau == 0.0 else tau
            vinf = np.abs(V).max(axis=1)
            near_T = np.zeros(n, bool) if math.isinf(T) else (np.abs(info["coarse"] + T) <= BAND).any(axis=0)
            near_tau = (np.abs(info["coarse"] + tau_eff) <= BAND).any(axis=0) if 0 <= tau_eff < math.inf else np.zeros(n, bool)
            for i, (b, g) in enumerate(blk):
                vmax[b, g] = max(vmax[b, g], float(vinf.max()))
                corr = P.refine_terms(kb, ke, qa[b, kvh * G + g], qb[b, kvh * G + g], eta[b, kvh * G + g])
                s_fin = info["coarse"][i] + np.where(info["refine"], corr, 0.0)
                p = np.exp2(s_fin)
                near = near_T if math.isinf(T) else (near_T | (np.abs(s_fin + T) <= BAND))
                slack[b, g] += (2.0 if tail else 1.0) * float((p[near] * vinf[near]).sum())   # (value <-> mean: twice)
                slack[b, g] += float((p[near_tau] * (np.exp2(np.abs(corr[near_tau])) - 1.0) * vinf[near_tau]).sum())
                s_all[b][g].append(P.refined_scores(ka, kb, ke, qa[b, kvh * G + g], qb[b, kvh * G + g], eta[b, kvh * G + g]))
        for b in range(B):
            for g in range(G):
                h = kvh * G + g
                o_ref = A[b, g] / L[b, g]
                d = out[b, h] - o_ref
                assert np.abs(d).max() <= DENSE_MAX_ABS * vmax[b, g] + slack[b, g] / L[b, g] + 1e-30, (b, h, np.abs(d).max())
                rels.append(np.linalg.norm(d) / max(np.linalg.norm(o_ref), 1e-300))
                assert abs(lse[b, h] - (z[b, h] + math.log2(L[b, g]))) <= LSE_TOL, (b, h)
                if check_estimate:
                    s_cat = np.concatenate(s_all[b][g])
                    dz = max(dz, abs(O.estimate_z(lambda idx: s_cat[idx], len(s_cat)) - z[b, h]))
    if math.isinf(T):
        assert float(np.mean(rels)) <= DENSE_MEAN_REL, np.mean(rels)
    if check_estimate:
        assert dz <= Z_TOL, dz
    return dict(mean_rel=float(np.mean(rels)), dz=dz)


@pytest.mark.parametrize("T,tau", [(math.inf, 0.0), (16.0, 0.0), (12.0, 6.0), (math.inf, math.inf)])
@pytest.mark.parametrize("B,Hq,Hkv,paged", [(4, 8, 2, False), (3, 4, 1, True), (16, 2, 2, False), (2, 8, 1, False),
                                            (20, 8, 2, False), (7, 8, 1, True)])          # 80 and 56 stacked rows: blocks of 16
def test_shared_prefix_cascade_on_two_plane_keys(T, tau, B, Hq, Hkv, paged):
    # the prefix level stacks every request's rows (up to 16 per kv head) on the shared keys; suffixes ragged, one empty
    suffixes = ([500, 1, 0, 257] * 5)[:B]
    lv = _planes_cascade(B, Hq, Hkv, 128, 3000, suffixes, seed=131, T=T, tau=tau, paged=paged)
    _compare_planes_cascade(*lv, T=T, tau=tau, check_estimate=True)
    # the call is its parts: estimate over both levels, two scans, one order-free add -- bit for bit
    sp = _planes_cascade(B, Hq, Hkv, 128, 3000, suffixes, seed=131, T=T, tau=tau, paged=paged, separate_calls=True)
    assert same_bits(sp[5].out, lv[5].out) and same_bits(sp[5].lse, lv[5].lse) and same_bits(sp[5].z, lv[5].z)
    # a given reference, and the first level on the caller's side stream: the same bits again
    gv = _planes_cascade(B, Hq, Hkv, 128, 3000, suffixes, seed=131, T=T, tau=tau, paged=paged, z_mode=F.Z_GIVEN,
                         z=lv[5].z.clone(), side=F.CascadeSide(DEV))
    assert same_bits(gv[5].out, lv[5].out) and same_bits(gv[5].lse, lv[5].lse)


def test_cascade_on_two_plane_keys_head_dim_64_and_graph_replay():
    lv = _planes_cascade(4, 8, 2, 64, 1000, [100, 0, 64, 33], seed=137, T=16.0, tau=0.0)
    _compare_planes_cascade(*lv, T=16.0, tau=0.0, check_estimate=True)
    pre, suf, cp, cs, bp, bs = lv
    o, l = bs.out.clone(), bs.lse.clone()
    common = dict(z=bs.z, depth_T=16.0, out=bs.out, lse=bs.lse, row_status=bs.row_status)
    levels = [F.make_args(pre.q, cp, stack=4, workspace=bp.workspace, **common), F.make_args(pre.q, cs, workspace=bs.workspace, **common)]
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        F.fold_decode_cascade(levels, torch.cuda.current_stream())
    for _ in range(2):
        bs.out.zero_(); bs.lse.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert same_bits(bs.out, o) and same_bits(bs.lse, l)
    # levels of two key formats are refused
    mixed = [F.make_args(pre.q, cache_of(pre), stack=4, workspace=bp.workspace, **common), levels[1]]
    with pytest.raises(F.FoldError):
        F.fold_decode_cascade(mixed)
    torch.cuda.synchronize()


@pytest.mark.parametrize("tail,vfp8", [(True, False), (False, True), (True, True)])
@pytest.mark.parametrize("B,Hq,Hkv,paged", [(4, 8, 2, False), (6, 4, 1, True)])
def test_cascade_on_two_plane_keys_with_the_block_tail_and_e4m3_values(tail, vfp8, B, Hq, Hkv, paged):
    # every level brings its own cut model (block means, or with 8-bit values the sequence's mean row) and value planes
    suffixes = ([500, 1, 0, 257] * 2)[:B]
    for T in (8.0, 14.0):
        lv = _planes_cascade(B, Hq, Hkv, 128, 2000, suffixes, seed=151, T=T, tau=0.0, paged=paged, tail=tail, vfp8=vfp8)
        _compare_planes_cascade(*lv, T=T, tau=0.0, check_estimate=True, tail=tail, vfp8=vfp8)
        sp = _planes_cascade(B, Hq, Hkv, 128, 2000, suffixes, seed=151, T=T, tau=0.0, paged=paged, tail=tail, vfp8=vfp8,
                             separate_calls=True)
        assert same_bits(sp[5].out, lv[5].out) and same_bits(sp[5].lse, lv[5].lse)


@pytest.mark.parametrize("vfp8", [False, True])
@pytest.mark.parametrize("paged", [False, True])
def test_host_buffer_entry_point_takes_the_two_plane_format(vfp8, paged):
    # the planes, scales (and value planes) are copied from pinned host memory like the BF16 tensors: same bits as the
    # device path on the same codes
    kw = dict(paged=True, page_size=64) if paged else dict(capacity=2600)
    w = make_decode_workload(2, 8, 2, 128, [2500, 700], seed=163, device=DEV, **kw)
    cache = plane_cache(w)
    if vfp8:
        value_planes_of(w, cache)
    ref = run_planes(w, cache, T=16.0)
    pin = lambda t: None if t is None else t.cpu().pin_memory()
    hcache = F.KVCache(pin(w.k), pin(w.v), pin(w.seqlens), w.max_seqlen, pin(w.page_table), None, pin(cache.k_plane_a),
                       pin(cache.k_plane_b), pin(cache.k_scale), pin(cache.v_plane_1), pin(cache.v_plane_2), cache.v_scale_log2)
    hq = w.q.cpu().pin_memory()
    hout = torch.empty(2, 8, 128, dtype=torch.bfloat16).pin_memory()
    hlse = torch.empty(2, 8, dtype=torch.float32).pin_memory()
    hz = torch.empty(2, 8, dtype=torch.float32).pin_memory()
    hst = torch.empty(2, 8, dtype=torch.int32).pin_memory()
    args = F.make_args(hq, hcache, scale=w.scale, depth_T=16.0, z=hz, out=hout, lse=hlse, row_status=hst)
    staging = torch.empty(F.fold_host_staging_bytes(args), dtype=torch.uint8, device=DEV)
    F.fold_decode_host(args, staging)
    torch.cuda.synchronize()
    assert same_bits(hout, ref.out.cpu()) and same_bits(hlse, ref.lse.cpu()) and same_bits(hz, ref.z.cpu())
    assert not hst.any()
