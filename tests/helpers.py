"""Shared pieces of the GPU parity tests: run the CUDA path through the C ABI binding, run
the float64 oracle on the same seeded inputs, and compare with the stated tolerances."""
from __future__ import annotations

import math

import numpy as np
import torch

import paper_2609_33410_b200 as F
from oracle import fold_oracle as O
from paper_2609_33410_b200.workloads import DecodeWorkload, bf16_bits

# Tolerances of the build target, written out:
#   dense (T = inf): max abs error <= 1e-2 * max|V| and mean row-relative l2 error <= 5e-3
#                    against the float64 result;
#   finite T:        global relative l2 error against the float64 declared-reference result
#                    at the same Z and T  <=  1.5 x the error of a plain BF16 online-softmax
#                    kernel (emulated) against float64 softmax attention, plus the mass of keys
#                    within 2^-10 binades of the threshold (fp32 vs fp64 scores may flip them).
#   every row by itself, finite T:  |out - oracle|_inf <= 1e-2 * max|V| + that row's threshold slack, and
#                    |out - oracle|_2 <= 3 x (that row's own yardstick error, or 5e-3 |oracle|_2 where no yardstick is
#                    computed) + sqrt(D) x the row's slack: one wrong row or channel among many cannot hide in a pooled norm.
DENSE_MAX_ABS = 1e-2
DENSE_MEAN_REL = 5e-3
FINITE_T_FACTOR = 1.5
ROW_FACTOR = 3.0
Z_TOL = 1e-3
LSE_TOL = 2e-3


def cache_of(w: DecodeWorkload, v_block_mean=None) -> F.KVCache:
    return F.KVCache(w.k, w.v, w.seqlens, w.max_seqlen, w.page_table, v_block_mean)


def oracle_block_means(w: DecodeWorkload) -> torch.Tensor:
    """The block-mean table of a workload computed by the ORACLE (float64, rounded to BF16), as a device
    tensor [num_seqs, blocks, Hkv, D]: the block tail's input in the parity tests."""
    nb = max((w.max_seqlen + 63) // 64, 1)
    t = torch.zeros(w.num_seqs, nb, w.num_kv_heads, w.head_dim, dtype=torch.float32)
    for s in range(w.num_seqs):
        for h in range(w.num_kv_heads):
            V = O.widen_bf16(bf16_bits(w.logical_rows("v", s, h)))
            if V.shape[0]:
                m = O.block_means(V)
                t[s, :m.shape[0], h] = torch.from_numpy(m).float()
    return t.to(torch.bfloat16).to(w.k.device)                # exact: the oracle's means are BF16 values already


def run_gpu(w: DecodeWorkload, T=math.inf, z_mode=F.Z_ESTIMATE, num_splits=0, z=None, bufs=None, v_block_mean=None,
            draft=None, live_hint=0.0):
    """`draft` = (masks int32 [batch], draft_len): draft / tree-verification rows."""
    cache = cache_of(w, v_block_mean)
    if bufs is None:
        bufs = F.alloc_buffers(w.q, cache, w.stack)
    if z is not None:
        bufs.z.copy_(z)
    F.decode(w.q, cache, bufs, depth_T=T, z_mode=z_mode, num_splits=num_splits, stack=w.stack, scale=w.scale,
             draft_mask=None if draft is None else draft[0], draft_len=0 if draft is None else draft[1],
             live_hint=live_hint)
    torch.cuda.synchronize()
    assert bufs.header().wait_timeouts == 0
    return bufs


def row_inputs(w: DecodeWorkload, b: int, h: int):
    G = w.num_q_heads // w.num_kv_heads
    seq, kvh = b // w.stack, h // G
    K = O.widen_bf16(bf16_bits(w.logical_rows("k", seq, kvh)))
    V = O.widen_bf16(bf16_bits(w.logical_rows("v", seq, kvh)))
    q = O.widen_bf16(bf16_bits(w.q[b, h]))
    return q, K, V


def all_rows(w: DecodeWorkload):
    return [(b, h) for b in range(w.batch) for h in range(w.num_q_heads)]


def compare(w: DecodeWorkload, bufs, T=math.inf, rows=None, check_estimate=False, yardstick=True, v_block_mean=None,
            draft=None):
    """Element-by-element comparison of the CUDA outputs with the oracle run at the GPU's own
    references.  Returns a dict of the measured errors; asserts the tolerances.  `v_block_mean`
    (the table the GPU was given) switches the oracle's block tail on; a key that flips at the threshold
    then moves between its value and its block's mean, so the threshold slack counts twice."""
    vm = None if v_block_mean is None else v_block_mean.float().cpu().numpy().astype(np.float64)
    dmask = None if draft is None else [int(x) & 0xffffffff for x in draft[0].cpu().tolist()]
    G = w.num_q_heads // w.num_kv_heads
    out = bufs.out.float().cpu().numpy().astype(np.float64)
    lse = bufs.lse.cpu().numpy().astype(np.float64)
    z = bufs.z.cpu().numpy().astype(np.float64)
    status = bufs.row_status.cpu().numpy()
    rows = rows if rows is not None else all_rows(w)
    num = den = ynum = 0.0
    max_abs = 0.0
    vmax = 0.0
    rel_rows, slack_sum, dz = [], 0.0, 0.0
    per_row = []                                             # (b, h, |d|_2, |d|_inf, |ref|_2, slack, max|V| of the row's cache)
    for (b, h) in rows:
        q, K, V = row_inputs(w, b, h)
        n = K.shape[0]
        if n == 0:
            assert not out[b, h].any() and lse[b, h] == -np.inf and status[b, h] == F.ROW_EMPTY
            continue
        s = O.scores(q, K, w.scale)
        if draft is not None:                                 # keys the row does not use: weight exactly 0
            s = O.mask_draft_scores(s, draft[1], dmask[b])
        v_mean = None if vm is None else vm[b // w.stack, :(n + 63) // 64, h // G]
        o_ref, lse_ref, _, L = O.fold_row(s, V, z[b, h], T, v_mean=v_mean)
        d = out[b, h] - o_ref
        num += float(d @ d); den += float(o_ref @ o_ref)
        max_abs = max(max_abs, float(np.abs(d).max())); vmax = max(vmax, float(np.abs(V).max()))
        rel_rows.append(np.linalg.norm(d) / max(np.linalg.norm(o_ref), 1e-300))
        assert abs(lse[b, h] - lse_ref) <= LSE_TOL, (b, h, lse[b, h], lse_ref)
        if 0.5 <= L <= 2.0 ** 100:
            assert status[b, h] == 0, (b, h, status[b, h], L)
        if check_estimate:
            dz = max(dz, abs(O.estimate_z(lambda i: s[i], n) - z[b, h]))
        if not math.isinf(T):
            row_slack = (2.0 if vm is not None else 1.0) * O.cut_report(s, V, z[b, h], T)["slack"]
            slack_sum += row_slack ** 2 * V.shape[1]
            yard_row = None
            if yardstick:
                o_dense, _ = O.dense_row(s, V)
                vis = np.isfinite(s)
                y = O.online_softmax_bf16(q, K[vis], V[vis], w.scale) - o_dense
                ynum += float(y @ y)
                yard_row = float(np.linalg.norm(y))
            per_row.append((b, h, float(np.linalg.norm(d)), float(np.abs(d).max()), float(np.linalg.norm(o_ref)), row_slack,
                            float(np.abs(V).max()), yard_row))
    res = dict(rel_l2=math.sqrt(num / max(den, 1e-300)), max_abs=max_abs, vmax=vmax,
               mean_rel=float(np.mean(rel_rows)) if rel_rows else 0.0, dz=dz)
    if math.isinf(T):
        assert max_abs <= DENSE_MAX_ABS * vmax, res
        assert res["mean_rel"] <= DENSE_MEAN_REL, res
    elif yardstick:
        res["yard"] = math.sqrt(ynum / max(den, 1e-300))
        res["slack"] = math.sqrt(slack_sum / max(den, 1e-300))
        # (1e-12: a one-key row is exact on both sides, and 0 <= 1.5 x 0 must not hinge on the oracle's own rounding)
        assert res["rel_l2"] <= FINITE_T_FACTOR * res["yard"] + res["slack"] + 1e-12, res
    if not math.isinf(T):
        # row by row, element by element: the pooled norm above cannot see one bad row among dozens
        D = w.head_dim
        for (b, h, d2, dinf, r2, row_slack, row_vmax, yard_row) in per_row:
            tol = yard_row if yard_row is not None else DENSE_MEAN_REL * r2
            assert dinf <= DENSE_MAX_ABS * row_vmax + row_slack + 1e-30, (b, h, dinf, row_vmax, row_slack)
            assert d2 <= ROW_FACTOR * tol + math.sqrt(D) * row_slack + 1e-12, (b, h, d2, r2, tol, row_slack)
        res["max_row_rel"] = max([d2 / max(r2, 1e-300) for (_, _, d2, _, r2, _, _, _) in per_row] + [0.0])
    if check_estimate:
        assert dz <= Z_TOL, res
    return res


def same_bits(a: torch.Tensor, b: torch.Tensor) -> bool:
    return torch.equal(a.contiguous().view(torch.uint8), b.contiguous().view(torch.uint8))
