"""Parity of the CUDA decode path (through the C ABI) with the float64 oracle, element by
element on the same seeded inputs: sizes span several tiles, several chunks and ragged tails."""
import math

import numpy as np
import pytest
import torch

import paper_2609_33410_b200 as F
from oracle import fold_oracle as O
from paper_2609_33410_b200.workloads import make_decode_workload, config_workload
from helpers import run_gpu, compare, all_rows, row_inputs, cache_of, same_bits

pytestmark = pytest.mark.gpu
DEV = "cuda"


def test_config1_mha_dense_and_t16():
    w = config_workload("c1", device=DEV)
    r = compare(w, run_gpu(w), check_estimate=True)
    assert r["rel_l2"] < 4e-3
    r16 = compare(w, run_gpu(w, T=16.0), T=16.0)
    assert r16["rel_l2"] <= 1.5 * r16["yard"] + r16["slack"]


@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("n", [1, 63, 64, 65, 127, 128, 129, 191, 192, 193, 255, 257, 1000])
def test_edge_lengths(D, n):
    w = make_decode_workload(2, 4, 2, D, [n, max(1, n - 17)], seed=100 + n, device=DEV, poison_padding=True,
                             capacity=n + 70)
    compare(w, run_gpu(w), check_estimate=True)
    compare(w, run_gpu(w, T=16.0), T=16.0, yardstick=n >= 64)
    compare(w, run_gpu(w, T=4.0), T=4.0, yardstick=False)


@pytest.mark.parametrize("Hq,Hkv,stack", [(1, 1, 1), (8, 8, 1), (4, 2, 1), (8, 1, 1), (16, 1, 1), (8, 2, 2), (8, 2, 4),
                                          (2, 2, 8)])
def test_group_and_stack_shapes(Hq, Hkv, stack):
    # rows per (sequence, kv head) = stack * G from 1 to 16: both halves of the MMA row block
    w = make_decode_workload(2 * stack, Hq, Hkv, 128, [700, 300], seed=7, device=DEV, stack=stack)
    compare(w, run_gpu(w))
    compare(w, run_gpu(w, T=12.0), T=12.0)


@pytest.mark.parametrize("Hq,Hkv,stack,D", [(8, 2, 5, 128), (8, 2, 16, 128), (8, 2, 20, 128), (4, 4, 33, 64),
                                            (8, 2, 64, 128), (8, 2, 40, 128), (4, 1, 75, 128)])
def test_stacked_rows_beyond_one_row_block(Hq, Hkv, stack, D):
    # 20 .. 300 query rows per (sequence, kv head): the stacked-row kernels, with ragged 16-, 64- and 128-row groups
    # (160 rows: a full and a partial 128-row tile in one pair; 300 rows: a second pair whose second tile is empty)
    w = make_decode_workload(2 * stack, Hq, Hkv, D, [1500, 333], seed=9, device=DEV, stack=stack,
                             poison_padding=True, capacity=1600)
    rows = [(b, h) for b in (0, 1, stack - 1, stack, 2 * stack - 1) for h in (0, Hq - 1)]
    compare(w, run_gpu(w), rows=rows, check_estimate=True)
    compare(w, run_gpu(w, T=12.0), T=12.0, rows=rows)
    p = make_decode_workload(stack, Hq, Hkv, D, [9000], seed=10, device=DEV, stack=stack, paged=True, page_size=32)
    rows = [(b, h) for b in (0, stack // 2, stack - 1) for h in (1, Hq - 2)]
    compare(p, run_gpu(p, T=16.0), T=16.0, rows=rows)


@pytest.mark.parametrize("page_size", [16, 32, 64, 128])
@pytest.mark.parametrize("D", [64, 128])
def test_paged_layout_and_poisoned_tails(page_size, D):
    w = make_decode_workload(3, 8, 2, D, [1500, 64, 333], seed=11, device=DEV, paged=True, page_size=page_size,
                             poison_padding=True)
    compare(w, run_gpu(w), check_estimate=True)
    compare(w, run_gpu(w, T=16.0), T=16.0)


def test_several_chunks_long_context_sampled_rows():
    # > 8192 keys: 1024-key chunks; ragged batch; sampled rows keep the oracle to seconds
    w = make_decode_workload(3, 8, 2, 128, [20000, 9001, 8192], seed=13, device=DEV)
    rows = [(0, 0), (0, 7), (1, 3), (2, 4)]
    compare(w, run_gpu(w), rows=rows, check_estimate=True)
    compare(w, run_gpu(w, T=16.0), T=16.0, rows=rows)
    compare(w, run_gpu(w, T=8.0), T=8.0, rows=rows, yardstick=False)


def test_head_major_cache_strides():
    # [seq, head, token, D] storage viewed as [seq, token, head, D]: only strides differ
    w = make_decode_workload(2, 8, 4, 128, [900, 400], seed=17, device=DEV)
    base = run_gpu(w)
    k2 = w.k.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    v2 = w.v.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    assert k2.stride() != w.k.stride()
    cache = F.KVCache(k2, v2, w.seqlens, w.max_seqlen)
    bufs = F.alloc_buffers(w.q, cache)
    for T in (math.inf, 16.0):
        F.decode(w.q, cache, bufs, depth_T=T)
        ref = run_gpu(w, T=T, bufs=base)
        torch.cuda.synchronize()
        assert same_bits(bufs.out, ref.out) and same_bits(bufs.lse, ref.lse)


def test_range_certificate_rerun_repairs_flagged_rows_and_leaves_the_others_alone():
    # Section 3, "Choosing the reference": a row whose L leaves [2^-1, 2^100] is decoded again with Z = its lse
    w = make_decode_workload(2, 8, 2, 128, [3000, 1111], seed=23, device=DEV)
    cache = cache_of(w)
    good = run_gpu(w, T=16.0)
    z = good.z.clone()
    z[0, 3] += 40.0                                             # L = 2^-40: below the certificate's range
    z[1, 6] -= 110.0                                            # L = 2^110: above it
    bufs = F.alloc_buffers(w.q, cache, w.stack)
    bufs.z.copy_(z)
    F.decode(w.q, cache, bufs, depth_T=16.0, z_mode=F.Z_GIVEN, scale=w.scale)
    torch.cuda.synchronize()
    st = bufs.row_status.cpu().numpy()
    assert (st[0, 3] & F.ROW_RANGE) and (st[1, 6] & F.ROW_RANGE) and (st != 0).sum() == 2
    bufs.z.copy_(z)
    assert F.decode_certified(w.q, cache, bufs, depth_T=16.0, z_mode=F.Z_GIVEN, scale=w.scale) == 1
    torch.cuda.synchronize()
    assert not bufs.row_status.any()
    keep = torch.ones_like(bufs.row_status, dtype=torch.bool); keep[0, 3] = False; keep[1, 6] = False
    assert same_bits(bufs.out[keep], good.out[keep]) and same_bits(bufs.lse[keep], good.lse[keep])
    assert abs(float(bufs.z[0, 3] - good.lse[0, 3])) < 1e-2 and abs(float(bufs.z[1, 6] - good.lse[1, 6])) < 1e-2
    compare(w, bufs, T=16.0)                                    # every row against the oracle at its final reference
    assert F.decode_certified(w.q, cache, bufs, depth_T=16.0, scale=w.scale) == 0      # estimated references are in range


def test_reference_modes_and_fp32_range():
    w = make_decode_workload(2, 8, 2, 128, [3000, 1111], seed=19, device=DEV)
    est = run_gpu(w)
    lse = est.lse.clone()
    base = compare(w, est)
    # Prop. 1(ii)/(iii): any reference within 80 binades of the row's scores gives the same output
    for dz in (-80.0, -30.0, 30.0, 80.0):
        b = run_gpu(w, z_mode=F.Z_GIVEN, z=lse + dz)
        r = compare(w, b)
        assert abs(r["rel_l2"] - base["rel_l2"]) < 1e-3
        st = b.row_status.cpu().numpy()
        # the range certificate flags rows whose L leaves [2^-1, 2^100]  (L = 2^(lse - z))
        assert np.all((st & F.ROW_RANGE) != 0) if dz > 1 else np.all(st == 0)
    compare(w, run_gpu(w, z_mode=F.Z_ZERO))
    mx = run_gpu(w, z_mode=F.Z_EXACT_MAX)
    compare(w, mx)
    z = mx.z.cpu().numpy()
    for (b_, h) in [(0, 0), (1, 5)]:
        q, K, V = row_inputs(w, b_, h)
        assert abs(O.scores(q, K).max() - z[b_, h]) < 1e-3


def test_empty_and_mixed_empty_sequences():
    w = make_decode_workload(3, 4, 2, 128, [0, 500, 0], seed=23, device=DEV, capacity=512)
    b = run_gpu(w)
    compare(w, b)
    st = b.row_status.cpu().numpy()
    assert np.all(st[0] == F.ROW_EMPTY) and np.all(st[2] == F.ROW_EMPTY) and np.all(st[1] == 0)
    compare(w, run_gpu(w, T=16.0), T=16.0)


def test_constant_values_show_the_cut_mass_is_kept():
    # all values equal c: dense output is c; at depth T it is c * (1 - cut mass), not c
    w = make_decode_workload(1, 4, 4, 128, 4096, seed=29, device=DEV)
    w.v.fill_(1.5)
    d = run_gpu(w)
    assert torch.allclose(d.out.float(), torch.full_like(d.out.float(), 1.5), rtol=1e-2)
    t = run_gpu(w, T=6.0)
    o = t.out.float().cpu().numpy()
    z = t.z.cpu().numpy()
    for h in range(4):
        q, K, V = row_inputs(w, 0, h)
        cm = O.cut_report(O.scores(q, K), V, z[0, h], 6.0)["cut_mass"]
        assert cm > 0.02
        assert np.allclose(o[0, h], 1.5 * (1 - cm), rtol=2e-2)
    assert same_bits(d.lse, t.lse)            # L, hence lse, is the same at every depth


def test_host_buffer_entry_point_matches_device_path():
    w = make_decode_workload(2, 8, 2, 128, [2500, 700], seed=31, device=DEV, paged=True, page_size=64)
    ref = run_gpu(w, T=16.0)
    hq, hk, hv = w.q.cpu().pin_memory(), w.k.cpu().pin_memory(), w.v.cpu().pin_memory()
    hlen, htab = w.seqlens.cpu().pin_memory(), w.page_table.cpu().pin_memory()
    hout = torch.empty(2, 8, 128, dtype=torch.bfloat16).pin_memory()
    hlse = torch.empty(2, 8, dtype=torch.float32).pin_memory()
    hz = torch.empty(2, 8, dtype=torch.float32).pin_memory()
    hst = torch.empty(2, 8, dtype=torch.int32).pin_memory()
    cache = F.KVCache(hk, hv, hlen, w.max_seqlen, htab)
    args = F.make_args(hq, cache, depth_T=16.0, z=hz, out=hout, lse=hlse, row_status=hst)
    nbytes = F.fold_host_staging_bytes(args)
    assert nbytes > 2 * hk.numel() * 2
    staging = torch.empty(nbytes, dtype=torch.uint8, device=DEV)
    F.fold_decode_host(args, staging)
    torch.cuda.synchronize()
    assert same_bits(hout, ref.out.cpu()) and same_bits(hlse, ref.lse.cpu()) and same_bits(hz, ref.z.cpu())
    assert not hst.any()


def test_rejects_bad_arguments_with_status_codes():
    w = make_decode_workload(1, 4, 2, 128, 300, seed=37, device=DEV)
    cache = cache_of(w)
    bufs = F.alloc_buffers(w.q, cache)

    def status(**kw):
        a = F.make_args(w.q, cache, z=bufs.z, workspace=bufs.workspace, out=bufs.out, lse=bufs.lse, **kw)
        return a

    a = status(depth_T=-1.0)
    assert F.lib().fold_decode(a, None) == F.FOLD_EINVAL
    a = status(depth_T=float("nan"))
    assert F.lib().fold_decode(a, None) == F.FOLD_EINVAL
    a = status(); a.workspace_bytes = 64
    assert F.lib().fold_decode(a, None) == F.FOLD_EWORKSPACE
    a = status(); a.head_dim = 96
    assert F.lib().fold_decode(a, None) == F.FOLD_EUNSUPPORTED
    a = status(); a.q = a.q + 2
    assert F.lib().fold_decode(a, None) == F.FOLD_EINVAL
    a = status(); a.num_q_heads = 64; a.num_kv_heads = 2      # a group of 32 rows is wider than one row block
    assert F.lib().fold_decode(a, None) == F.FOLD_EUNSUPPORTED
    torch.cuda.synchronize()
