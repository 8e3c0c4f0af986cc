"""Block tail (Section 4, "Depth as a dial": the block model's mean): cut keys add their weight times the mean
value of their 64-key block.  The table of means is an INPUT of the scan: the parity tests take it from the oracle;
the library's own table builder is checked against the oracle separately, bit for bit."""
import math

import numpy as np
import pytest
import torch

import paper_2609_33410_b200 as F
from oracle import fold_oracle as O
from paper_2609_33410_b200.workloads import make_decode_workload, bf16_bits
from helpers import run_gpu, compare, cache_of, same_bits, oracle_block_means

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("paged", [False, True])
def test_block_means_match_the_oracle_bit_for_bit(D, paged):
    lens = [1, 63, 64, 65, 1000, 4133]
    w = make_decode_workload(len(lens), 4, 2, D, lens, seed=81, device=DEV, paged=paged, page_size=32,
                             poison_padding=True, capacity=None if paged else 4200)
    cache = cache_of(w)
    table = torch.full_like(cache.alloc_block_means(), 7.0)   # blocks past a sequence's end must stay untouched
    cache.v_block_mean = table
    F.fold_block_means(cache)
    torch.cuda.synchronize()
    ref = oracle_block_means(w)
    for s, n in enumerate(lens):
        nb = (n + 63) // 64
        assert same_bits(table[s, :nb], ref[s, :nb]), (s, n)
        assert bool((table[s, nb:] == 7.0).all())


@pytest.mark.parametrize("Hq,Hkv", [(8, 8), (8, 2), (8, 1)])
@pytest.mark.parametrize("D", [64, 128])
def test_block_tail_matches_the_oracle(Hq, Hkv, D):
    w = make_decode_workload(2, Hq, Hkv, D, [3000, 733], seed=83, device=DEV, poison_padding=True, capacity=3100)
    vm = oracle_block_means(w)
    for T in (8.0, 12.0, 16.0):
        b = run_gpu(w, T=T, v_block_mean=vm)
        r = compare(w, b, T=T, v_block_mean=vm)
        plain = run_gpu(w, T=T, z_mode=F.Z_GIVEN, z=b.z.clone())
        if T == 8.0:                                           # plenty is cut at depth 8: the tail must show
            assert not torch.equal(plain.out, b.out)
        assert same_bits(plain.lse, b.lse)                     # the mass is the same either way


def test_block_tail_paged_long_context_sampled_rows():
    w = make_decode_workload(2, 8, 2, 128, [40000, 9000], seed=85, device=DEV, paged=True, page_size=16)
    vm = oracle_block_means(w)
    rows = [(0, 0), (0, 5), (1, 2), (1, 7)]
    b = run_gpu(w, T=16.0, v_block_mean=vm)
    compare(w, b, T=16.0, rows=rows, v_block_mean=vm)
    # scheduling never changes a bit, with the tail on as well
    for s in (1, 3, 8):
        c = run_gpu(w, T=16.0, num_splits=s, v_block_mean=vm)
        assert same_bits(c.out, b.out) and same_bits(c.lse, b.lse)


def test_block_tail_is_exact_for_values_constant_within_blocks():
    # every key holds its block's mean: cutting changes nothing, so a shallow depth must reproduce dense decode
    w = make_decode_workload(2, 8, 2, 128, [2048, 1000], seed=87, device=DEV)
    blk = (torch.arange(w.v.shape[1], device=DEV) // 64)
    w.v.copy_(w.v[:, (blk * 64).clamp(max=w.v.shape[1] - 1)])
    cache = cache_of(w)
    vm = F.fold_block_means(cache)
    torch.cuda.synchronize()
    dense = run_gpu(w)
    z = dense.z.clone()
    shallow = run_gpu(w, T=6.0, z_mode=F.Z_GIVEN, z=z, v_block_mean=vm)
    cut = run_gpu(w, T=6.0, z_mode=F.Z_GIVEN, z=z)
    a, b, c = dense.out.float(), shallow.out.float(), cut.out.float()
    assert (a - b).norm() / a.norm() < 4e-3                    # two BF16 output roundings apart
    assert (a - c).norm() / a.norm() > 5e-2                    # without the tail the cut shows
    assert bool(shallow.header().v_rows_fetched < 0.6 * shallow.header().v_rows_total)


@pytest.mark.parametrize("Hq,Hkv,stack,D", [(16, 1, 1, 128), (12, 1, 1, 64), (8, 2, 4, 128), (8, 2, 5, 128), (4, 4, 33, 64),
                                            (8, 2, 16, 128), (8, 2, 40, 128), (8, 2, 75, 128)])
def test_block_tail_with_wider_row_blocks_and_stacked_rows(Hq, Hkv, stack, D):
    # 9..16 rows per (sequence, kv head): the rows-on-M gated kernel; more: the stacked-row kernels (from 64 rows at
    # head_dim 128 on tcgen05: 64, 160 and 300 rows here, i.e. one, two and three row tiles)
    w = make_decode_workload(2 * stack, Hq, Hkv, D, [1500, 333], seed=91, device=DEV, stack=stack,
                             poison_padding=True, capacity=1600)
    vm = oracle_block_means(w)
    rows = [(b, h) for b in (0, stack - 1, stack, 2 * stack - 1) for h in (0, Hq - 1)]
    for T in (8.0, 14.0):
        b = run_gpu(w, T=T, v_block_mean=vm)
        compare(w, b, T=T, rows=rows, v_block_mean=vm)
        plain = run_gpu(w, T=T, z_mode=F.Z_GIVEN, z=b.z.clone())
        # the mass is the same either way (a stacked level without the table may run on another kernel: not the same bits)
        assert torch.allclose(plain.lse, b.lse, atol=1e-4, rtol=0)
        if T == 8.0:
            assert not torch.equal(plain.out, b.out)
    b1 = run_gpu(w, T=14.0, num_splits=1, v_block_mean=vm)
    assert same_bits(b1.out, b.out)


def test_block_tail_in_a_shared_prefix_cascade():
    # each level has its own table (blocks are local to a level's sequence); the oracle walks prefix ++ suffix with
    # the two tables one after the other
    B, Hq, Hkv, D, P = 6, 8, 2, 128, 1000
    suffixes = [300, 1, 0, 257, 64, 65]
    g = torch.Generator(device=DEV); g.manual_seed(93)
    q = torch.randn(B, Hq, D, generator=g, device=DEV).to(torch.bfloat16)
    pre = make_decode_workload(B, Hq, Hkv, D, P, seed=94, device=DEV, stack=B, q=q)
    suf = make_decode_workload(B, Hq, Hkv, D, suffixes, seed=95, device=DEV, q=q, sink_gain=1.0)
    vmp, vms = oracle_block_means(pre), oracle_block_means(suf)
    cp, cs = cache_of(pre, vmp), cache_of(suf, vms)
    bp, bs = F.alloc_buffers(q, cp, stack=B), F.alloc_buffers(q, cs)
    T = 10.0
    ap = F.make_args(q, cp, z=bs.z, depth_T=T, stack=B, workspace=bp.workspace, out=bs.out, lse=bs.lse,
                     row_status=bs.row_status)
    as_ = F.make_args(q, cs, z=bs.z, depth_T=T, workspace=bs.workspace, out=bs.out, lse=bs.lse, row_status=bs.row_status)
    F.fold_decode_cascade([ap, as_])
    torch.cuda.synchronize()
    assert bp.header().wait_timeouts == 0 and bs.header().wait_timeouts == 0
    out = bs.out.float().cpu().numpy().astype(np.float64)
    z = bs.z.cpu().numpy().astype(np.float64)
    mp, ms = vmp.float().cpu().numpy().astype(np.float64), vms.float().cpu().numpy().astype(np.float64)
    nbp = (P + 63) // 64
    num = den = 0.0
    for b in range(B):
        for h in (0, 3, 7):
            kvh = h // (Hq // Hkv)
            n_s = suffixes[b]
            K = np.concatenate([O.widen_bf16(bf16_bits(pre.logical_rows("k", 0, kvh))),
                                O.widen_bf16(bf16_bits(suf.logical_rows("k", b, kvh)))])
            V = np.concatenate([O.widen_bf16(bf16_bits(pre.logical_rows("v", 0, kvh))),
                                O.widen_bf16(bf16_bits(suf.logical_rows("v", b, kvh)))])
            s = O.scores(O.widen_bf16(bf16_bits(q[b, h])), K)
            table = np.concatenate([mp[0, :nbp, kvh], ms[b, :(n_s + 63) // 64, kvh]])
            block_of = np.concatenate([np.arange(P) // 64, nbp + np.arange(n_s) // 64])
            A, L = O.fold_partial(s, V, z[b, h], T, tail=(table, block_of))
            d = out[b, h] - A / L
            num += d @ d; den += (A / L) @ (A / L)
    assert math.sqrt(num / den) < 4e-3


