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


def test_block_tail_is_refused_where_it_is_not_built():
    w = make_decode_workload(1, 16, 1, 128, [500], seed=89, device=DEV)        # 16 rows per kv head
    vm = oracle_block_means(w)
    cache = cache_of(w, vm)
    bufs = F.alloc_buffers(w.q, cache)
    with pytest.raises(F.FoldError) as e:
        F.decode(w.q, cache, bufs, depth_T=16.0)
    assert e.value.status == F.FOLD_EUNSUPPORTED
    F.decode(w.q, cache, bufs, depth_T=math.inf)               # dense decode ignores the table
    torch.cuda.synchronize()
