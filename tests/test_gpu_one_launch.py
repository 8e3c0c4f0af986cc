"""A decode of one wave can run reference, scan and partial add inside one cooperative launch (Section 3's three
steps, Algorithm 1 unchanged; FOLD_ONE_LAUNCH, and the default with a given reference).  The bar is bit equality with
the separate launches -- out, lse, z, the row flags and the header's counters -- plus parity with the oracle."""
import math

import pytest
import torch

import paper_2609_33410_b200 as F
from paper_2609_33410_b200.workloads import make_decode_workload
from helpers import cache_of, compare, same_bits, oracle_block_means

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _decode(w, T, flags, z_mode=F.Z_ESTIMATE, z=None, vm=None, draft=None, poison=True):
    cache = cache_of(w, vm)
    bufs = F.alloc_buffers(w.q, cache, w.stack)
    if poison:                                                 # whatever the buffers held before must not matter
        bufs.workspace.fill_(0xA5)
        bufs.out.fill_(7.0); bufs.lse.fill_(7.0); bufs.row_status.fill_(-1)
        if z is None:
            bufs.z.fill_(7.0)
    if z is not None:
        bufs.z.copy_(z)
    args = F.decode(w.q, cache, bufs, depth_T=T, z_mode=z_mode, stack=w.stack, scale=w.scale, flags=flags,
                    draft_mask=None if draft is None else draft[0], draft_len=0 if draft is None else draft[1])
    torch.cuda.synchronize()
    assert bufs.header().wait_timeouts == 0
    return bufs, F.fold_decode_launches(args)


def _same(a, b):
    assert same_bits(a.out, b.out)
    assert same_bits(a.lse, b.lse)
    assert same_bits(a.z, b.z)
    assert torch.equal(a.row_status, b.row_status)
    ha, hb = a.header(), b.header()
    assert (ha.v_rows_fetched, ha.v_rows_total, ha.v_slices_skipped) == (hb.v_rows_fetched, hb.v_rows_total, hb.v_slices_skipped)


SHAPES = [
    # batch, q heads, kv heads, lengths, paged
    (1, 8, 8, [4096], False),                  # config 1: 8 x 16 chunks, one per worker
    (1, 8, 8, [4001], True),
    (3, 8, 2, [3000, 0, 777], False),          # GQA group of 4, an empty sequence, ragged tails
    (2, 16, 2, [1500, 129], True),             # 8 rows per kv head
    (4, 4, 4, [1, 255, 256, 257], False),      # one key; a tile and a chunk boundary
    (1, 2, 1, [30000], False),                 # 1024-key chunks, 30 slots for one row pair
]


@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("T", [math.inf, 16.0, 8.0])
def test_one_launch_equals_three_launches_bit_for_bit(shape, T):
    B, Hq, Hkv, lens, paged = shape
    w = make_decode_workload(B, Hq, Hkv, 128, lens, seed=101, device=DEV, paged=paged, page_size=16,
                             poison_padding=True, capacity=None if paged else max(lens) + 70)
    one, n1 = _decode(w, T, F.ONE_LAUNCH)
    three, n3 = _decode(w, T, F.SEPARATE_LAUNCHES)
    assert (n1, n3) == (1, 3)
    _same(one, three)
    compare(w, one, T=T, check_estimate=True)
    # a given reference: two launches become one
    given1, m1 = _decode(w, T, 0, z_mode=F.Z_GIVEN, z=three.z.clone())
    given2, m2 = _decode(w, T, F.SEPARATE_LAUNCHES, z_mode=F.Z_GIVEN, z=three.z.clone())
    assert (m1, m2) == (1, 2)
    _same(given1, given2)
    assert same_bits(given1.out, one.out) and same_bits(given1.lse, one.lse)


def test_one_launch_with_the_block_tail_and_with_draft_rows():
    w = make_decode_workload(2, 8, 2, 128, [3000, 733], seed=103, device=DEV, poison_padding=True, capacity=3100)
    vm = oracle_block_means(w)
    for T in (8.0, 16.0):
        one, n1 = _decode(w, T, F.ONE_LAUNCH, vm=vm)
        three, n3 = _decode(w, T, F.SEPARATE_LAUNCHES, vm=vm)
        assert (n1, n3) == (1, 3)
        _same(one, three)
        compare(w, one, T=T, v_block_mean=vm)
    masks = torch.tensor([0b1011, 0b0110], dtype=torch.int32, device=DEV)
    one, n1 = _decode(w, 16.0, F.ONE_LAUNCH, draft=(masks, 4))
    three, _ = _decode(w, 16.0, F.SEPARATE_LAUNCHES, draft=(masks, 4))
    assert n1 == 1
    _same(one, three)


def test_larger_problems_and_other_shapes_keep_their_separate_launches():
    # more chunks than two per SM; head_dim 64; a split hint that bounds the grid
    big = make_decode_workload(2, 16, 16, 128, [8192, 8192], seed=105, device=DEV)   # 1024 chunks
    d64 = make_decode_workload(1, 8, 8, 64, [4096], seed=105, device=DEV)
    for w in (big, d64):
        cache = cache_of(w)
        bufs = F.alloc_buffers(w.q, cache, w.stack)
        args = F.make_args(w.q, cache, scale=w.scale, z=bufs.z, workspace=bufs.workspace, out=bufs.out, lse=bufs.lse,
                           row_status=bufs.row_status, flags=F.ONE_LAUNCH)
        assert F.fold_decode_launches(args) == 3
    small = make_decode_workload(1, 8, 8, 128, [4096], seed=105, device=DEV)
    cache = cache_of(small)
    bufs = F.alloc_buffers(small.q, cache, 1)
    hinted = F.make_args(small.q, cache, scale=small.scale, z=bufs.z, workspace=bufs.workspace, out=bufs.out, lse=bufs.lse,
                         row_status=bufs.row_status, num_splits=2, flags=F.ONE_LAUNCH)
    assert F.fold_decode_launches(hinted) == 3
    # with neither flag: one launch for a given reference, separate kernels for the estimate
    for zm, want in ((F.Z_ESTIMATE, 3), (F.Z_GIVEN, 1)):
        a = F.make_args(small.q, cache, scale=small.scale, z=bufs.z, z_mode=zm, workspace=bufs.workspace, out=bufs.out,
                        lse=bufs.lse, row_status=bufs.row_status)
        assert F.fold_decode_launches(a) == want


def test_one_launch_decode_under_stream_capture_and_replay():
    w = make_decode_workload(1, 8, 8, 128, [4096], seed=107, device=DEV)
    cache = cache_of(w)
    ref, _ = _decode(w, 16.0, F.SEPARATE_LAUNCHES, poison=False)
    bufs = F.alloc_buffers(w.q, cache, 1)
    args = F.make_args(w.q, cache, scale=w.scale, z=bufs.z, depth_T=16.0, workspace=bufs.workspace, out=bufs.out,
                       lse=bufs.lse, row_status=bufs.row_status, flags=F.ONE_LAUNCH)
    assert F.fold_decode_launches(args) == 1
    F.fold_decode(args)                                         # first launch of the kernel outside the capture
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    s = torch.cuda.Stream()
    with torch.cuda.graph(g, stream=s):
        F.fold_decode(args, stream=s)
    for _ in range(3):
        bufs.out.zero_()
        g.replay()
    torch.cuda.synchronize()
    assert same_bits(bufs.out, ref.out) and same_bits(bufs.lse, ref.lse)
    assert bufs.header().wait_timeouts == 0
