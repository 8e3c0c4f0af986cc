"""Draft and tree-verification rows (Section 4 "Value product"; Appendix "Cascades and drafts"): the requests stacked
on a sequence each use the committed keys and the draft keys their mask names."""
import math

import numpy as np
import pytest
import torch

import paper_2609_33410_b200 as F
from oracle import fold_oracle as O
from paper_2609_33410_b200.workloads import make_draft_workload
from helpers import run_gpu, compare, same_bits, oracle_block_means

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.mark.parametrize("Hq,Hkv,m,D", [(4, 4, 2, 128), (8, 2, 2, 128), (8, 2, 4, 128), (8, 2, 8, 128), (8, 8, 5, 64),
                                        (8, 2, 16, 128), (8, 1, 32, 128), (4, 2, 7, 64)])
@pytest.mark.parametrize("tree", [False, True])
def test_draft_rows_match_the_oracle(Hq, Hkv, m, D, tree):
    # rows per (sequence, kv head) = m * group: 2 .. 256, so every scan kernel meets the masks;
    # contexts around tile and estimator boundaries (n <= 192: exact reference; drafts straddling a tile edge)
    ctx = [1000, 60, 190 - m]
    w, masks, m = make_draft_workload(len(ctx), m, Hq, Hkv, D, ctx, seed=101 + m, device=DEV, tree=tree,
                                      poison_padding=True, capacity=1100)
    rows = [(b, h) for b in (0, m - 1, m, 2 * m - 1, 3 * m - 1) for h in (0, Hq - 1)]
    dense = run_gpu(w, draft=(masks, m))
    compare(w, dense, rows=rows, check_estimate=True, draft=(masks, m))
    gated = run_gpu(w, T=12.0, draft=(masks, m))
    compare(w, gated, T=12.0, rows=rows, draft=(masks, m))
    # a chain's last row uses every key: it must equal the same row decoded without any mask
    if not tree:
        plain = run_gpu(w, z_mode=F.Z_GIVEN, z=dense.z.clone())
        for s in range(len(ctx)):
            b = s * m + m - 1
            assert same_bits(plain.out[b], dense.out[b]) and same_bits(plain.lse[b], dense.lse[b])
            if m > 1:
                assert not torch.equal(plain.out[s * m], dense.out[s * m])


def test_draft_rows_long_context_paged_split_invariance_and_tail():
    w, masks, m = make_draft_workload(2, 4, 8, 2, 128, [20000, 5000], seed=111, device=DEV, tree=True, paged=True,
                                      page_size=16)
    rows = [(0, 0), (3, 7), (4, 2), (7, 5)]
    b = run_gpu(w, T=16.0, draft=(masks, m))
    compare(w, b, T=16.0, rows=rows, check_estimate=True, draft=(masks, m))
    for s in (1, 4, 16):
        c = run_gpu(w, T=16.0, num_splits=s, draft=(masks, m))
        assert same_bits(c.out, b.out) and same_bits(c.lse, b.lse)
    vm = oracle_block_means(w)                                 # masks and the block tail together
    t = run_gpu(w, T=10.0, draft=(masks, m), v_block_mean=vm)
    compare(w, t, T=10.0, rows=rows, draft=(masks, m), v_block_mean=vm)


def test_bad_draft_arguments_are_refused():
    w, masks, m = make_draft_workload(1, 2, 4, 4, 128, [100], seed=113, device=DEV)
    cache = F.KVCache(w.k, w.v, w.seqlens, w.max_seqlen)
    bufs = F.alloc_buffers(w.q, cache, 2)
    a = F.make_args(w.q, cache, z=bufs.z, stack=2, workspace=bufs.workspace, out=bufs.out, lse=bufs.lse,
                    row_status=bufs.row_status, draft_mask=masks, draft_len=2)
    a.draft_len = 33
    with pytest.raises(F.FoldError) as e:
        F.fold_decode(a)
    assert e.value.status == F.FOLD_EINVAL
    a.draft_len = 2
    a.draft_mask = None
    with pytest.raises(F.FoldError) as e:
        F.fold_decode(a)
    assert e.value.status == F.FOLD_EINVAL
