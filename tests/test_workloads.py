"""Seeded input generator: shapes, determinism, the sink, the boosted keys, the paged scatter."""
import numpy as np
import torch

from paper_2609_33410_b200.workloads import make_decode_workload, config_workload, bf16_bits


def test_deterministic_and_shapes():
    a = make_decode_workload(2, 8, 2, 64, [300, 257], seed=3)
    b = make_decode_workload(2, 8, 2, 64, [300, 257], seed=3)
    c = make_decode_workload(2, 8, 2, 64, [300, 257], seed=4)
    assert torch.equal(a.k, b.k) and torch.equal(a.q, b.q) and not torch.equal(a.k, c.k)
    assert a.k.shape == (2, 300, 2, 64) and a.q.shape == (2, 8, 64) and a.k.dtype == torch.bfloat16
    assert a.seqlens.tolist() == [300, 257] and a.cache_bytes() == (300 + 257) * 2 * 4 * 64
    assert bf16_bits(a.q).dtype == np.uint16


def test_sink_and_boosted_keys():
    n, D = 20001, 128
    w = make_decode_workload(1, 4, 1, D, n, seed=5)
    plain = make_decode_workload(1, 4, 1, D, n, seed=5, peak_frac=0.0, sink_gain=1.0)
    k, k0 = w.k[0, :, 0].float(), plain.k[0, :, 0].float()
    assert torch.allclose(k[0], 8 * k0[0], rtol=1e-2)           # sink: key 0 scaled x8
    changed = (k[1:] != k0[1:]).any(dim=1)
    assert changed.sum().item() == round(0.01 * (n - 1))        # 1 % of tokens j >= 1 boosted
    # each boosted key moved by 4 * q_hat of exactly one head of the group
    qhat = torch.nn.functional.normalize(w.q[0].float(), dim=-1)
    delta = (k[1:] - k0[1:])[changed]
    cos = torch.nn.functional.normalize(delta, dim=-1) @ qhat.T
    assert (cos.max(dim=1).values > 0.99).all()
    assert torch.allclose(delta.norm(dim=1), torch.full((delta.shape[0],), 4.0), atol=0.1)
    assert torch.equal(w.v, plain.v)


def test_paged_layout_holds_the_same_logical_rows():
    w = make_decode_workload(3, 4, 2, 64, [130, 64, 1], seed=7, paged=True, page_size=16, poison_padding=True)
    assert w.paged and w.k.shape[1] == 16
    used = sum((n + 15) // 16 for n in (130, 64, 1))
    assert w.k.shape[0] == used
    ids = torch.cat([w.page_table[s, : (n + 15) // 16] for s, n in enumerate((130, 64, 1))])
    assert sorted(ids.tolist()) == list(range(used))           # a permutation of the pool
    for s, n in enumerate((130, 64, 1)):
        rows = w.logical_rows("k", s, 1)
        assert rows.shape == (n, 64) and not torch.isnan(rows.float()).any()
    assert torch.isnan(w.k.float()).any()                       # page tails are poisoned


def test_stacked_requests_share_one_sequence():
    w = make_decode_workload(6, 4, 2, 64, [100, 90], seed=8, stack=3)
    assert w.num_seqs == 2 and w.batch == 6 and w.k.shape[0] == 2


def test_named_configs_small():
    w = config_workload("c1")
    assert (w.batch, w.num_q_heads, w.num_kv_heads, w.head_dim, w.max_seqlen) == (1, 8, 8, 128, 4096)
    w = config_workload("c3", small=True)
    assert w.paged and w.page_size == 64


def test_draft_workload_masks_are_chains_or_ancestor_closed_trees():
    from paper_2609_33410_b200.workloads import make_draft_workload
    w, masks, m = make_draft_workload(3, 5, 4, 2, 64, [10, 20, 7], seed=5)
    assert w.batch == 15 and w.stack == 5 and [int(x) for x in w.seqlens] == [15, 25, 12]
    assert [int(x) for x in masks[:5]] == [1, 3, 7, 15, 31]
    w, masks, m = make_draft_workload(4, 8, 4, 2, 64, 9, seed=6, tree=True)
    for s in range(4):
        row = [int(x) & 0xffffffff for x in masks[s * 8:(s + 1) * 8]]
        for r, mk in enumerate(row):
            assert (mk >> r) & 1 and mk < (1 << (r + 1))                  # itself, and nothing later
            for t in range(r):
                if (mk >> t) & 1:
                    assert row[t] & mk == row[t]                          # an ancestor's ancestors are ancestors
    w, masks, m = make_draft_workload(1, 32, 2, 2, 64, 3, seed=7)
    assert int(masks[31]) == -1                                           # all 32 bits, stored as int32
