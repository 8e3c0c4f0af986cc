"""The benchmark configurations at full size, in the launch configuration bench.py times
(split hint 0 = the library's choice), checked against the oracle on sampled rows the
oracle can compute one by one."""
import math

import numpy as np
import pytest
import torch

import paper_2609_33410_b200 as F
from oracle import fold_oracle as O
from paper_2609_33410_b200.workloads import make_decode_workload, make_cascade_workload, DecodeWorkload, bf16_bits
from helpers import run_gpu, compare, cache_of, same_bits

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _free_gb():
    free, _ = torch.cuda.mem_get_info()
    return free / 2 ** 30


def test_config2_gqa_batch16_32k_sampled_rows():
    if _free_gb() < 12:
        pytest.skip("not enough free device memory")
    w = make_decode_workload(16, 32, 8, 128, 32768, seed=1, device=DEV)
    rows = [(0, 0), (3, 13), (7, 31), (15, 18)]
    b = run_gpu(w, T=16.0)
    r = compare(w, b, T=16.0, rows=rows, check_estimate=True)
    ref = b.out.clone()
    assert same_bits(run_gpu(w, T=16.0, num_splits=8).out, ref)          # the configuration's 8-way split: same bits
    # the benchmark's timed steps carry the live fraction of their warm-up steps as a hint (here: all live, so the scan
    # runs two key and four value stages); a low hint picks four and two: the same bits, and parity holds for them
    hdr = b.header()
    hinted = run_gpu(w, T=16.0, live_hint=hdr.v_rows_fetched / hdr.v_rows_total)
    assert same_bits(hinted.out, ref) and same_bits(hinted.lse, b.lse)
    compare(w, hinted, T=16.0, rows=rows)
    assert same_bits(run_gpu(w, T=16.0, live_hint=0.001).out, ref)
    compare(w, run_gpu(w), rows=rows)
    del w
    torch.cuda.empty_cache()


def test_config3_paged_128k_sampled_rows():
    if _free_gb() < 12:
        pytest.skip("not enough free device memory")
    w = make_decode_workload(4, 32, 8, 128, 131072, seed=2, device=DEV, paged=True, page_size=64)
    rows = [(0, 5), (1, 30), (3, 0)]
    b = run_gpu(w, T=16.0)
    compare(w, b, T=16.0, rows=rows, check_estimate=True)
    assert same_bits(run_gpu(w, T=16.0, num_splits=32).out, b.out.clone())
    hdr = b.header()
    assert same_bits(run_gpu(w, T=16.0, live_hint=hdr.v_rows_fetched / hdr.v_rows_total).out, b.out)   # as bench.py times it
    compare(w, run_gpu(w), rows=rows)
    del w
    torch.cuda.empty_cache()


def test_config3_with_the_block_tail_sampled_rows():
    if _free_gb() < 12:
        pytest.skip("not enough free device memory")
    w = make_decode_workload(4, 32, 8, 128, 131072, seed=2, device=DEV, paged=True, page_size=64)
    cache = cache_of(w)
    vm = F.fold_block_means(cache)                           # the library's table; sampled heads checked bit for bit
    torch.cuda.synchronize()
    for (s, kvh) in [(0, 1), (3, 7)]:
        V = O.widen_bf16(bf16_bits(w.logical_rows("v", s, kvh)))
        ref = torch.from_numpy(O.block_means(V)).float().to(torch.bfloat16).to(DEV)
        assert same_bits(vm[s, :, kvh], ref)
    rows = [(0, 5), (3, 28)]
    b = run_gpu(w, T=16.0, v_block_mean=vm)
    compare(w, b, T=16.0, rows=rows, v_block_mean=vm)
    assert same_bits(run_gpu(w, T=16.0, num_splits=32, v_block_mean=vm).out, b.out.clone())
    del w, vm, cache
    torch.cuda.empty_cache()


def test_config5_cell_mha_head_dim_64_sampled_rows():
    # one cell of the sweep at full size: MHA, 32 heads, D = 64 (128-key tiles), batch 8, 32768 keys, T in {8, 16, inf}
    if _free_gb() < 12:
        pytest.skip("not enough free device memory")
    w = make_decode_workload(8, 32, 32, 64, 32768, seed=5000 + 64 * 7 + 8 * 131 + 32768, device=DEV)
    rows = [(0, 0), (3, 17), (7, 31)]
    for T in (8.0, 16.0, math.inf):
        b = run_gpu(w, T=T)
        compare(w, b, T=T, rows=rows, check_estimate=True)
        if T == 8.0:
            h = b.header()
            assert h.v_rows_fetched < 0.05 * h.v_rows_total          # nearly every value row is cut and not read
            assert same_bits(run_gpu(w, T=T, num_splits=4).out, b.out.clone())
    del w
    torch.cuda.empty_cache()


def test_config4_shared_prefix_cascade_sampled_rows():
    if _free_gb() < 8:
        pytest.skip("not enough free device memory")
    B, Hq, Hkv, D, P, S = 64, 32, 8, 128, 16384, 2048
    pre, suf = make_cascade_workload(B, Hq, Hkv, D, P, S, seed=3, device=DEV)
    cp, cs = cache_of(pre), cache_of(suf)
    bp, bs = F.alloc_buffers(pre.q, cp, stack=B), F.alloc_buffers(pre.q, cs)
    ap = F.make_args(pre.q, cp, z=bs.z, depth_T=16.0, stack=B, workspace=bp.workspace, out=bs.out, lse=bs.lse,
                     row_status=bs.row_status)
    as_ = F.make_args(pre.q, cs, z=bs.z, depth_T=16.0, workspace=bs.workspace, out=bs.out, lse=bs.lse,
                      row_status=bs.row_status)
    F.fold_decode_cascade([ap, as_])
    torch.cuda.synchronize()
    assert bp.header().wait_timeouts == 0 and bs.header().wait_timeouts == 0
    out = bs.out.float().cpu().numpy().astype(np.float64)
    z = bs.z.cpu().numpy().astype(np.float64)
    num = den = ynum = 0.0
    for (b, h) in [(0, 0), (17, 9), (63, 31)]:
        kvh = h // 4
        K = np.concatenate([O.widen_bf16(bf16_bits(pre.logical_rows("k", 0, kvh))),
                            O.widen_bf16(bf16_bits(suf.logical_rows("k", b, kvh)))])
        V = np.concatenate([O.widen_bf16(bf16_bits(pre.logical_rows("v", 0, kvh))),
                            O.widen_bf16(bf16_bits(suf.logical_rows("v", b, kvh)))])
        q = O.widen_bf16(bf16_bits(pre.q[b, h]))
        s = O.scores(q, K)
        assert abs(O.estimate_z(lambda i: s[i], len(s)) - z[b, h]) < 1e-3
        ref, _, _, _ = O.fold_row(s, V, z[b, h], 16.0)
        d = out[b, h] - ref
        num += d @ d; den += ref @ ref
        y = O.online_softmax_bf16(q, K, V) - O.dense_row(s, V)[0]
        ynum += y @ y
    assert math.sqrt(num / den) <= 1.5 * math.sqrt(ynum / den) + 1e-4


@pytest.mark.parametrize("n,Hq,Hkv,D,paged", [(2_000_003, 2, 1, 128, False), (4_194_304 + 17, 1, 1, 64, True)])
def test_multi_million_key_sequences(n, Hq, Hkv, D, paged):
    # far beyond the paper's 128K contexts: thousands of canonical chunks per row, token offsets past 2^31 bytes
    if _free_gb() < 6:
        pytest.skip("not enough free device memory")
    kw = dict(paged=True, page_size=64) if paged else {}
    w = make_decode_workload(1, Hq, Hkv, D, n, seed=5, device=DEV, **kw)
    for T in (math.inf, 16.0):
        b = run_gpu(w, T=T)
        compare(w, b, T=T, rows=[(0, Hq - 1)], check_estimate=True)
        assert same_bits(run_gpu(w, T=T, num_splits=3).out, b.out)
    del w
    torch.cuda.empty_cache()
