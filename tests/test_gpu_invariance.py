"""Bit-identity of the CUDA path under everything that only regroups the same sum
(Prop. 1(i) made exact by canonical chunks + the integer-grid partial add), and the
shared-prefix cascade."""
import math

import numpy as np
import pytest
import torch

import paper_2609_33410_b200 as F
from oracle import fold_oracle as O
from paper_2609_33410_b200.workloads import make_decode_workload, DecodeWorkload
from helpers import run_gpu, compare, cache_of, same_bits, row_inputs

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.mark.parametrize("T", [math.inf, 16.0])
def test_split_count_never_changes_a_bit(T):
    w = make_decode_workload(2, 8, 2, 128, [40000, 9000], seed=41, device=DEV)
    ref = run_gpu(w, T=T, num_splits=1)
    o, l = ref.out.clone(), ref.lse.clone()
    for s in (2, 3, 4, 8, 16, 32, 0):
        b = run_gpu(w, T=T, num_splits=s)
        assert same_bits(b.out, o) and same_bits(b.lse, l), s


@pytest.mark.parametrize("T", [math.inf, 16.0])
def test_alone_equals_in_batch(T):
    w = make_decode_workload(4, 8, 2, 128, [5000, 333, 12000, 64], seed=43, device=DEV)
    full = run_gpu(w, T=T)
    for b in range(4):
        n = int(w.seqlens[b])
        solo = DecodeWorkload(w.q[b:b + 1].contiguous(), w.k[b:b + 1, :max(n, 1)].contiguous(),
                              w.v[b:b + 1, :max(n, 1)].contiguous(), w.seqlens[b:b + 1].contiguous(), n,
                              w.num_q_heads, w.num_kv_heads, w.head_dim, scale=w.scale)
        r = run_gpu(solo, T=T)
        assert same_bits(r.out[0], full.out[b]) and same_bits(r.lse[0], full.lse[b]), b


@pytest.mark.parametrize("T", [math.inf, 16.0])
@pytest.mark.parametrize("page_size", [16, 64])
def test_paged_equals_contiguous(T, page_size):
    w = make_decode_workload(2, 8, 2, 128, [3000, 10000], seed=47, device=DEV)
    ref = run_gpu(w, T=T)
    # scatter the same logical rows into a randomly permuted page pool
    g = torch.Generator(device=DEV); g.manual_seed(5)
    lens = [3000, 10000]
    npg = [(n + page_size - 1) // page_size for n in lens]
    perm = torch.randperm(sum(npg) + 3, generator=g, device=DEV)
    kp = torch.full((sum(npg) + 3, page_size, 2, 128), float("nan"), dtype=torch.bfloat16, device=DEV)
    vp = torch.full_like(kp, float("nan"))
    table = torch.zeros(2, max(npg), dtype=torch.int32, device=DEV)
    cur = 0
    for s, n in enumerate(lens):
        ids = perm[cur:cur + npg[s]]; cur += npg[s]
        table[s, :npg[s]] = ids.to(torch.int32)
        pad = npg[s] * page_size - n
        kk = torch.cat([w.k[s, :n], torch.full((pad, 2, 128), float("nan"), dtype=torch.bfloat16, device=DEV)])
        vv = torch.cat([w.v[s, :n], torch.full((pad, 2, 128), float("nan"), dtype=torch.bfloat16, device=DEV)])
        kp[ids] = kk.view(npg[s], page_size, 2, 128); vp[ids] = vv.view(npg[s], page_size, 2, 128)
    wp = DecodeWorkload(w.q, kp, vp, w.seqlens, w.max_seqlen, 8, 2, 128, 1, table, page_size, w.scale)
    r = run_gpu(wp, T=T)
    assert same_bits(r.out, ref.out) and same_bits(r.lse, ref.lse) and same_bits(r.z, ref.z)


def _split_then_merge(w, T, z, order=None, perm_seed=None):
    cache = cache_of(w)
    bufs = F.alloc_buffers(w.q, cache, w.stack)
    bufs.z.copy_(z)
    args = F.make_args(w.q, cache, scale=w.scale, z_mode=F.Z_GIVEN, z=bufs.z, depth_T=T, stack=w.stack,
                       workspace=bufs.workspace)
    part = F.fold_decode_split(args)
    torch.cuda.synchronize()
    if perm_seed is not None:                     # permute the valid slots of every (sequence, kv head)
        sv = F.slots_view(part, bufs.workspace)
        g = torch.Generator(device=DEV); g.manual_seed(perm_seed)
        for s in range(part.num_seqs):
            c = F.fold_num_chunks(int(w.seqlens[s]))
            for h in range(part.num_kv_heads):
                sv[s, h, :c] = sv[s, h, :c][torch.randperm(c, generator=g, device=DEV)]
    return part, bufs


@pytest.mark.parametrize("T", [math.inf, 16.0])
def test_slot_order_never_changes_a_bit(T):
    w = make_decode_workload(2, 8, 2, 128, [30000, 7000], seed=53, device=DEV)
    z = run_gpu(w, T=T).z.clone()
    part, bufs = _split_then_merge(w, T, z)
    F.fold_cascade_merge([part], bufs.out, bufs.lse, bufs.row_status)
    torch.cuda.synchronize()
    o, l = bufs.out.clone(), bufs.lse.clone()
    ref = run_gpu(w, T=T, z_mode=F.Z_GIVEN, z=z)
    assert same_bits(o, ref.out) and same_bits(l, ref.lse)
    for seed in (1, 2, 3):
        part2, bufs2 = _split_then_merge(w, T, z, perm_seed=seed)
        F.fold_cascade_merge([part2], bufs2.out, bufs2.lse, bufs2.row_status)
        torch.cuda.synchronize()
        assert same_bits(bufs2.out, o) and same_bits(bufs2.lse, l)


def _cascade(B, Hq, Hkv, D, n_prefix, suffix_lens, seed, T):
    """Requests share one prefix and own private suffixes.  Returns (out, lse, z, flat workload)."""
    g = torch.Generator(device=DEV); g.manual_seed(seed)
    q = torch.randn(B, Hq, D, generator=g, device=DEV).to(torch.bfloat16)
    pre = make_decode_workload(B, Hq, Hkv, D, n_prefix, seed=seed + 1, device=DEV, stack=B, q=q)
    suf = make_decode_workload(B, Hq, Hkv, D, suffix_lens, seed=seed + 2, device=DEV, q=q, sink_gain=1.0)
    cp, cs = cache_of(pre), cache_of(suf)
    bp, bs = F.alloc_buffers(q, cp, stack=B), F.alloc_buffers(q, cs)
    z = bs.z
    ap = F.make_args(q, cp, z_mode=F.Z_GIVEN, z=z, depth_T=T, stack=B, workspace=bp.workspace)
    as_ = F.make_args(q, cs, z_mode=F.Z_GIVEN, z=z, depth_T=T, workspace=bs.workspace)
    F.fold_estimate_z([ap, as_])                  # one estimate over prefix ++ suffix, used by both levels
    pp, ps = F.fold_decode_split(ap), F.fold_decode_split(as_)
    F.fold_cascade_merge([pp, ps], bs.out, bs.lse, bs.row_status)
    torch.cuda.synchronize()
    out, lse = bs.out.clone(), bs.lse.clone()
    F.fold_cascade_merge([ps, pp], bp.out, bp.lse, bp.row_status)       # level order swapped
    torch.cuda.synchronize()
    assert same_bits(bp.out, out) and same_bits(bp.lse, lse)
    # the same requests as a flat batch over the concatenated sequences
    lens = [n_prefix + s for s in suffix_lens]
    cap = max(lens)
    kf = torch.zeros(B, cap, Hkv, D, dtype=torch.bfloat16, device=DEV); vf = torch.zeros_like(kf)
    for b in range(B):
        kf[b, :n_prefix] = pre.k[0, :n_prefix]; vf[b, :n_prefix] = pre.v[0, :n_prefix]
        kf[b, n_prefix:lens[b]] = suf.k[b, :suffix_lens[b]]; vf[b, n_prefix:lens[b]] = suf.v[b, :suffix_lens[b]]
    flat = DecodeWorkload(q, kf, vf, torch.tensor(lens, dtype=torch.int32, device=DEV), cap, Hq, Hkv, D,
                          scale=1.0 / math.sqrt(D))
    return bs, flat


@pytest.mark.parametrize("T", [math.inf, 16.0])
@pytest.mark.parametrize("B", [4, 20])
def test_shared_prefix_cascade_matches_oracle_and_flat_decode(T, B):
    Hq, Hkv, D = 8, 2, 128                        # B requests x group 4 = 16 or 80 stacked rows on the prefix
    suffixes = ([500, 1, 0, 257] * 5)[:B]
    bs, flat = _cascade(B, Hq, Hkv, D, 3000, suffixes, seed=61, T=T)
    # oracle on the concatenated sequence at the cascade's references
    rows = None if B == 4 else [(b, h) for b in (0, 1, 2, 7, 19) for h in (0, 5)]
    r = compare(flat, bs, T=T, check_estimate=True, rows=rows)
    # flat decode of the same requests under the same references: same values within tolerance
    fb = run_gpu(flat, T=T, z_mode=F.Z_GIVEN, z=bs.z.clone())
    assert same_bits(fb.z, bs.z)
    a, b = fb.out.float(), bs.out.float()
    assert (a - b).norm() / a.norm() < 3e-3
    assert torch.allclose(fb.lse, bs.lse, atol=1e-4)
    # and the flat estimate equals the cascade's two-level estimate bit for bit
    fe = run_gpu(flat, T=T)
    assert same_bits(fe.z, bs.z)


@pytest.mark.parametrize("T", [math.inf, 16.0])
def test_graph_replay_equals_eager_call(T):
    # the whole call (header memset, estimate, scan, partial add) is capturable: nothing allocates or synchronises
    w = make_decode_workload(2, 8, 2, 128, [20000, 700], seed=71, device=DEV)
    eager = run_gpu(w, T=T)
    o, l, z = eager.out.clone(), eager.lse.clone(), eager.z.clone()
    cache = cache_of(w)
    bufs = F.alloc_buffers(w.q, cache, w.stack)
    args = F.make_args(w.q, cache, scale=w.scale, z=bufs.z, depth_T=T, workspace=bufs.workspace, out=bufs.out,
                       lse=bufs.lse, row_status=bufs.row_status)
    F.fold_decode(args, torch.cuda.current_stream())          # first call outside capture: one-time set-up
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        F.fold_decode(args, torch.cuda.current_stream())
    for _ in range(2):
        bufs.out.zero_(); bufs.lse.zero_(); bufs.z.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert same_bits(bufs.out, o) and same_bits(bufs.lse, l) and same_bits(bufs.z, z)
        assert bufs.header().wait_timeouts == 0


@pytest.mark.parametrize("with_side", [False, True])
def test_cascade_call_is_graph_capturable_with_its_side_stream(with_side):
    # with a side stream and two events of the CALLER's the cascade forks its first level onto that stream and joins it
    # back: still one capturable call, and the same bits as on one stream
    B, Hq, Hkv, D = 6, 8, 2, 128
    suffixes = [300, 1, 0, 257, 64, 65]
    g = torch.Generator(device=DEV); g.manual_seed(97)
    q = torch.randn(B, Hq, D, generator=g, device=DEV).to(torch.bfloat16)
    pre = make_decode_workload(B, Hq, Hkv, D, 2000, seed=98, device=DEV, stack=B, q=q)
    suf = make_decode_workload(B, Hq, Hkv, D, suffixes, seed=99, device=DEV, q=q, sink_gain=1.0)
    cp, cs = cache_of(pre), cache_of(suf)
    bp, bs = F.alloc_buffers(q, cp, stack=B), F.alloc_buffers(q, cs)
    common = dict(z=bs.z, depth_T=16.0, out=bs.out, lse=bs.lse, row_status=bs.row_status)
    one = [F.make_args(q, cp, stack=B, workspace=bp.workspace, **common), F.make_args(q, cs, workspace=bs.workspace, **common)]
    F.fold_decode_cascade(one, torch.cuda.current_stream())
    torch.cuda.synchronize()
    o, l = bs.out.clone(), bs.lse.clone()
    side = F.CascadeSide(DEV) if with_side else None
    levels = [F.make_args(q, cp, stack=B, workspace=bp.workspace, side=side, **common), F.make_args(q, cs, workspace=bs.workspace, **common)]
    bs.out.zero_(); bs.lse.zero_()
    F.fold_decode_cascade(levels, torch.cuda.current_stream())
    torch.cuda.synchronize()
    assert same_bits(bs.out, o) and same_bits(bs.lse, l)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        F.fold_decode_cascade(levels, torch.cuda.current_stream())
    for _ in range(2):
        bs.out.zero_(); bs.lse.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert same_bits(bs.out, o) and same_bits(bs.lse, l)
        assert bp.header().wait_timeouts == 0 and bs.header().wait_timeouts == 0


@pytest.mark.parametrize("flags", [0, F.INPUTS_SETTLED])
def test_inputs_written_on_the_stream_just_before_a_call_are_seen(flags):
    # A decode loop appends the newest token's K / V rows, projects q and bumps seqlens with kernels on the stream right
    # before the call, with no host synchronisation.  Without FOLD_INPUTS_SETTLED the call's first kernel is launched in
    # plain stream order and must see all of it.  (With the flag the caller promises the inputs were complete earlier; the
    # writers here are ordinary kernels that end before the call's first kernel may run, so the bits agree there too.)
    w = make_decode_workload(3, 8, 2, 128, [5000, 777, 8200], seed=73, device=DEV, capacity=8300)
    cache = cache_of(w)
    bufs = F.alloc_buffers(w.q, cache)
    g = torch.Generator(device=DEV); g.manual_seed(74)
    new_k = torch.randn(3, 2, 128, generator=g, device=DEV).to(torch.bfloat16) * 3
    new_v = torch.randn(3, 2, 128, generator=g, device=DEV).to(torch.bfloat16)
    new_q = torch.randn(w.q.shape, generator=g, device=DEV).to(torch.bfloat16)
    lens = w.seqlens.clone()
    idx = torch.arange(3, device=DEV)
    F.decode(w.q, cache, bufs, depth_T=16.0)                     # a step before: the stream is busy with the library's kernels
    # the append + projection of the next step, then the call, all enqueued without a host synchronisation
    w.k[idx, lens.long()] = new_k
    w.v[idx, lens.long()] = new_v
    w.q.copy_(new_q)
    w.seqlens.add_(1)
    F.decode(w.q, cache, bufs, depth_T=16.0, flags=flags)
    torch.cuda.synchronize()
    got = (bufs.out.clone(), bufs.lse.clone(), bufs.z.clone())
    ref = F.alloc_buffers(w.q, cache)                            # the same state decoded after a full synchronisation
    F.decode(w.q, cache, ref, depth_T=16.0)
    torch.cuda.synchronize()
    assert same_bits(got[0], ref.out) and same_bits(got[1], ref.lse) and same_bits(got[2], ref.z)


@pytest.mark.parametrize("planes", [False, True])
def test_back_to_back_calls_that_share_z_and_workspace_do_not_disturb_each_other(planes):
    # The reference kernel of a call may start while the partial add of the call before it is still running (programmatic
    # dependent launch); it must not write z, the header or the workspace before that add is done.  Two different
    # workloads of one shape alternate on ONE z buffer and ONE workspace, without a host synchronisation between calls.
    wa = make_decode_workload(4, 8, 2, 128, [9000, 700, 4000, 33], seed=71, device=DEV)
    wb = make_decode_workload(4, 8, 2, 128, [8000, 9000, 100, 5000], seed=72, device=DEV, capacity=wa.k.shape[1])
    ca, cb = cache_of(wa), cache_of(wb)
    if planes:
        F.fold_quantize_keys(ca); F.fold_quantize_keys(cb)
    ref = []
    for w, c in ((wa, ca), (wb, cb)):
        b = F.alloc_buffers(w.q, c)
        F.decode(w.q, c, b, depth_T=16.0)
        torch.cuda.synchronize()
        ref.append((b.out.clone(), b.lse.clone()))
    shared = F.alloc_buffers(wa.q, ca)
    outs = [torch.empty_like(ref[0][0]) for _ in range(2)]
    lses = [torch.empty_like(ref[0][1]) for _ in range(2)]
    args = [F.make_args(w.q, c, depth_T=16.0, z=shared.z, workspace=shared.workspace, out=outs[i], lse=lses[i],
                        row_status=shared.row_status) for i, (w, c) in enumerate(((wa, ca), (wb, cb)))]
    for _ in range(25):
        F.fold_decode(args[0])
        F.fold_decode(args[1])
    torch.cuda.synchronize()
    for i in range(2):
        assert same_bits(outs[i], ref[i][0]) and same_bits(lses[i], ref[i][1]), i


@pytest.mark.parametrize("paged", [False, True])
def test_the_live_hint_never_changes_a_bit(paged):
    # fold_args.live_hint picks how the depth-gated row-block scan splits its on-chip ring between key and value tiles
    # (two and four stages, three and three, four and two): scheduling only, so every hint must give the same bits
    w = make_decode_workload(3, 8, 2, 128, [9000, 2500, 700], seed=61, device=DEV, paged=paged, page_size=32)
    cache = cache_of(w)
    ref = run_gpu(w, T=14.0)
    for hint in (1.0, 0.9, 0.5, 0.1, 1e-6, -3.0, float("nan"), 7.0):
        bufs = F.alloc_buffers(w.q, cache, w.stack)
        F.decode(w.q, cache, bufs, depth_T=14.0, scale=w.scale, live_hint=hint)
        torch.cuda.synchronize()
        assert bufs.header().wait_timeouts == 0
        assert same_bits(bufs.out, ref.out) and same_bits(bufs.lse, ref.lse) and same_bits(bufs.z, ref.z), hint
