"""Seeded random shapes: head dimension, group size, stacking, lengths around every tile / chunk / estimator boundary,
paged or contiguous, depth, block tail and draft masks drawn together, each case checked against the oracle on
sampled rows and for split invariance.  The draw is fixed by the seed, so a failure names its case."""
import math
import random

import pytest
import torch

import paper_2609_33410_b200 as F
from paper_2609_33410_b200.workloads import make_decode_workload, make_draft_workload
from helpers import run_gpu, compare, oracle_block_means, same_bits

pytestmark = pytest.mark.gpu
DEV = "cuda"
LENGTHS = [0, 1, 15, 17, 63, 64, 65, 127, 128, 129, 191, 192, 193, 255, 256, 257, 1000, 2047, 5000, 9000]


def _case(rnd):
    D = rnd.choice([64, 128])
    G = rnd.choice([1, 2, 3, 4, 5, 8, 12, 16])
    Hkv = rnd.choice([1, 2, 3])
    stack = rnd.choice([1, 1, 1, 2, 3, 5, 7, 20])
    while stack * G > 300:
        stack //= 2
    nseq = rnd.choice([1, 2, 3])
    lens = [rnd.choice(LENGTHS) for _ in range(nseq)]
    if max(lens) == 0:
        lens[0] = 33
    T = rnd.choice([math.inf, 16.0, 12.0, 8.0])
    return dict(D=D, Hq=G * Hkv, Hkv=Hkv, stack=stack, lens=lens, paged=rnd.random() < 0.4,
                page_size=rnd.choice([16, 32, 64, 128]), T=T, tail=(not math.isinf(T)) and rnd.random() < 0.4,
                drafts=stack > 1 and rnd.random() < 0.5, tree=rnd.random() < 0.5, slack=rnd.choice([0, 5, 100]),
                splits=rnd.choice([1, 2, 5]))


@pytest.mark.parametrize("seed", range(6))
def test_random_shapes_match_the_oracle(seed):
    rnd = random.Random(4200 + seed)
    for i in range(8):
        c = _case(rnd)
        kw = dict(device=DEV, poison_padding=True)
        if c["paged"]:
            kw.update(paged=True, page_size=c["page_size"])
        draft = None
        if c["drafts"]:
            w, masks, m = make_draft_workload(len(c["lens"]), c["stack"], c["Hq"], c["Hkv"], c["D"],
                                              [max(n, 1) for n in c["lens"]], seed=seed * 100 + i, tree=c["tree"], **kw)
            draft = (masks, m)
        else:
            if not c["paged"]:
                kw.update(capacity=max(c["lens"]) + c["slack"])
            w = make_decode_workload(len(c["lens"]) * c["stack"], c["Hq"], c["Hkv"], c["D"], c["lens"],
                                     seed=seed * 100 + i, stack=c["stack"], **kw)
        vm = oracle_block_means(w) if c["tail"] else None
        rows = [(b, h) for b in sorted({0, w.batch // 2, w.batch - 1}) for h in sorted({0, c["Hq"] // 2, c["Hq"] - 1})]
        try:
            b = run_gpu(w, T=c["T"], v_block_mean=vm, draft=draft)
            compare(w, b, T=c["T"], rows=rows, check_estimate=True, v_block_mean=vm, draft=draft)
            s = run_gpu(w, T=c["T"], num_splits=c["splits"], v_block_mean=vm, draft=draft)
            assert same_bits(s.out, b.out) and same_bits(s.lse, b.lse), "split count changed a bit"
        except AssertionError as e:
            raise AssertionError(f"case {c}: {e}") from e


@pytest.mark.parametrize("seed", range(3))
def test_random_shared_prefix_cascades_match_the_oracle(seed):
    import numpy as np
    from oracle import fold_oracle as O
    from paper_2609_33410_b200.workloads import bf16_bits
    from helpers import cache_of
    rnd = random.Random(9100 + seed)
    for i in range(6):
        D = rnd.choice([64, 128]); G = rnd.choice([1, 2, 4, 8]); Hkv = rnd.choice([1, 2]); Hq = G * Hkv
        B = rnd.choice([2, 3, 9, 16, 17, 33, 40, 64, 70])                  # stacked rows on the prefix: 2 .. 560
        P = rnd.choice([1, 63, 64, 200, 1000, 1024, 3000, 9000])
        suffixes = [rnd.choice([0, 1, 5, 64, 65, 300, 700]) for _ in range(B)]
        T = rnd.choice([math.inf, 16.0, 10.0])
        tail = (not math.isinf(T)) and rnd.random() < 0.4
        case = dict(D=D, Hq=Hq, Hkv=Hkv, B=B, P=P, T=T, tail=tail)
        g = torch.Generator(device=DEV); g.manual_seed(seed * 100 + i)
        q = torch.randn(B, Hq, D, generator=g, device=DEV).to(torch.bfloat16)
        pre = make_decode_workload(B, Hq, Hkv, D, P, seed=seed * 300 + 3 * i + 1, device=DEV, stack=B, q=q)
        suf = make_decode_workload(B, Hq, Hkv, D, suffixes, seed=seed * 300 + 3 * i + 2, device=DEV, q=q, sink_gain=1.0)
        vmp, vms = (oracle_block_means(pre), oracle_block_means(suf)) if tail else (None, None)
        cp, cs = cache_of(pre, vmp), cache_of(suf, vms)
        bp, bs = F.alloc_buffers(q, cp, stack=B), F.alloc_buffers(q, cs)
        common = dict(z=bs.z, depth_T=T, out=bs.out, lse=bs.lse, row_status=bs.row_status)
        F.fold_decode_cascade([F.make_args(q, cp, stack=B, workspace=bp.workspace, **common),
                               F.make_args(q, cs, workspace=bs.workspace, **common)])
        torch.cuda.synchronize()
        assert bp.header().wait_timeouts == 0 and bs.header().wait_timeouts == 0, case
        out = bs.out.float().cpu().numpy().astype(np.float64)
        z = bs.z.cpu().numpy().astype(np.float64)
        lse = bs.lse.cpu().numpy()
        nbp = (P + 63) // 64
        num = den = 0.0
        for b in sorted({0, B // 2, B - 1}):
            for h in sorted({0, Hq - 1}):
                kvh, n_s = h // G, suffixes[b]
                K = np.concatenate([O.widen_bf16(bf16_bits(pre.logical_rows("k", 0, kvh))),
                                    O.widen_bf16(bf16_bits(suf.logical_rows("k", b, kvh)))])
                V = np.concatenate([O.widen_bf16(bf16_bits(pre.logical_rows("v", 0, kvh))),
                                    O.widen_bf16(bf16_bits(suf.logical_rows("v", b, kvh)))])
                s = O.scores(O.widen_bf16(bf16_bits(q[b, h])), K)
                assert abs(O.estimate_z(lambda j: s[j], len(s)) - z[b, h]) < 1e-3, case
                tl = None
                if tail:                                       # each level's own table, one after the other
                    mp = vmp.float().cpu().numpy().astype(np.float64)
                    ms = vms.float().cpu().numpy().astype(np.float64)
                    tl = (np.concatenate([mp[0, :nbp, kvh], ms[b, :(n_s + 63) // 64, kvh]]),
                          np.concatenate([np.arange(P) // 64, nbp + np.arange(n_s) // 64]))
                A, L = O.fold_partial(s, V, z[b, h], T, tail=tl)
                d = out[b, h] - A / L
                num += d @ d; den += (A / L) @ (A / L)
                assert abs(lse[b, h] - (z[b, h] + math.log2(L))) < 2e-3, case
        assert math.sqrt(num / max(den, 1e-300)) < 4e-3, case
