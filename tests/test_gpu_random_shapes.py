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
