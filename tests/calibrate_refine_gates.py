#!/usr/bin/env python
"""Regenerates the calibration tables behind the automatic refine gates of the two-plane key format and the E4M3
value planes (the paper gives no formula for either gate; the defaults are  tau_K = max(log2 n - 2, 4)  and
tau_V = max(log2 n + 1, 4)).  CPU only: it calls the float64 oracle and the seeded input generator, nothing else.

For seeded synthetic rows (the parity tests' generator: N(0,1) keys and values, a x8 sink, 1 % of the keys boosted
towards one query head) and each candidate gate  log2 n + offset  it prints
  * keys:   the relative l2 error of dense two-plane attention against exact attention on the BF16 inputs, and the
            fraction of keys whose plane B is read (after the OR over the group's rows);
  * values: the same error for attention over E4M3 value planes with exact BF16 keys, and the fraction of keys whose
            second value plane is read (per row);
next to the error of the emulated BF16 online-softmax kernel on the same rows (the yardstick a gate should stay under).

    python tests/calibrate_refine_gates.py            # about two minutes on 8 cores
"""
from __future__ import annotations

import math
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

from oracle import fold_oracle as O                                   # noqa: E402
from oracle import fold_planes_oracle as P                            # noqa: E402
from paper_2609_33410_b200.workloads import make_decode_workload, bf16_bits   # noqa: E402  (inputs only)

G = 4                     # query rows per kv head
OFFSETS_K = (None, -4, -2, 0, 2, 4, 7, math.inf)      # None: plane A only; inf: every key refined
OFFSETS_V = (None, -6, -4, -2, 0, 1, 2, math.inf)


def rows_of(n: int):
    w = make_decode_workload(2, 2 * G, 2, 128, [n, n], seed=5, device="cpu")
    for seq in range(2):
        for kvh in range(2):
            K = O.widen_bf16(bf16_bits(w.logical_rows("k", seq, kvh)))
            V = O.widen_bf16(bf16_bits(w.logical_rows("v", seq, kvh)))
            q = np.stack([O.widen_bf16(bf16_bits(w.q[seq, kvh * G + g])) for g in range(G)])
            yield w.scale, q, K, V


def key_gate_table(n: int):
    acc = {}
    for scale, q, K, V in rows_of(n):
        ka, kb, ke = P.quantize_rows(K)
        qa, qb, qe = P.quantize_rows(q)
        eta = qe.astype(np.float64) * (O.LOG2E * scale)
        dense = [O.dense_row(O.scores(q[g], K, scale), V) for g in range(G)]
        Z = np.array([d[1] for d in dense]) - 0.7          # a reference a little under the log-sum-exp, as the estimate is
        yard = [O.online_softmax_bf16(q[g], K, V, scale) - dense[g][0] for g in range(G)]
        for off in OFFSETS_K:
            tau = -1.0 if off is None else (math.inf if math.isinf(off) else math.log2(n) + off)
            A, L, info = P.fold_group_planes(ka, kb, ke, V, qa, qb, eta, Z, math.inf, tau)
            e = acc.setdefault(off, [0.0, 0.0, 0.0, 0.0, 0])
            for g in range(G):
                d = A[g] / L[g] - dense[g][0]
                e[0] += d @ d; e[1] += dense[g][0] @ dense[g][0]; e[3] += yard[g] @ yard[g]
            e[2] += float(info["refine"].mean()); e[4] += 1
    return {off: (math.sqrt(e[0] / e[1]), e[2] / e[4], math.sqrt(e[3] / e[1])) for off, e in acc.items()}


def value_gate_table(n: int):
    acc = {}
    for scale, q, K, V in rows_of(n):
        vk = int(math.ceil(math.log2(np.abs(V).max() / 448.0)))
        p1, p2 = P.quantize_values(V, vk)
        for g in range(G):
            s = O.scores(q[g], K, scale)
            o, lse = O.dense_row(s, V)
            p = np.exp2(s - lse)
            yard = O.online_softmax_bf16(q[g], K, V, scale) - o
            for off in OFFSETS_V:
                tau = None if off is None else (math.inf if math.isinf(off) else math.log2(n) + off)
                refined = np.zeros(len(s), bool) if tau is None else (s - lse >= -tau)
                Vq = P.widen_values(p1, p2, vk, refined)
                d = (p[:, None] * Vq).sum(0) - o
                e = acc.setdefault(off, [0.0, 0.0, 0.0, 0.0, 0])
                e[0] += d @ d; e[1] += o @ o; e[2] += float(refined.mean()); e[3] += yard @ yard; e[4] += 1
    return {off: (math.sqrt(e[0] / e[1]), e[2] / e[4], math.sqrt(e[3] / e[1])) for off, e in acc.items()}


def label(off):
    return "first plane only" if off is None else ("every key" if math.isinf(off) else f"log2 n {off:+d}")


def main():
    for n in (4096, 32768):
        print(f"\n== keys, n = {n}: gate tau_K | rel l2 vs exact attention | plane-B rows read | BF16 online-softmax yardstick")
        for off, (err, frac, yard) in key_gate_table(n).items():
            print(f"   {label(off):>18} | {err:.2e} | {frac:.3f} | {yard:.2e}")
        print(f"== values, n = {n}: gate tau_V | rel l2 vs exact attention | second-plane rows read (per row) | yardstick")
        for off, (err, frac, yard) in value_gate_table(n).items():
            print(f"   {label(off):>18} | {err:.2e} | {frac:.3f} | {yard:.2e}")


if __name__ == "__main__":
    main()
