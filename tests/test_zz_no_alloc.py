"""fold_decode_static: the decode entry point for callers that are not allowed to allocate device
memory (a plugin under a host program that owns the device heap, a loop that must never reach the
synchronising allocator).  Its scratch is an array built into the library, shared by every call on
the device and never cleared between calls, so this test makes two different calls in a row and
checks each against the ordinary entry point, which works in a caller-allocated workspace.

Collected last on purpose: a run that stops at the first failure has then already run every other test."""
import math

import pytest
import torch

import paper_2609_33410_b200 as F
from paper_2609_33410_b200.workloads import make_decode_workload
from helpers import cache_of, run_gpu, same_bits

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _static_decode(w, T):
    """Through the C ABI with no workspace at all: out / lse / z / status are the only buffers passed."""
    cache = cache_of(w)
    B, Hq, D = w.q.shape
    out = torch.empty(B, Hq, D, dtype=torch.bfloat16, device=DEV)
    lse = torch.empty(B, Hq, dtype=torch.float32, device=DEV)
    z = torch.empty(B, Hq, dtype=torch.float32, device=DEV)
    st = torch.full((B, Hq), -1, dtype=torch.int32, device=DEV)
    args = F.make_args(w.q, cache, scale=w.scale, z=z, depth_T=T, out=out, lse=lse, row_status=st)
    assert args.workspace is None and args.workspace_bytes == 0
    F.fold_decode_static(args)
    torch.cuda.synchronize()
    return out, lse, z, st


def _agree(got, ref_bufs, w):
    # the same kernels on the same slot layout, only the scratch lives elsewhere: the same bits, not merely close values
    out, lse, z, st = got
    assert same_bits(out, ref_bufs.out) and same_bits(lse, ref_bufs.lse) and same_bits(z, ref_bufs.z)
    assert torch.equal(st, ref_bufs.row_status)


def test_two_static_calls_in_a_row_match_the_workspace_entry_point():
    # two shapes, so the second call finds the first call's slots and header in the shared array
    w1 = make_decode_workload(3, 8, 2, 128, [5000, 700, 0], seed=71, device=DEV, capacity=5000)
    w2 = make_decode_workload(2, 4, 4, 64, [300, 9000], seed=72, device=DEV, paged=True, page_size=32)
    ref1 = run_gpu(w1, T=16.0)
    ref2 = run_gpu(w2, T=math.inf)
    _agree(_static_decode(w1, 16.0), ref1, w1)
    _agree(_static_decode(w2, math.inf), ref2, w2)
    _agree(_static_decode(w1, 16.0), ref1, w1)          # and back: stale slots of the other shape are harmless


def test_static_calls_leave_device_memory_alone():
    # what the entry point is for: after a first call has looked the array up, further calls of either shape neither
    # allocate nor free -- the driver's free memory and torch's allocator counters stay where they were
    w1 = make_decode_workload(3, 8, 2, 128, [5000, 700, 0], seed=71, device=DEV, capacity=5000)
    w2 = make_decode_workload(2, 4, 4, 64, [300, 9000], seed=72, device=DEV, paged=True, page_size=32)
    calls = []
    for (w, T) in ((w1, 16.0), (w2, math.inf)):
        cache = cache_of(w)
        B, Hq, D = w.q.shape
        out = torch.empty(B, Hq, D, dtype=torch.bfloat16, device=DEV)
        lse = torch.empty(B, Hq, dtype=torch.float32, device=DEV)
        z = torch.empty(B, Hq, dtype=torch.float32, device=DEV)
        calls.append((F.make_args(w.q, cache, scale=w.scale, z=z, depth_T=T, out=out, lse=lse), (cache, out, lse, z)))
    for a, _ in calls:
        F.fold_decode_static(a)                          # warm: symbol lookup, kernels loaded
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    alloc0, reserved0 = torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
    for _ in range(5):
        for a, _ in calls:
            F.fold_decode_static(a)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0
    assert torch.cuda.memory_allocated() == alloc0 and torch.cuda.memory_reserved() == reserved0


def test_static_call_refuses_what_does_not_fit():
    w = make_decode_workload(1, 4, 2, 128, 300, seed=73, device=DEV)
    cache = cache_of(w)
    bufs = F.alloc_buffers(w.q, cache)
    args = F.make_args(w.q, cache, z=bufs.z, out=bufs.out, lse=bufs.lse)
    args.kv.max_seqlen = 1 << 28                         # would need far more than the built-in array
    assert F.fold_workspace_bytes(args) > F.STATIC_SCRATCH_BYTES
    assert F.lib().fold_decode_static(args, None) == F.FOLD_ETOOLARGE
    assert b"built-in" in F.lib().fold_status_string(F.FOLD_ETOOLARGE)
