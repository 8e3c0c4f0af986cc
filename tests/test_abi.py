"""The C-ABI library without a GPU: it builds, loads, exports every symbol the header
declares, the Python structs mirror the C ones byte for byte, and host-side argument
checks answer with status codes before any CUDA call is made."""
import ctypes as C
import os
import re
import subprocess
import sys
import tempfile

import pytest
import torch

import paper_2609_33410_b200 as F
from paper_2609_33410_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "fold.h")


def declared_functions():
    src = open(HEADER).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(fold_[a-z_0-9]+)\s*\(", src)))


def test_library_exports_every_declared_symbol():
    names = declared_functions()
    assert set(names) == set(binding.EXPORTS), (names, binding.EXPORTS)
    L = F.lib()
    for n in names:
        assert getattr(L, n) is not None
    assert L.fold_version() >= 100
    assert L.fold_status_string(F.FOLD_EWORKSPACE) == b"workspace too small"


def test_python_structs_mirror_the_header():
    prog = r"""
#include <stdio.h>
#include <stddef.h>
#include "fold.h"
int main(void) {
  printf("%zu %zu %zu %zu\n", sizeof(fold_kv), sizeof(fold_args), sizeof(fold_partials), sizeof(fold_ws_header));
  printf("%zu %zu %zu %zu %zu\n", offsetof(fold_kv, seqlens), offsetof(fold_kv, max_seqlen), offsetof(fold_args, kv),
         offsetof(fold_args, depth_T), offsetof(fold_args, row_status));
  printf("%zu %zu %zu\n", offsetof(fold_partials, rows), offsetof(fold_partials, slot_stride),
         offsetof(fold_ws_header, v_rows_total));
  printf("%zu %zu %zu %zu\n", offsetof(fold_args, flags), offsetof(fold_args, side_stream), offsetof(fold_args, side_join_event),
         offsetof(fold_args, live_hint));
  return 0;
}
"""
    with tempfile.TemporaryDirectory() as d:
        src = os.path.join(d, "t.c"); exe = os.path.join(d, "t")
        open(src, "w").write(prog)
        subprocess.run(["gcc", "-std=c99", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"), src, "-o", exe],
                       check=True)
        out = subprocess.run([exe], check=True, capture_output=True, text=True).stdout.split()
    got = [int(x) for x in out]
    want = [C.sizeof(F.FoldKV), C.sizeof(F.FoldArgs), C.sizeof(F.FoldPartials), C.sizeof(F.FoldWsHeader),
            F.FoldKV.seqlens.offset, F.FoldKV.max_seqlen.offset, F.FoldArgs.kv.offset, F.FoldArgs.depth_T.offset,
            F.FoldArgs.row_status.offset, F.FoldPartials.rows.offset, F.FoldPartials.slot_stride.offset,
            F.FoldWsHeader.v_rows_total.offset, F.FoldArgs.flags.offset, F.FoldArgs.side_stream.offset,
            F.FoldArgs.side_join_event.offset, F.FoldArgs.live_hint.offset]
    assert got == want


def test_chunk_rule_depends_on_length_only():
    assert F.fold_chunk_keys(1) == 256 and F.fold_chunk_keys(8192) == 256 and F.fold_chunk_keys(8193) == 1024
    assert [F.fold_num_chunks(n) for n in (0, 1, 256, 257, 8192, 8193, 131072)] == [0, 1, 1, 2, 32, 9, 128]


def _cpu_args(B=2, Hq=8, Hkv=2, D=128, n=1000, **kw):
    q = torch.zeros(B, Hq, D, dtype=torch.bfloat16)
    k = torch.zeros(B, n, Hkv, D, dtype=torch.bfloat16)
    v = torch.zeros_like(k)
    lens = torch.full((B,), n, dtype=torch.int32)
    z = torch.zeros(B, Hq)
    out = torch.zeros(B, Hq, D, dtype=torch.bfloat16)
    cache = F.KVCache(k, v, lens, n)
    a = F.make_args(q, cache, z=z, out=out, **kw)
    keep = (q, k, v, lens, z, out)
    return a, keep


def test_workspace_size_formula():
    a, _ = _cpu_args()
    G, R = 4, 4
    slots = (1000 + 255) // 256
    assert F.fold_workspace_bytes(a) == 256 + 2 * 2 * slots * (R * 128 + 4) * 4
    a, _ = _cpu_args(n=40000)
    assert F.fold_workspace_bytes(a) == 256 + 2 * 2 * 40 * (R * 128 + 4) * 4
    a.head_dim = 80
    assert F.fold_workspace_bytes(a) == 0


def test_host_checks_answer_before_any_cuda_call():
    L = F.lib()
    a, keep = _cpu_args()
    ws = torch.zeros(F.fold_workspace_bytes(a) + 256, dtype=torch.uint8)
    off = (-ws.data_ptr()) % 256
    a.workspace = ws.data_ptr() + off
    a.workspace_bytes = ws.numel() - 256
    for field, value, want in [("depth_T", -0.5, F.FOLD_EINVAL), ("depth_T", float("nan"), F.FOLD_EINVAL),
                               ("head_dim", 96, F.FOLD_EUNSUPPORTED), ("softmax_scale", 0.0, F.FOLD_EINVAL),
                               ("z_mode", 7, F.FOLD_EINVAL), ("num_splits", -1, F.FOLD_EINVAL),
                               ("workspace_bytes", 100, F.FOLD_EWORKSPACE), ("stack", 3, F.FOLD_EINVAL),
                               ("num_kv_heads", 3, F.FOLD_EINVAL), ("out", None, F.FOLD_EINVAL)]:
        old = getattr(a, field)
        setattr(a, field, value)
        assert L.fold_decode(a, None) == want, field
        setattr(a, field, old)
    a.kv.page_table = keep[3].data_ptr(); a.kv.page_size = 24; a.kv.num_pages = 4; a.kv.max_pages_per_seq = 100
    assert L.fold_decode(a, None) == F.FOLD_EUNSUPPORTED          # page size not a power of two
    a.kv.page_size = 64; a.kv.max_pages_per_seq = 2
    assert L.fold_decode(a, None) == F.FOLD_EINVAL                # table cannot hold max_seqlen
    assert L.fold_cascade_merge(None, 1, None, None, None, None) == F.FOLD_EINVAL
    assert L.fold_estimate_z(None, 0, None) == F.FOLD_EINVAL
    a.kv.page_table = None
    a.batch, a.kv.num_seqs = 70000, 70000                         # requests index a grid dimension: at most 65535
    assert L.fold_decode(a, None) == F.FOLD_EUNSUPPORTED


def test_broadcast_strides_are_refused():
    # an axis with more than one entry must have a stride that spans a row: a zero (broadcast) stride would let the
    # tensor maps and the plain loads disagree about where the rows lie
    L = F.lib()
    a, keep = _cpu_args()
    ws = torch.zeros(F.fold_workspace_bytes(a) + 256, dtype=torch.uint8)
    a.workspace = ws.data_ptr() + (-ws.data_ptr()) % 256
    a.workspace_bytes = ws.numel() - 256
    for field in ("stride_head", "stride_seq"):
        old = getattr(a.kv, field)
        setattr(a.kv, field, 0)
        assert L.fold_decode(a, None) == F.FOLD_EINVAL, field
        setattr(a.kv, field, old)
    a1, keep1 = _cpu_args(B=1, Hq=4, Hkv=1)                  # one sequence, one kv head: their strides carry no information
    a1.kv.stride_head = 0; a1.kv.stride_seq = 0
    a1.depth_T = -1.0                                        # (a later check must be the one that answers)
    assert L.fold_decode(a1, None) == F.FOLD_EINVAL


def test_new_argument_fields_default_to_plain_behaviour():
    a, _ = _cpu_args()
    assert a.flags == 0 and not a.side_stream and not a.side_fork_event and not a.side_join_event and a.live_hint == 0.0
    b, _ = _cpu_args(flags=F.INPUTS_SETTLED)
    assert b.flags == 1


def test_host_checks_of_draft_masks_and_block_means():
    L = F.lib()
    a, keep = _cpu_args()
    ws = torch.zeros(F.fold_workspace_bytes(a) + 256, dtype=torch.uint8)
    a.workspace = ws.data_ptr() + ((-ws.data_ptr()) % 256)
    a.workspace_bytes = ws.numel() - 256
    masks = torch.ones(64, dtype=torch.int32)
    for length, ptr, want in [(33, masks.data_ptr(), F.FOLD_EINVAL), (-1, masks.data_ptr(), F.FOLD_EINVAL),
                              (4, None, F.FOLD_EINVAL), (4, masks.data_ptr() + 2, F.FOLD_EINVAL)]:
        a.draft_len, a.draft_mask = length, ptr
        assert L.fold_decode(a, None) == want, (length, ptr)
    a.draft_len, a.draft_mask = 0, None
    means = torch.zeros(4096, dtype=torch.bfloat16)
    a.kv.v_block_mean = means.data_ptr() + 2                        # rows must start on 16 bytes
    a.kv.mean_stride_seq, a.kv.mean_stride_block, a.kv.mean_stride_head = 1024, 256, 128
    assert L.fold_decode(a, None) == F.FOLD_EINVAL
    a.kv.v_block_mean = means.data_ptr() + ((-means.data_ptr()) % 16)
    a.kv.mean_stride_block = 100                                    # not a multiple of 8, shorter than a row
    assert L.fold_decode(a, None) == F.FOLD_EINVAL
    kv = F.FoldKV()
    assert L.fold_block_means(None, 2, 128, None) == F.FOLD_EINVAL
    assert L.fold_block_means(kv, 2, 96, None) == F.FOLD_EUNSUPPORTED
    assert L.fold_block_means(kv, 2, 128, None) == F.FOLD_EINVAL    # no table to fill


@pytest.mark.skipif(torch.cuda.is_available(), reason="only meaningful without a device")
def test_no_device_means_a_loud_error_not_a_fallback():
    a, keep = _cpu_args()
    ws = torch.zeros(F.fold_workspace_bytes(a) + 256, dtype=torch.uint8)
    a.workspace = ws.data_ptr() + ((-ws.data_ptr()) % 256)
    a.workspace_bytes = ws.numel() - 256
    with pytest.raises(F.FoldError) as e:
        F.fold_decode(a, stream=0)
    assert e.value.status == F.FOLD_ECUDA


def test_host_checks_of_two_plane_keys():
    L = F.lib()
    a, keep = _cpu_args()
    plain = F.fold_workspace_bytes(a)
    k = keep[1]
    pa, pb = torch.zeros(k.shape, dtype=torch.int8), torch.zeros(k.shape, dtype=torch.int8)
    sc = torch.zeros(k.shape[0], k.shape[2], 1024, dtype=torch.bfloat16)
    a.kv.k_plane_a, a.kv.k_plane_b, a.kv.k_scale = pa.data_ptr(), pb.data_ptr(), sc.data_ptr()
    a.kv.plane_stride_seq, a.kv.plane_stride_tok, a.kv.plane_stride_head = pa.stride(0), pa.stride(1), pa.stride(2)
    a.kv.scale_stride_seq, a.kv.scale_stride_head = sc.stride(0), sc.stride(1)
    # the workspace also holds the split query rows: [row][2][D] codes and one scale per row, each part 256-aligned
    assert F.fold_workspace_bytes(a) == (plain + 255) // 256 * 256 + 2 * 8 * 2 * 128 + 256
    ws = torch.zeros(F.fold_workspace_bytes(a) + 256, dtype=torch.uint8)
    a.workspace = ws.data_ptr() + ((-ws.data_ptr()) % 256)
    a.workspace_bytes = plain                                      # enough for BF16 keys, not for the planes
    assert L.fold_decode(a, None) == F.FOLD_EWORKSPACE
    a.workspace_bytes = ws.numel() - 256
    for field, value, want in [("k_plane_b", None, F.FOLD_EINVAL), ("k_scale", None, F.FOLD_EINVAL),
                               ("k_plane_a", pa.data_ptr() + 4, F.FOLD_EINVAL), ("plane_stride_tok", 100, F.FOLD_EINVAL),
                               ("plane_stride_head", 72, F.FOLD_EINVAL), ("scale_stride_head", 1001, F.FOLD_EINVAL)]:
        old = getattr(a.kv, field)
        setattr(a.kv, field, value)
        assert L.fold_decode(a, None) == want, field
        setattr(a.kv, field, old)
    a.refine_tau = float("nan")
    assert L.fold_decode(a, None) == F.FOLD_EINVAL
    a.refine_tau = 0.0
    for field, value in [("z_mode", F.Z_EXACT_MAX), ("stack", 2)]:
        old = getattr(a, field)
        setattr(a, field, value)
        if field == "stack":                                        # 2 requests x group 12 on one sequence: 24 rows are two
            a.num_q_heads, a.num_kv_heads = 12, 1                   # 16-row blocks, and draft rows must stay within one
            a.kv.num_seqs = 1
            masks = torch.ones(2, dtype=torch.int32)
            a.draft_mask, a.draft_len = masks.data_ptr(), 2
        assert L.fold_decode(a, None) == F.FOLD_EUNSUPPORTED, field
        setattr(a, field, old)
        a.num_q_heads, a.num_kv_heads = 8, 2; a.kv.num_seqs = 2
        a.draft_mask, a.draft_len = None, 0
    args2 = (F.FoldArgs * 2)(a, a)
    args2[1].kv.k_plane_a = None
    ptrs = (C.POINTER(F.FoldArgs) * 2)(C.pointer(args2[0]), C.pointer(args2[1]))
    assert L.fold_decode_cascade(ptrs, 2, None) == F.FOLD_EUNSUPPORTED     # a cascade keeps to one key format
    assert L.fold_estimate_z(ptrs, 2, None) == F.FOLD_EUNSUPPORTED
    assert L.fold_quantize_keys(None, 2, 128, None, None) == F.FOLD_EINVAL
    kv = F.FoldKV()
    assert L.fold_quantize_keys(kv, 2, 96, None, None) == F.FOLD_EUNSUPPORTED
    assert L.fold_quantize_keys(kv, 2, 128, None, None) == F.FOLD_EINVAL  # nothing to read or write


def test_host_checks_of_e4m3_value_planes():
    L = F.lib()
    a, keep = _cpu_args()
    k = keep[1]
    pa, pb = torch.zeros(k.shape, dtype=torch.int8), torch.zeros(k.shape, dtype=torch.int8)
    sc = torch.zeros(k.shape[0], k.shape[2], 1024, dtype=torch.bfloat16)
    v1, v2 = torch.zeros(k.shape, dtype=torch.uint8), torch.zeros(k.shape, dtype=torch.uint8)
    a.kv.v_plane_1, a.kv.v_plane_2 = v1.data_ptr(), v2.data_ptr()
    ws = torch.zeros(1 << 20, dtype=torch.uint8)
    a.workspace = ws.data_ptr() + ((-ws.data_ptr()) % 256)
    a.workspace_bytes = ws.numel() - 256
    assert L.fold_decode(a, None) == F.FOLD_EUNSUPPORTED             # value planes without the two-plane keys
    a.kv.k_plane_a, a.kv.k_plane_b, a.kv.k_scale = pa.data_ptr(), pb.data_ptr(), sc.data_ptr()
    a.kv.plane_stride_seq, a.kv.plane_stride_tok, a.kv.plane_stride_head = pa.stride(0), pa.stride(1), pa.stride(2)
    a.kv.scale_stride_seq, a.kv.scale_stride_head = sc.stride(0), sc.stride(1)
    for field, value, want in [("v_plane_2", None, F.FOLD_EINVAL), ("v_plane_1", v1.data_ptr() + 8, F.FOLD_EINVAL),
                               ("v_scale_log2", 500, F.FOLD_EINVAL)]:
        old = getattr(a.kv, field)
        setattr(a.kv, field, value)
        assert L.fold_decode(a, None) == want, field
        setattr(a.kv, field, old)
    a.refine_tau_v = float("nan")
    assert L.fold_decode(a, None) == F.FOLD_EINVAL
    a.refine_tau_v = 0.0
    # the format's cut model (the sequences' mean value rows): host checks of its builder
    assert L.fold_running_means(None, 2, 128, None) == F.FOLD_EINVAL
    assert L.fold_running_means(a.kv, 2, 96, None) == F.FOLD_EUNSUPPORTED
    assert L.fold_running_means(a.kv, 2, 128, None) == F.FOLD_EINVAL           # no table
    vm = torch.zeros(k.shape[0], 1, k.shape[2], k.shape[3], dtype=torch.bfloat16)
    a.kv.v_block_mean = vm.data_ptr() + 2
    a.kv.mean_stride_seq, a.kv.mean_stride_block, a.kv.mean_stride_head = vm.stride(0), vm.stride(1), vm.stride(2)
    assert L.fold_running_means(a.kv, 2, 128, None) == F.FOLD_EINVAL           # misaligned table
    a.kv.v_block_mean = vm.data_ptr()
    a.kv.v = None
    assert L.fold_running_means(a.kv, 2, 128, None) == F.FOLD_EINVAL           # it reads the BF16 values
    a.kv.v = keep[2].data_ptr()
    a.kv.v_block_mean = None
    kv = F.FoldKV()
    assert L.fold_quantize_values(None, 2, 128, None, None) == F.FOLD_EINVAL
    assert L.fold_quantize_values(kv, 2, 96, None, None) == F.FOLD_EUNSUPPORTED
    assert L.fold_quantize_values(kv, 2, 128, None, None) == F.FOLD_EINVAL
