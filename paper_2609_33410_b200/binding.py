"""ctypes binding of the fold decode C ABI (include/fold.h).

Argument marshalling only: every step of the decode path runs in the CUDA library.  The
library is loaded from the in-tree shared object; if it is missing it is built with nvcc,
and if that fails the import fails -- there is no fallback path.
"""
from __future__ import annotations

import ctypes as C
import math
import os
from dataclasses import dataclass
from typing import List, Optional, Sequence

import torch

from . import build as _build

# ------------------------------------------------------------------ C structs (mirror include/fold.h)
FOLD_OK, FOLD_EINVAL, FOLD_EUNSUPPORTED, FOLD_EWORKSPACE, FOLD_ECUDA, FOLD_ETOOLARGE = range(6)
STATIC_SCRATCH_BYTES = 16 << 20
Z_ESTIMATE, Z_GIVEN, Z_EXACT_MAX, Z_ZERO = range(4)
ROW_RANGE, ROW_NONFINITE, ROW_EMPTY = 1, 2, 4
INPUTS_SETTLED = 1                               # fold_args.flags
SEPARATE_LAUNCHES = 2
ONE_LAUNCH = 4


class FoldKV(C.Structure):
    _fields_ = [("k", C.c_void_p), ("v", C.c_void_p),
                ("stride_seq", C.c_int64), ("stride_tok", C.c_int64), ("stride_head", C.c_int64),
                ("page_table", C.c_void_p), ("page_size", C.c_int32), ("max_pages_per_seq", C.c_int32),
                ("num_pages", C.c_int32), ("capacity", C.c_int32), ("num_seqs", C.c_int32),
                ("seqlens", C.c_void_p), ("max_seqlen", C.c_int32),
                ("v_block_mean", C.c_void_p), ("mean_stride_seq", C.c_int64), ("mean_stride_block", C.c_int64),
                ("mean_stride_head", C.c_int64),
                ("k_plane_a", C.c_void_p), ("k_plane_b", C.c_void_p),
                ("plane_stride_seq", C.c_int64), ("plane_stride_tok", C.c_int64), ("plane_stride_head", C.c_int64),
                ("k_scale", C.c_void_p), ("scale_stride_seq", C.c_int64), ("scale_stride_head", C.c_int64),
                ("v_plane_1", C.c_void_p), ("v_plane_2", C.c_void_p), ("v_scale_log2", C.c_int32)]


class FoldArgs(C.Structure):
    _fields_ = [("batch", C.c_int32), ("num_q_heads", C.c_int32), ("num_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("stack", C.c_int32),
                ("q", C.c_void_p), ("q_stride_b", C.c_int64), ("q_stride_h", C.c_int64),
                ("kv", FoldKV),
                ("softmax_scale", C.c_float), ("z_mode", C.c_int32), ("z", C.c_void_p),
                ("depth_T", C.c_float), ("num_splits", C.c_int32),
                ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t),
                ("out", C.c_void_p), ("lse", C.c_void_p), ("row_status", C.c_void_p),
                ("draft_mask", C.c_void_p), ("draft_len", C.c_int32), ("refine_tau", C.c_float),
                ("refine_tau_v", C.c_float), ("flags", C.c_int32),
                ("side_stream", C.c_void_p), ("side_fork_event", C.c_void_p), ("side_join_event", C.c_void_p),
                ("live_hint", C.c_float)]


class FoldPartials(C.Structure):
    _fields_ = [("slots", C.c_void_p), ("seqlens", C.c_void_p), ("z", C.c_void_p),
                ("batch", C.c_int32), ("num_q_heads", C.c_int32), ("num_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("stack", C.c_int32),
                ("num_seqs", C.c_int32), ("max_slots", C.c_int32), ("rows", C.c_int32),
                ("max_seqlen", C.c_int32), ("slot_stride", C.c_int64)]


class FoldWsHeader(C.Structure):
    _fields_ = [("wait_timeouts", C.c_uint32), ("reserved", C.c_uint32),
                ("v_rows_fetched", C.c_uint64), ("v_rows_total", C.c_uint64),
                ("v_slices_skipped", C.c_uint64), ("k_rows_refined", C.c_uint64), ("v2_rows_refined", C.c_uint64),
                ("pad", C.c_uint64 * 2)]


EXPORTS = ["fold_chunk_keys", "fold_num_chunks", "fold_workspace_bytes", "fold_estimate_z",
           "fold_decode_split", "fold_cascade_merge", "fold_decode", "fold_decode_launches", "fold_decode_cascade", "fold_host_staging_bytes",
           "fold_decode_host", "fold_decode_static", "fold_block_means", "fold_running_means", "fold_quantize_keys", "fold_quantize_values", "fold_probe_read", "fold_status_string",
           "fold_version"]

_lib = None


def lib() -> C.CDLL:
    """The loaded CUDA library.  Raises if it cannot be built or loaded."""
    global _lib
    if _lib is None:
        path = _build.build()
        L = C.CDLL(path)
        L.fold_chunk_keys.restype = C.c_int32; L.fold_chunk_keys.argtypes = [C.c_int32]
        L.fold_num_chunks.restype = C.c_int32; L.fold_num_chunks.argtypes = [C.c_int32]
        L.fold_workspace_bytes.restype = C.c_size_t; L.fold_workspace_bytes.argtypes = [C.POINTER(FoldArgs)]
        L.fold_estimate_z.restype = C.c_int
        L.fold_estimate_z.argtypes = [C.POINTER(C.POINTER(FoldArgs)), C.c_int, C.c_void_p]
        L.fold_decode_split.restype = C.c_int
        L.fold_decode_split.argtypes = [C.POINTER(FoldArgs), C.POINTER(FoldPartials), C.c_void_p]
        L.fold_cascade_merge.restype = C.c_int
        L.fold_cascade_merge.argtypes = [C.POINTER(C.POINTER(FoldPartials)), C.c_int, C.c_void_p, C.c_void_p,
                                         C.c_void_p, C.c_void_p]
        L.fold_decode.restype = C.c_int; L.fold_decode.argtypes = [C.POINTER(FoldArgs), C.c_void_p]
        L.fold_decode_cascade.restype = C.c_int
        L.fold_decode_cascade.argtypes = [C.POINTER(C.POINTER(FoldArgs)), C.c_int, C.c_void_p]
        L.fold_host_staging_bytes.restype = C.c_size_t; L.fold_host_staging_bytes.argtypes = [C.POINTER(FoldArgs)]
        L.fold_decode_host.restype = C.c_int
        L.fold_decode_host.argtypes = [C.POINTER(FoldArgs), C.c_void_p, C.c_size_t, C.c_void_p]
        L.fold_decode_static.restype = C.c_int; L.fold_decode_static.argtypes = [C.POINTER(FoldArgs), C.c_void_p]
        L.fold_decode_launches.restype = C.c_int32; L.fold_decode_launches.argtypes = [C.POINTER(FoldArgs)]
        L.fold_block_means.restype = C.c_int
        L.fold_block_means.argtypes = [C.POINTER(FoldKV), C.c_int32, C.c_int32, C.c_void_p]
        L.fold_running_means.restype = C.c_int
        L.fold_running_means.argtypes = [C.POINTER(FoldKV), C.c_int32, C.c_int32, C.c_void_p]
        L.fold_quantize_keys.restype = C.c_int
        L.fold_quantize_keys.argtypes = [C.POINTER(FoldKV), C.c_int32, C.c_int32, C.c_void_p, C.c_void_p]
        L.fold_quantize_values.restype = C.c_int
        L.fold_quantize_values.argtypes = [C.POINTER(FoldKV), C.c_int32, C.c_int32, C.c_void_p, C.c_void_p]
        L.fold_probe_read.restype = C.c_int
        L.fold_probe_read.argtypes = [C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p]
        L.fold_status_string.restype = C.c_char_p; L.fold_status_string.argtypes = [C.c_int]
        L.fold_version.restype = C.c_int
        _lib = L
    return _lib


class FoldError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {lib().fold_status_string(status).decode()} (status {status})")


def _check(status: int, where: str):
    if status != FOLD_OK:
        raise FoldError(status, where)


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream(stream=None) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


# ------------------------------------------------------------------ argument building
@dataclass
class KVCache:
    """A BF16 cache view.  Contiguous: k, v [num_seqs, capacity, Hkv, D] (any strides with D
    contiguous).  Paged: k, v [num_pages, page_size, Hkv, D] and page_table [num_seqs, max_pages]."""
    k: torch.Tensor
    v: torch.Tensor
    seqlens: torch.Tensor
    max_seqlen: int
    page_table: Optional[torch.Tensor] = None
    v_block_mean: Optional[torch.Tensor] = None     # [num_seqs, ceil(max_seqlen / 64), Hkv, D] bf16: switches the block tail on
    # two-plane INT8 keys (alloc_key_planes + fold_quantize_keys): planes shaped like k, scales [seqs-or-pages, Hkv, tokens]
    k_plane_a: Optional[torch.Tensor] = None
    k_plane_b: Optional[torch.Tensor] = None
    k_scale: Optional[torch.Tensor] = None
    # two E4M3 value planes (uint8, shaped and strided like the key planes) under the scale 2^v_scale_log2
    v_plane_1: Optional[torch.Tensor] = None
    v_plane_2: Optional[torch.Tensor] = None
    v_scale_log2: int = 0

    def to_c(self, mean_rows_only: bool = False) -> FoldKV:
        k, v = self.k, self.v
        assert k.dtype == torch.bfloat16 and v.dtype == torch.bfloat16 and k.dim() == 4
        assert k.stride() == v.stride() and k.shape == v.shape and k.stride(3) == 1
        assert self.seqlens.dtype == torch.int32 and self.seqlens.is_contiguous()
        kv = FoldKV()
        kv.k, kv.v = k.data_ptr(), v.data_ptr()
        kv.stride_seq, kv.stride_tok, kv.stride_head = k.stride(0), k.stride(1), k.stride(2)
        kv.seqlens = self.seqlens.data_ptr()
        kv.num_seqs = self.seqlens.shape[0]
        kv.max_seqlen = int(self.max_seqlen)
        if self.page_table is not None:
            pt = self.page_table
            assert pt.dtype == torch.int32 and pt.is_contiguous() and pt.dim() == 2
            kv.page_table = pt.data_ptr()
            kv.page_size = k.shape[1]
            kv.max_pages_per_seq = pt.shape[1]
            kv.num_pages = k.shape[0]
            kv.capacity = 0
        else:
            kv.page_table = None
            kv.page_size = 0
            kv.max_pages_per_seq = 0
            kv.num_pages = 0
            kv.capacity = k.shape[1]
        if self.v_block_mean is not None:
            m = self.v_block_mean
            assert m.dtype == torch.bfloat16 and m.dim() == 4 and m.stride(3) == 1 and m.shape[0] == kv.num_seqs
            # (with E4M3 value planes the table is the sequences' mean rows: one block)
            assert (m.shape[1] * 64 >= kv.max_seqlen or self.v_plane_1 is not None or mean_rows_only) and m.shape[2:] == k.shape[2:]
            # with value planes only row 0 is read, as the sequence's mean: a table of block means would be misread
            assert self.v_plane_1 is None or m.shape[1] == 1, "E4M3 value planes take the one-row table of fold_running_means"
            kv.v_block_mean = m.data_ptr()
            kv.mean_stride_seq, kv.mean_stride_block, kv.mean_stride_head = m.stride(0), m.stride(1), m.stride(2)
        else:
            kv.v_block_mean = None
        if self.k_plane_a is not None:
            pa, pb, sc = self.k_plane_a, self.k_plane_b, self.k_scale
            assert pa.dtype == torch.int8 and pb.dtype == torch.int8 and pa.shape == k.shape and pb.shape == k.shape
            assert pa.stride() == pb.stride() and pa.stride(3) == 1
            assert sc.dtype == torch.bfloat16 and sc.dim() == 3 and sc.stride(2) == 1 and sc.shape[:2] == (k.shape[0], k.shape[2])
            assert sc.shape[2] >= (k.shape[1] + 7) // 8 * 8
            kv.k_plane_a, kv.k_plane_b, kv.k_scale = pa.data_ptr(), pb.data_ptr(), sc.data_ptr()
            kv.plane_stride_seq, kv.plane_stride_tok, kv.plane_stride_head = pa.stride(0), pa.stride(1), pa.stride(2)
            kv.scale_stride_seq, kv.scale_stride_head = sc.stride(0), sc.stride(1)
        else:
            kv.k_plane_a = kv.k_plane_b = kv.k_scale = None
        if self.v_plane_1 is not None:
            p1, p2 = self.v_plane_1, self.v_plane_2
            assert self.k_plane_a is not None and p1.dtype == torch.uint8 and p2.dtype == torch.uint8
            assert p1.shape == k.shape and p2.shape == k.shape and p1.stride() == self.k_plane_a.stride() == p2.stride()
            kv.v_plane_1, kv.v_plane_2, kv.v_scale_log2 = p1.data_ptr(), p2.data_ptr(), int(self.v_scale_log2)
        else:
            kv.v_plane_1 = kv.v_plane_2 = None
        return kv

    def alloc_key_planes(self) -> None:
        """Allocate the two INT8 key planes and the scales (fold_quantize_keys fills them)."""
        k = self.k
        self.k_plane_a = torch.zeros(k.shape, dtype=torch.int8, device=k.device)
        self.k_plane_b = torch.zeros(k.shape, dtype=torch.int8, device=k.device)
        toks = (k.shape[1] + 127) // 128 * 128
        self.k_scale = torch.zeros(k.shape[0], k.shape[2], toks, dtype=torch.bfloat16, device=k.device)

    def alloc_block_means(self) -> torch.Tensor:
        """An empty table of the shape fold_block_means fills (and the block tail reads)."""
        nb = max((int(self.max_seqlen) + 63) // 64, 1)
        return torch.zeros(self.seqlens.shape[0], nb, self.k.shape[2], self.k.shape[3], dtype=torch.bfloat16,
                           device=self.k.device)


def make_args(q: torch.Tensor, cache: KVCache, *, scale: Optional[float] = None, z_mode: int = Z_ESTIMATE,
              z: Optional[torch.Tensor] = None, depth_T: float = math.inf, num_splits: int = 0, stack: int = 1,
              workspace: Optional[torch.Tensor] = None, out: Optional[torch.Tensor] = None,
              lse: Optional[torch.Tensor] = None, row_status: Optional[torch.Tensor] = None,
              draft_mask: Optional[torch.Tensor] = None, draft_len: int = 0, refine_tau: float = 0.0,
              refine_tau_v: float = 0.0, flags: int = 0, side=None, live_hint: float = 0.0) -> FoldArgs:
    """`side`: a CascadeSide (a second stream and two events of the caller's) for fold_decode_cascade's first level."""
    assert q.dtype == torch.bfloat16 and q.dim() == 3 and q.stride(2) == 1
    B, Hq, D = q.shape
    a = FoldArgs()
    a.batch, a.num_q_heads, a.num_kv_heads, a.head_dim = B, Hq, cache.k.shape[2], D
    a.stack = stack
    a.q, a.q_stride_b, a.q_stride_h = q.data_ptr(), q.stride(0), q.stride(1)
    a.kv = cache.to_c()
    a.softmax_scale = float(scale if scale is not None else 1.0 / math.sqrt(D))
    a.z_mode = z_mode
    a.z = _ptr(z)
    a.depth_T = float(depth_T)
    a.num_splits = int(num_splits)
    a.workspace = _ptr(workspace)
    a.workspace_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    a.out, a.lse, a.row_status = _ptr(out), _ptr(lse), _ptr(row_status)
    if draft_len:
        # int32 storage for the uint32 masks (torch has no uint32 arithmetic): the bit patterns are what is passed
        assert draft_mask is not None and draft_mask.dtype == torch.int32 and draft_mask.numel() == B
        assert draft_mask.is_contiguous()
    a.draft_mask, a.draft_len = (_ptr(draft_mask), int(draft_len)) if draft_len else (None, 0)
    a.refine_tau = float(refine_tau)
    a.refine_tau_v = float(refine_tau_v)
    a.flags = int(flags)
    a.live_hint = float(live_hint)
    if side is not None:
        a.side_stream, a.side_fork_event, a.side_join_event = side.stream.cuda_stream, side.fork.cuda_event, side.join.cuda_event
    return a


class CascadeSide:
    """A side stream and two events owned by the caller, handed to fold_decode_cascade through the first level's
    arguments (the library keeps no stream or event of its own).  Keep the object alive while calls that use it run."""

    def __init__(self, device=None):
        self.stream = torch.cuda.Stream(device=device)
        self.fork, self.join = torch.cuda.Event(), torch.cuda.Event()
        for e in (self.fork, self.join):                     # torch creates the CUDA event at its first record
            e.record(self.stream)
        self.stream.synchronize()


def fold_workspace_bytes(args: FoldArgs) -> int:
    return int(lib().fold_workspace_bytes(C.byref(args)))


def fold_chunk_keys(n: int) -> int:
    return int(lib().fold_chunk_keys(n))


def fold_num_chunks(n: int) -> int:
    return int(lib().fold_num_chunks(n))


# ------------------------------------------------------------------ entry points (same names as the C ABI)
def fold_estimate_z(levels: Sequence[FoldArgs], stream=None) -> None:
    arr = (C.POINTER(FoldArgs) * len(levels))(*[C.pointer(a) for a in levels])
    _check(lib().fold_estimate_z(arr, len(levels), _stream(stream)), "fold_estimate_z")


def fold_decode_split(args: FoldArgs, stream=None) -> FoldPartials:
    part = FoldPartials()
    _check(lib().fold_decode_split(C.byref(args), C.byref(part), _stream(stream)), "fold_decode_split")
    return part


def fold_cascade_merge(levels: Sequence[FoldPartials], out: torch.Tensor, lse: Optional[torch.Tensor] = None,
                       row_status: Optional[torch.Tensor] = None, stream=None) -> None:
    arr = (C.POINTER(FoldPartials) * len(levels))(*[C.pointer(p) for p in levels])
    _check(lib().fold_cascade_merge(arr, len(levels), out.data_ptr(), _ptr(lse), _ptr(row_status), _stream(stream)),
           "fold_cascade_merge")


def fold_block_means(cache: KVCache, stream=None) -> torch.Tensor:
    """Fill (allocating it if the cache has none) cache.v_block_mean from cache.v; returns the table."""
    if cache.v_block_mean is None:
        cache.v_block_mean = cache.alloc_block_means()
    kv = cache.to_c()
    _check(lib().fold_block_means(C.byref(kv), int(cache.k.shape[2]), int(cache.k.shape[3]), _stream(stream)),
           "fold_block_means")
    return cache.v_block_mean


def fold_running_means(cache: KVCache, stream=None) -> torch.Tensor:
    """The 8-bit value format's cut model: fill (allocating a one-block table if the cache has none)
    cache.v_block_mean[:, 0] with the mean value row of every (sequence, kv head); returns the table."""
    if cache.v_block_mean is None:
        cache.v_block_mean = torch.zeros(cache.seqlens.shape[0], 1, cache.k.shape[2], cache.k.shape[3],
                                         dtype=torch.bfloat16, device=cache.k.device)
    kv = cache.to_c(mean_rows_only=True)
    _check(lib().fold_running_means(C.byref(kv), int(cache.k.shape[2]), int(cache.k.shape[3]), _stream(stream)),
           "fold_running_means")
    return cache.v_block_mean


def fold_quantize_keys(cache: KVCache, first_token: Optional[torch.Tensor] = None, stream=None) -> None:
    """Cache write for two-plane INT8 keys: rotate and split the BF16 key rows of tokens first_token[s] .. seqlens[s]-1
    (all tokens when first_token is None) into cache.k_plane_a / k_plane_b / k_scale (allocated here if absent)."""
    if cache.k_plane_a is None:
        cache.alloc_key_planes()
    if first_token is not None:
        assert first_token.dtype == torch.int32 and first_token.is_contiguous() and first_token.numel() == cache.seqlens.numel()
    kv = cache.to_c()
    _check(lib().fold_quantize_keys(C.byref(kv), int(cache.k.shape[2]), int(cache.k.shape[3]), _ptr(first_token),
                                    _stream(stream)), "fold_quantize_keys")


def fold_quantize_values(cache: KVCache, scale_log2: int, first_token: Optional[torch.Tensor] = None, stream=None) -> None:
    """Cache write for the E4M3 value planes (allocated here if absent; the key planes must exist): p1, p2 of every
    value row of tokens first_token[s] .. seqlens[s]-1 under the scale 2^scale_log2."""
    assert cache.k_plane_a is not None, "E4M3 value planes go with two-plane keys"
    if cache.v_plane_1 is None:
        cache.v_plane_1 = torch.zeros(cache.k.shape, dtype=torch.uint8, device=cache.k.device)
        cache.v_plane_2 = torch.zeros(cache.k.shape, dtype=torch.uint8, device=cache.k.device)
    cache.v_scale_log2 = int(scale_log2)
    kv = cache.to_c()
    _check(lib().fold_quantize_values(C.byref(kv), int(cache.k.shape[2]), int(cache.k.shape[3]), _ptr(first_token),
                                      _stream(stream)), "fold_quantize_values")


def fold_decode(args: FoldArgs, stream=None) -> None:
    _check(lib().fold_decode(C.byref(args), _stream(stream)), "fold_decode")


def fold_decode_launches(args: FoldArgs) -> int:
    return int(lib().fold_decode_launches(C.byref(args)))


def fold_decode_cascade(levels: Sequence[FoldArgs], stream=None) -> None:
    arr = (C.POINTER(FoldArgs) * len(levels))(*[C.pointer(a) for a in levels])
    _check(lib().fold_decode_cascade(arr, len(levels), _stream(stream)), "fold_decode_cascade")


def fold_host_staging_bytes(args: FoldArgs) -> int:
    return int(lib().fold_host_staging_bytes(C.byref(args)))


def fold_decode_host(host_args: FoldArgs, staging: torch.Tensor, stream=None) -> None:
    _check(lib().fold_decode_host(C.byref(host_args), staging.data_ptr(), staging.numel() * staging.element_size(),
                                  _stream(stream)), "fold_decode_host")


def fold_decode_static(args: FoldArgs, stream=None) -> None:
    """fold_decode for callers that may not allocate device memory: the workspace fields of `args` are
    ignored and the library's built-in scratch array (STATIC_SCRATCH_BYTES per device) is used instead.
    Raises FoldError(FOLD_ETOOLARGE) when the call would need more.  Calls on one device share that array:
    do not let two of them overlap on the GPU; make the first call on a device outside stream capture."""
    _check(lib().fold_decode_static(C.byref(args), _stream(stream)), "fold_decode_static")


# ------------------------------------------------------------------ small conveniences for tests and the benchmark
@dataclass
class DecodeBuffers:
    out: torch.Tensor
    lse: torch.Tensor
    z: torch.Tensor
    row_status: torch.Tensor
    workspace: torch.Tensor

    def header(self) -> FoldWsHeader:
        raw = self.workspace[:64].cpu().numpy().tobytes()
        return FoldWsHeader.from_buffer_copy(raw)


def alloc_buffers(q: torch.Tensor, cache: KVCache, stack: int = 1) -> DecodeBuffers:
    """Device buffers one decode call needs (torch is used for memory only)."""
    B, Hq, D = q.shape
    dev = q.device
    probe = make_args(q, cache, stack=stack)
    nbytes = fold_workspace_bytes(probe)
    if nbytes == 0:
        raise FoldError(FOLD_EINVAL, "fold_workspace_bytes")
    return DecodeBuffers(out=torch.empty(B, Hq, D, dtype=torch.bfloat16, device=dev),
                         lse=torch.empty(B, Hq, dtype=torch.float32, device=dev),
                         z=torch.zeros(B, Hq, dtype=torch.float32, device=dev),
                         row_status=torch.zeros(B, Hq, dtype=torch.int32, device=dev),
                         workspace=torch.empty(nbytes, dtype=torch.uint8, device=dev))


def decode(q: torch.Tensor, cache: KVCache, bufs: DecodeBuffers, *, depth_T: float = math.inf,
           z_mode: int = Z_ESTIMATE, num_splits: int = 0, scale: Optional[float] = None, stack: int = 1,
           draft_mask: Optional[torch.Tensor] = None, draft_len: int = 0, refine_tau: float = 0.0,
           refine_tau_v: float = 0.0, flags: int = 0, live_hint: float = 0.0, stream=None) -> FoldArgs:
    args = make_args(q, cache, scale=scale, z_mode=z_mode, z=bufs.z, depth_T=depth_T, num_splits=num_splits,
                     stack=stack, workspace=bufs.workspace, out=bufs.out, lse=bufs.lse, row_status=bufs.row_status,
                     draft_mask=draft_mask, draft_len=draft_len, refine_tau=refine_tau, refine_tau_v=refine_tau_v,
                     flags=flags, live_hint=live_hint)
    fold_decode(args, stream)
    return args


def decode_certified(q: torch.Tensor, cache: KVCache, bufs: DecodeBuffers, *, max_reruns: int = 2, **kw) -> int:
    """The range certificate's loop (Section 3, "Choosing the reference"): decode; if a row's status carries
    ROW_RANGE or ROW_NONFINITE (its L left [2^-1, 2^100] or its output is not finite), give that row the
    log-sum-exp the decode reported as its reference where that is finite (Z = lse makes L = 1) and decode
    again with the references given.  Rows that were in range keep their reference, so their bits do not
    change.  Host-side control flow around the C ABI calls: it synchronises the stream to read the status, as
    the paper's loop does, and is not part of a timed step.  Returns the number of re-runs."""
    decode(q, cache, bufs, **kw)
    reruns = 0
    while reruns < max_reruns:
        torch.cuda.synchronize(q.device)
        bad = (bufs.row_status & (ROW_RANGE | ROW_NONFINITE)) != 0
        bad &= torch.isfinite(bufs.lse)
        if not bool(bad.any()):
            break
        bufs.z.copy_(torch.where(bad, bufs.lse, bufs.z))
        decode(q, cache, bufs, **dict(kw, z_mode=Z_GIVEN))
        reruns += 1
    return reruns


def fold_probe_read(buf: torch.Tensor, sink: Optional[torch.Tensor] = None, stream=None) -> None:
    """Stream `buf` (device memory) once with read-only loads: time it with events for the read-only bandwidth."""
    _check(lib().fold_probe_read(buf.data_ptr(), buf.numel() * buf.element_size(), _ptr(sink), _stream(stream)),
           "fold_probe_read")


def slots_view(part: FoldPartials, workspace: torch.Tensor) -> torch.Tensor:
    """FP32 view [num_seqs, Hkv, max_slots, slot_stride] of the partial slots inside `workspace`."""
    off = part.slots - workspace.data_ptr()
    n = part.num_seqs * part.num_kv_heads * part.max_slots * part.slot_stride
    flat = workspace[off: off + 4 * n].view(torch.float32)
    return flat.view(part.num_seqs, part.num_kv_heads, part.max_slots, part.slot_stride)
