"""The order-free partial add (Eq. 3 / Prop. 2 applied to the forward pass) against the oracle's exact integer
arithmetic.  The add is integer work, so the bar is bit equality: the FP32 slots a scan left (or slots written here by
hand) are read back, every output element's terms are summed with oracle.grid_sum in Python integers, rounded the
way the method states (the integer sum to the nearest double, an exact power-of-two scaling, one rounding to FP32,
an IEEE FP32 division A / L, round-to-nearest-even to BF16), and `out` must agree BIT FOR BIT; lse = z + log2 L may
differ by the last place of the device's log2."""
import math

import numpy as np
import pytest
import torch

import paper_2609_33410_b200 as F
from oracle import fold_oracle as O
from paper_2609_33410_b200.workloads import make_decode_workload
from helpers import cache_of, run_gpu

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _bf16_bits_rne(x32: np.ndarray) -> np.ndarray:
    """Bit patterns of round-to-nearest-even BF16 of finite FP32 values."""
    u = x32.astype(np.float32).view(np.uint32).astype(np.uint64)
    return (((u + 0x7FFF + ((u >> 16) & 1)) >> 16) & 0xFFFF).astype(np.uint16)


def _f32_of_grid_sum(terms) -> np.float32:
    """Eq. 3 in exact integers (the oracle), then the two roundings the add performs: integer -> double, -> FP32."""
    value, _total, _shift = O.grid_sum([float(t) for t in terms])
    return np.float32(value)


def _expect_row(a_terms: np.ndarray, l_terms: np.ndarray, z: float):
    """a_terms [C, D], l_terms [C] FP32 -> (BF16 bit patterns [D], lse as float32, L as float32)."""
    C, D = a_terms.shape
    Lf = _f32_of_grid_sum(l_terms)
    out = np.empty(D, dtype=np.float32)
    for d in range(D):
        out[d] = _f32_of_grid_sum(a_terms[:, d]) / Lf                   # float32 / float32: IEEE division
    lse = np.float32(z) + np.float32(math.log2(float(Lf))) if Lf > 0 else np.float32(-np.inf)
    return _bf16_bits_rne(out), lse, Lf


def _row_terms(levels, b, h):
    """Every valid slot's (A row, L) of request b, head h over all levels, as the add sees them.
    levels: list of (slots_view tensor on the host as numpy, part, seqlens list)."""
    a_all, l_all = [], []
    for (sv, part, lens) in levels:
        G = part.num_q_heads // part.num_kv_heads
        D = part.head_dim
        seq, r = b // part.stack, (b % part.stack) * G + h % G
        c = F.fold_num_chunks(int(lens[seq]))
        blk = sv[seq, h // G, :c]
        a_all.append(blk[:, r * D:(r + 1) * D])
        l_all.append(blk[:, part.rows * D + r])
    return np.concatenate(a_all).astype(np.float32), np.concatenate(l_all).astype(np.float32)


def _check_rows(levels, rows, out, lse, z):
    out_bits = out.view(torch.int16).cpu().numpy().view(np.uint16)
    lse_h, z_h = lse.cpu().numpy(), z.cpu().numpy()
    for (b, h) in rows:
        a_terms, l_terms = _row_terms(levels, b, h)
        want_bits, want_lse, Lf = _expect_row(a_terms, l_terms, float(z_h[b, h]))
        assert np.array_equal(out_bits[b, h], want_bits), (b, h, np.flatnonzero(out_bits[b, h] != want_bits)[:8])
        ulp = np.spacing(np.float32(max(abs(float(z_h[b, h])), abs(math.log2(float(Lf))), abs(float(want_lse)), 1e-30)))
        assert abs(float(lse_h[b, h]) - float(want_lse)) <= 2.0 * float(ulp), (b, h, lse_h[b, h], want_lse)


def _split(w, T, z=None):
    cache = cache_of(w)
    bufs = F.alloc_buffers(w.q, cache, w.stack)
    if z is not None:
        bufs.z.copy_(z)
    args = F.make_args(w.q, cache, scale=w.scale, z_mode=F.Z_ESTIMATE if z is None else F.Z_GIVEN, z=bufs.z, depth_T=T,
                       stack=w.stack, workspace=bufs.workspace)
    part = F.fold_decode_split(args)
    torch.cuda.synchronize()
    return part, bufs


@pytest.mark.parametrize("T", [math.inf, 16.0])
def test_one_level_matches_exact_integer_sums_bit_for_bit(T):
    # 30, 3 and 1 slots per row: a many-slot row, a short one and a single chunk
    lens = [30000, 700, 200]
    w = make_decode_workload(3, 8, 2, 128, lens, seed=91, device=DEV)
    part, bufs = _split(w, T)
    F.fold_cascade_merge([part], bufs.out, bufs.lse, bufs.row_status)
    torch.cuda.synchronize()
    sv = F.slots_view(part, bufs.workspace).cpu().numpy()
    _check_rows([(sv, part, lens)], [(0, 0), (0, 5), (1, 3), (2, 7)], bufs.out, bufs.lse, bufs.z)


def test_two_levels_are_added_flat_and_match_bit_for_bit():
    B, Hq, Hkv, D = 6, 8, 2, 128
    g = torch.Generator(device=DEV); g.manual_seed(92)
    q = torch.randn(B, Hq, D, generator=g, device=DEV).to(torch.bfloat16)
    suffixes = [900, 1, 0, 300, 5000, 64]
    pre = make_decode_workload(B, Hq, Hkv, D, 9000, seed=93, device=DEV, stack=B, q=q)
    suf = make_decode_workload(B, Hq, Hkv, D, suffixes, seed=94, device=DEV, q=q, sink_gain=1.0)
    cp, cs = cache_of(pre), cache_of(suf)
    bp, bs = F.alloc_buffers(q, cp, stack=B), F.alloc_buffers(q, cs)
    ap = F.make_args(q, cp, z_mode=F.Z_GIVEN, z=bs.z, depth_T=16.0, stack=B, workspace=bp.workspace)
    as_ = F.make_args(q, cs, z_mode=F.Z_GIVEN, z=bs.z, depth_T=16.0, workspace=bs.workspace)
    F.fold_estimate_z([ap, as_])
    pp, ps = F.fold_decode_split(ap), F.fold_decode_split(as_)
    F.fold_cascade_merge([pp, ps], bs.out, bs.lse, bs.row_status)
    torch.cuda.synchronize()
    levels = [(F.slots_view(pp, bp.workspace).cpu().numpy(), pp, [9000]),
              (F.slots_view(ps, bs.workspace).cpu().numpy(), ps, suffixes)]
    _check_rows(levels, [(0, 0), (1, 4), (2, 7), (4, 2), (5, 6)], bs.out, bs.lse, bs.z)


def test_hand_made_slots_subnormal_huge_and_cancelling_terms():
    # the slots of a real scan are replaced by values chosen to stress the grid: a column whose largest term is
    # subnormal (the grid exponent is held at -126), huge next to tiny terms, terms that cancel, ragged slot counts
    lens = [9000, 1025, 256, 31000]                 # 9, 2, 1 and 31 slots
    w = make_decode_workload(4, 4, 2, 128, lens, seed=95, device=DEV)
    part, bufs = _split(w, math.inf)
    sv = F.slots_view(part, bufs.workspace)
    rng = np.random.default_rng(96)
    R, D = part.rows, part.head_dim
    host = sv.cpu().numpy().copy()
    for s in range(4):
        c = F.fold_num_chunks(lens[s])
        for kvh in range(2):
            blk = host[s, kvh, :c]
            a = rng.standard_normal((c, R * D)).astype(np.float32) * np.float32(2.0) ** rng.integers(-20, 20, size=(c, 1))
            a[:, 0::D] = (rng.integers(1, 2000, size=(c, R)) * 2.0 ** -149).astype(np.float32)      # subnormal column
            a[:, 1::D] = np.where(rng.random((c, R)) < 0.5, 3.0e30, -1.5e-30).astype(np.float32)    # huge and tiny
            if c >= 2:                                                                            # exact cancellation
                a[0, 2::D] = np.float32(12345.678); a[1, 2::D] = -np.float32(12345.678); a[2:, 2::D] = 0.0
            blk[:, :R * D] = a
            blk[:, R * D:R * D + R] = (rng.random((c, R)).astype(np.float32) + np.float32(0.5)) * np.float32(2.0) ** rng.integers(-3, 40, size=(c, 1))
    sv.copy_(torch.from_numpy(host).to(DEV))
    F.fold_cascade_merge([part], bufs.out, bufs.lse, bufs.row_status)
    torch.cuda.synchronize()
    rows = [(0, 0), (0, 3), (1, 1), (2, 2), (3, 0), (3, 3)]
    _check_rows([(host, part, lens)], rows, bufs.out, bufs.lse, bufs.z)
