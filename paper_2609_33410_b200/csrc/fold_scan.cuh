// Split-KV scan (Algorithm 1, rebuilt for a BF16 cache on sm_100a).
//
// One CTA = 4 consumer warps + 1 producer warp, walking the 64-key tiles of its canonical
// chunks for one (KV sequence, kv head).  The producer thread stages K (and, for dense
// decode, V) tiles HBM -> shared memory with TMA through a ring of mbarriers.  Each
// consumer warp owns 16 keys of every tile: BF16 mma.sync scores them against the row
// block (query rows on M, keys on N), forms the final FP32 weights 2^(s - Z), gates them
// by the depth T, and multiplies the two-term BF16 weights into its FP32 A accumulator
// (rows on M, channels on N, its 16 keys on K).  With a finite depth, value rows are
// fetched only after scoring, row by row, by zero-filling 16-byte async copies, so cut
// rows cost no memory traffic.  At the end of a chunk the four warps' partials are added
// in a fixed order and the chunk's (A, L) goes to its own slot.
#pragma once

#include "fold_common.cuh"

namespace fold {

struct ScanParams {
  const __nv_bfloat16 *q;
  long long q_stride_b, q_stride_h;
  const float *z;
  const int *seqlens;
  const int *page_table;
  const __nv_bfloat16 *v;                         // gather path reads value rows directly
  long long v_stride_seq, v_stride_tok, v_stride_head;
  float *slots;
  long long slot_stride;
  fold_ws_header *hdr;
  int max_slots, max_seqlen, Hq, Hkv, G, stack, R;
  int paged, page_shift, max_pages, num_pages, box_tok;
  int num_splits, stages, vr;
  int pos_tok, pos_head, pos_seq;                 // which tensor-map coordinate (1..3) each axis is
  float scale_log2, neg_T;
};

template <int D, bool GATHER>
struct ScanLayout {
  static constexpr int kHalves = D / 64;
  static constexpr int kKTile = kTileKeys * D * 2;
  static constexpr int kStage = GATHER ? kKTile : 2 * kKTile;
  static constexpr int kVWarp = 16 * D * 2;
  __host__ __device__ static int pentry(int R) { return R > 8 ? 1024 : 512; }
  __host__ __device__ static int off_vring(int stages) { return stages * kStage; }
  __host__ __device__ static int off_pring(int stages, int vr) {
    return off_vring(stages) + (GATHER ? kConsumerWarps * vr * kVWarp : 0);
  }
  __host__ __device__ static int off_flags(int stages, int vr, int R) {
    return off_pring(stages, vr) + (GATHER ? kConsumerWarps * vr * pentry(R) : 0);
  }
  __host__ __device__ static int off_red(int stages, int vr, int R) {
    return off_flags(stages, vr, R) + (GATHER ? 64 : 0);
  }
  __host__ __device__ static int off_redl(int stages, int vr, int R) {
    return off_red(stages, vr, R) + kConsumerWarps * R * D * 4;
  }
  __host__ __device__ static int off_bar(int stages, int vr, int R) {
    return off_redl(stages, vr, R) + kConsumerWarps * kMaxRows * 4;
  }
  __host__ __device__ static int total(int stages, int vr, int R) {
    return off_bar(stages, vr, R) + 2 * stages * 8 + 1024;   // + slack to align the base to 1 KB
  }
};

__device__ __forceinline__ void consumer_bar() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

template <int D, bool GATHER>
__global__ void __launch_bounds__(kScanThreads, 2)
fold_scan_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                 const ScanParams p) {
  using LO = ScanLayout<D, GATHER>;
  constexpr int KSTEPS = D / 16;      // k-steps of the score product; also channel pairs of the value product
  constexpr int NT = D / 8;           // 8-channel n-tiles of the A accumulator
  constexpr int C16 = D / 8;          // 16-byte chunks per row

  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t *gen = smem_raw + (base - raw);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int split = blockIdx.x, kvh = blockIdx.y, seq = blockIdx.z;
  int n = p.seqlens[seq];
  n = n < 0 ? 0 : (n > p.max_seqlen ? p.max_seqlen : n);
  const int n_tiles = (n + kTileKeys - 1) / kTileKeys;
  const int ctiles = chunk_keys_of(n) / kTileKeys;
  const int n_chunks = num_chunks_of(n);
  if (split >= n_chunks) return;

  const int stages = p.stages, vr = p.vr, R = p.R;
  const uint32_t bar0 = base + LO::off_bar(stages, vr, R);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (stages + s); };

  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), kConsumerWarps);
    }
    mbar_fence_init();
  }
  __syncthreads();

  // ------------------------------------------------------------------ producer
  if (warp == kConsumerWarps) {
    if (lane == 0) {
      tma_prefetch_desc(&tmK);
      if (!GATHER) tma_prefetch_desc(&tmV);
      const uint64_t pol = policy_evict_first();
      bool dead = false;
      int it = 0;
      const int boxes_per_tile = kTileKeys / p.box_tok;
      const int page_mask = (1 << p.page_shift) - 1;
      for (int c = split; c < n_chunks && !dead; c += p.num_splits) {
        const int t_end = min((c + 1) * ctiles, n_tiles);
        for (int t = c * ctiles; t < t_end; ++t, ++it) {
          const int stage = it % stages, round = it / stages;
          if (round > 0 && !mbar_wait(empty_bar(stage), (round - 1) & 1, dead)) break;
          const int tok0 = t * kTileKeys;
          const int nbox = min(boxes_per_tile, (n - tok0 + p.box_tok - 1) / p.box_tok);
          mbar_expect_tx(full_bar(stage), nbox * p.box_tok * D * 2 * (GATHER ? 1 : 2));
          const uint32_t kdst = base + stage * LO::kStage;
          const uint32_t vdst = kdst + LO::kKTile;
          for (int bx = 0; bx < nbox; ++bx) {
            const int j0 = tok0 + bx * p.box_tok;
            int c_seq = seq, c_tok = j0;
            if (p.paged) {
              c_seq = p.page_table[(long long)seq * p.max_pages + (j0 >> p.page_shift)];
              c_tok = j0 & page_mask;
            }
            // the map's axes are ordered by stride; place each coordinate where its axis sits
            const int c1 = p.pos_tok == 1 ? c_tok : (p.pos_head == 1 ? kvh : c_seq);
            const int c2 = p.pos_tok == 2 ? c_tok : (p.pos_head == 2 ? kvh : c_seq);
            const int c3 = p.pos_tok == 3 ? c_tok : (p.pos_head == 3 ? kvh : c_seq);
#pragma unroll
            for (int h = 0; h < LO::kHalves; ++h) {
              const uint32_t o = (h * kTileKeys + bx * p.box_tok) * 128;
              tma_load_4d(kdst + o, &tmK, full_bar(stage), h * 64, c1, c2, c3, pol);
              if (!GATHER) tma_load_4d(vdst + o, &tmV, full_bar(stage), h * 64, c1, c2, c3, pol);
            }
          }
        }
      }
      if (dead) atomicOr(&p.hdr->wait_timeouts, 1u);
    }
    return;
  }

  // ------------------------------------------------------------------ consumers
  const int row_lo = lane >> 2, row_hi = row_lo + 8;
  const bool rv_lo = row_lo < R, rv_hi = row_hi < R;
  const bool two_blocks = R > 8;                       // warp-uniform
  const int qcol = (lane & 3) * 2;

  uint32_t qf[KSTEPS][4];
  float z_lo = 0.f, z_hi = 0.f;
  {
    const int req_lo = seq * p.stack + row_lo / p.G, head_lo = kvh * p.G + row_lo % p.G;
    const int req_hi = seq * p.stack + row_hi / p.G, head_hi = kvh * p.G + row_hi % p.G;
    const __nv_bfloat16 *ql = p.q + (long long)req_lo * p.q_stride_b + (long long)head_lo * p.q_stride_h;
    const __nv_bfloat16 *qh = p.q + (long long)req_hi * p.q_stride_b + (long long)head_hi * p.q_stride_h;
#pragma unroll
    for (int kk = 0; kk < KSTEPS; ++kk) {
      const int col = kk * 16 + qcol;
      qf[kk][0] = rv_lo ? *reinterpret_cast<const uint32_t *>(ql + col) : 0u;
      qf[kk][1] = rv_hi ? *reinterpret_cast<const uint32_t *>(qh + col) : 0u;
      qf[kk][2] = rv_lo ? *reinterpret_cast<const uint32_t *>(ql + col + 8) : 0u;
      qf[kk][3] = rv_hi ? *reinterpret_cast<const uint32_t *>(qh + col + 8) : 0u;
    }
    if (rv_lo) z_lo = p.z[(long long)req_lo * p.Hq + head_lo];
    if (rv_hi) z_hi = p.z[(long long)req_hi * p.Hq + head_hi];
  }

  float o[NT][4];
#pragma unroll
  for (int i = 0; i < NT; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
  float l_lo = 0.f, l_hi = 0.f;

  float *red = reinterpret_cast<float *>(gen + LO::off_red(stages, vr, R));
  float *redl = reinterpret_cast<float *>(gen + LO::off_redl(stages, vr, R));
  const uint32_t vring = base + LO::off_vring(stages) + warp * vr * LO::kVWarp;
  const int pentry = LO::pentry(R);
  uint32_t *pring = reinterpret_cast<uint32_t *>(gen + LO::off_pring(stages, vr) + warp * vr * pentry);
  const int page_mask = (1 << p.page_shift) - 1;

  bool dead = false;
  int it = 0;
  unsigned long long st_fetched = 0, st_total = 0, st_skipped = 0;

  // value product of one 16-key slice: A += P_hi V + P_lo V
  auto value_product = [&](uint32_t vbase, int rows_per_half, int key0, const uint32_t (&ah)[4],
                           const uint32_t (&al)[4]) {
    const int key = key0 + (((lane >> 3) & 1) << 3) + (lane & 7);
#pragma unroll
    for (int pr = 0; pr < KSTEPS; ++pr) {
      uint32_t b0, b1, b2, b3;
      ldsm_x4_trans(vbase + tile_off(key, pr * 2 + (lane >> 4), rows_per_half), b0, b1, b2, b3);
      mma_bf16(o[2 * pr], ah, b0, b1);
      mma_bf16(o[2 * pr], al, b0, b1);
      mma_bf16(o[2 * pr + 1], ah, b2, b3);
      mma_bf16(o[2 * pr + 1], al, b2, b3);
    }
  };

  for (int c = split; c < n_chunks; c += p.num_splits) {
    const int t_end = min((c + 1) * ctiles, n_tiles);
    int pend = 0, vslot = 0;                                  // gather pipeline state (per chunk)
    uint32_t pend_fetch = 0;                                  // bit i: pending tile (vslot-1-i) has rows to multiply
    for (int t = c * ctiles; t < t_end; ++t, ++it) {
      const int stage = it % stages, round = it / stages;
      if (!mbar_wait(full_bar(stage), round & 1, dead)) continue;
      const uint32_t kt = base + stage * LO::kStage;

      // ---- scores: S[rows, 16 keys] = Q K^T
      float s[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
      {
        const int key = warp * 16 + ((lane >> 4) << 3) + (lane & 7);
#pragma unroll
        for (int kk = 0; kk < KSTEPS; ++kk) {
          uint32_t b0, b1, b2, b3;
          ldsm_x4(kt + tile_off(key, kk * 2 + ((lane >> 3) & 1), kTileKeys), b0, b1, b2, b3);
          mma_bf16(s[0], qf[kk], b0, b1);
          mma_bf16(s[1], qf[kk], b2, b3);
        }
      }
      if (GATHER) {                                            // K is in registers: release the stage early
        __syncwarp();
        if (lane == 0) mbar_arrive(empty_bar(stage));
      }

      // ---- final weights against the declared reference, depth gate, mass
      const int kwarp0 = t * kTileKeys + warp * 16;
      uint32_t ah[4] = {0u, 0u, 0u, 0u}, al[4] = {0u, 0u, 0u, 0u};
      uint32_t livemask = 0;
#pragma unroll
      for (int nt = 0; nt < 2; ++nt) {
        float h0[2], l0[2], h1[2] = {0.f, 0.f}, l1[2] = {0.f, 0.f};
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const int kk16 = nt * 8 + qcol + e;
          const bool valid = (kwarp0 + kk16) < n;
          {
            const float x = fmaf(s[nt][e], p.scale_log2, -z_lo);
            const bool ok = valid && rv_lo;
            const bool live = ok && (x >= p.neg_T);
            const float pw = ok ? ex2_approx(x) : 0.f;
            float hi, lo;
            split_bf16(pw, hi, lo);
            l_lo += live ? (hi + lo) : pw;
            h0[e] = live ? hi : 0.f;
            l0[e] = live ? lo : 0.f;
            if (live) livemask |= 1u << kk16;
          }
          if (two_blocks) {
            const float x = fmaf(s[nt][2 + e], p.scale_log2, -z_hi);
            const bool ok = valid && rv_hi;
            const bool live = ok && (x >= p.neg_T);
            const float pw = ok ? ex2_approx(x) : 0.f;
            float hi, lo;
            split_bf16(pw, hi, lo);
            l_hi += live ? (hi + lo) : pw;
            h1[e] = live ? hi : 0.f;
            l1[e] = live ? lo : 0.f;
            if (live) livemask |= 1u << kk16;
          }
        }
        ah[nt * 2] = pack_bf16(h0[0], h0[1]);
        al[nt * 2] = pack_bf16(l0[0], l0[1]);
        ah[nt * 2 + 1] = pack_bf16(h1[0], h1[1]);
        al[nt * 2 + 1] = pack_bf16(l1[0], l1[1]);
      }
      const uint32_t fetch16 = __reduce_or_sync(0xffffffffu, livemask);   // verdicts ORed over the row block
      {
        const int nvalid = min(16, max(0, n - kwarp0));
        st_total += nvalid;
        st_fetched += __popc(fetch16);
        st_skipped += (fetch16 == 0 && nvalid > 0) ? 1 : 0;
      }

      if (!GATHER) {
        const uint32_t vt = kt + LO::kKTile;
        if (kwarp0 + 16 > n) {                                 // ragged tail: rows past n may hold anything
          for (int r = 0; r < 16; ++r)
            if (kwarp0 + r >= n && lane < C16)
              *reinterpret_cast<uint4 *>(gen + stage * LO::kStage + LO::kKTile +
                                         tile_off(warp * 16 + r, lane, kTileKeys)) = make_uint4(0, 0, 0, 0);
          __syncwarp();
        }
        if (fetch16 != 0) value_product(vt, kTileKeys, warp * 16, ah, al);
        if (kwarp0 + 16 > n) fence_proxy_async_smem();         // generic writes before the next TMA fill
        __syncwarp();
        if (lane == 0) mbar_arrive(empty_bar(stage));
      } else {
        // ---- request the live value rows (zero-fill the rest), defer the product
        const int slot = vslot % vr;
        __syncwarp();                                          // earlier ldmatrix reads of this slot are done
        if (fetch16 != 0) {
          int c_seq = seq, c_tok = kwarp0;
          if (p.paged) {
            const int pg = kwarp0 < n ? p.page_table[(long long)seq * p.max_pages + (kwarp0 >> p.page_shift)] : 0;
            c_seq = min(max(pg, 0), p.num_pages - 1);
            c_tok = kwarp0 & page_mask;
          }
          const __nv_bfloat16 *vsrc = p.v + (long long)c_seq * p.v_stride_seq + (long long)c_tok * p.v_stride_tok +
                                      (long long)kvh * p.v_stride_head;
          const uint32_t vdst = vring + slot * LO::kVWarp;
#pragma unroll
          for (int i = 0; i < (16 * C16) / 32; ++i) {
            const int id = i * 32 + lane;
            const int r = id / C16, c16 = id % C16;
            const bool f = (fetch16 >> r) & 1u;
            const __nv_bfloat16 *src = f ? vsrc + (long long)r * p.v_stride_tok + c16 * 8 : p.v;
            cp_async_16(vdst + tile_off(r, c16, 16), src, f ? 16u : 0u);
          }
        }
        cp_async_commit();
        {
          uint32_t *pe = pring + slot * (pentry / 4);
          if (two_blocks) {
            *reinterpret_cast<uint4 *>(pe + lane * 4) = make_uint4(ah[0], ah[1], ah[2], ah[3]);
            *reinterpret_cast<uint4 *>(pe + 128 + lane * 4) = make_uint4(al[0], al[1], al[2], al[3]);
          } else {
            *reinterpret_cast<uint4 *>(pe + lane * 4) = make_uint4(ah[0], ah[2], al[0], al[2]);
          }
        }
        pend_fetch = (pend_fetch << 1) | (fetch16 != 0 ? 1u : 0u);
        ++vslot;
        ++pend;
      }

      if (GATHER) {
        // multiply the oldest pending tile once the ring is full, or drain at the chunk's end
        const bool last = (t + 1 == t_end);
        while (pend > 0 && (pend == vr || last)) {
          switch (pend - 1) {
            case 0: cp_async_wait<0>(); break;
            case 1: cp_async_wait<1>(); break;
            case 2: cp_async_wait<2>(); break;
            default: cp_async_wait<3>(); break;
          }
          __syncwarp();
          const int old = vslot - pend;
          if ((pend_fetch >> (pend - 1)) & 1u) {
            const uint32_t *pe = pring + (old % vr) * (pentry / 4);
            uint32_t bh[4], bl[4];
            if (two_blocks) {
              const uint4 a = *reinterpret_cast<const uint4 *>(pe + lane * 4);
              const uint4 b = *reinterpret_cast<const uint4 *>(pe + 128 + lane * 4);
              bh[0] = a.x; bh[1] = a.y; bh[2] = a.z; bh[3] = a.w;
              bl[0] = b.x; bl[1] = b.y; bl[2] = b.z; bl[3] = b.w;
            } else {
              const uint4 a = *reinterpret_cast<const uint4 *>(pe + lane * 4);
              bh[0] = a.x; bh[1] = 0u; bh[2] = a.y; bh[3] = 0u;
              bl[0] = a.z; bl[1] = 0u; bl[2] = a.w; bl[3] = 0u;
            }
            value_product(vring + (old % vr) * LO::kVWarp, 16, 0, bh, bl);
          }
          --pend;
        }
      }
    }

    // ---- chunk end: add the four warps' partials in a fixed order, store the slot
    l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1);
    l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
    l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1);
    l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
    {
      float *mine = red + warp * R * D;
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        if (rv_lo) *reinterpret_cast<float2 *>(mine + row_lo * D + nt * 8 + qcol) = make_float2(o[nt][0], o[nt][1]);
        if (rv_hi) *reinterpret_cast<float2 *>(mine + row_hi * D + nt * 8 + qcol) = make_float2(o[nt][2], o[nt][3]);
        o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.f;
      }
      if ((lane & 3) == 0) {
        if (rv_lo) redl[warp * kMaxRows + row_lo] = l_lo;
        if (rv_hi) redl[warp * kMaxRows + row_hi] = l_hi;
      }
      l_lo = l_hi = 0.f;
    }
    consumer_bar();
    {
      float *slot = p.slots + (((long long)seq * p.Hkv + kvh) * p.max_slots + c) * p.slot_stride;
      const int RD = R * D;
      for (int i = threadIdx.x; i < RD; i += kConsumerWarps * 32)
        slot[i] = ((red[i] + red[RD + i]) + red[2 * RD + i]) + red[3 * RD + i];
      if (threadIdx.x < R)
        slot[RD + threadIdx.x] = ((redl[threadIdx.x] + redl[kMaxRows + threadIdx.x]) +
                                  redl[2 * kMaxRows + threadIdx.x]) + redl[3 * kMaxRows + threadIdx.x];
    }
    consumer_bar();
  }

  if (lane == 0) {
    if (dead) atomicOr(&p.hdr->wait_timeouts, 2u);
    atomicAdd(reinterpret_cast<unsigned long long *>(&p.hdr->v_rows_fetched), st_fetched);
    atomicAdd(reinterpret_cast<unsigned long long *>(&p.hdr->v_rows_total), st_total);
    if (st_skipped) atomicAdd(reinterpret_cast<unsigned long long *>(&p.hdr->v_slices_skipped), st_skipped);
  }
}

}  // namespace fold
