// Split-KV scan (Algorithm 1, rebuilt for a BF16 cache on sm_100a).
//
// A CTA walks the key tiles of its canonical chunks for one (KV sequence, kv head).  A producer thread
// stages tiles HBM -> shared memory with TMA through a ring of mbarriers.  Every tile is cut into four
// slices; slice w of every tile belongs to warp w of a role, which keeps the instruction sequence that
// forms a chunk's (A, L) independent of the grid, the batch and the split count.
//
//   scores   BF16 mma.sync over the slice's keys and the block's query rows
//   weights  p = 2^(s - Z) in FP32, final when computed; the depth gate s - Z >= -T decides per row
//            whether a key's value is used; L sums every key's weight
//   values   two-term BF16 weights (P_hi + P_lo) times V, FP32 accumulate
//
// Row blocks (up to 16 rows per (sequence, kv head)) put the rows on the MMA's N side (keys, then
// channels, on M) in one or two 8-row N tiles: half the MMAs and accumulators of a rows-on-M form,
// which only the mma.sync stacked-row kernel still uses.  Row-block kernels walk 16 KB key tiles at
// either head dimension (a warp's slice is 4 KB of keys: 16 keys at D = 128, 32 at D = 64); the
// stacked-row kernel walks 64-key tiles with 16-key slices.
//
// Kernels:
//   fold_scan_dense_kernel<D> / fold_scan_dense_nt2_kernel<D> (T = inf; up to 8 / 9..16 rows): K and V
//     tiles arrive together by TMA; four consumer warps score and multiply in place.
//   fold_scan_gated_narrow_kernel<D, TAIL, NT> (finite T): only K is prefetched.
//     Four scorer warps score a slice, publish its weights and request just the value rows some row of
//     the group keeps -- a whole 16-key sub-slice by one TMA box when most of it is live, else row by
//     row with zero-filling 16-byte async copies; four multiplier warps wait for those rows and
//     accumulate A.  Scoring never waits for values and values never wait for keys, so both memory
//     latencies are covered by ring depth, and cut rows cost no traffic.
//   fold_scan_stacked_kernel<D, GATED>: more than 16 rows per (sequence, kv head) on mma.sync (the
//     tcgen05 kernels take head_dim 128 with 64 rows or more).
// At the end of a chunk the four warps of a role add their partials in a fixed order and write the
// chunk's slot.  Grid: kv heads on x, so CTAs that run together read neighbouring rows of the same
// tokens; splits on y; KV sequences on z.
#pragma once

#include "fold_common.cuh"

namespace fold {

struct ScanParams {
  const __nv_bfloat16 *q;
  long long q_stride_b, q_stride_h;
  const float *z;
  const int *seqlens;
  const int *page_table;
  const __nv_bfloat16 *v;                         // gated path reads value rows directly
  const __nv_bfloat16 *k;                         // key rows (same strides as v): L2 prefetches of the tcgen05 row-block kernel
  long long v_stride_seq, v_stride_tok, v_stride_head;
  const uint32_t *draft_mask;                     // drafts: per request, which of the last draft_len keys it uses
  int draft_len;
  const __nv_bfloat16 *vmean;                     // block tail: mean value row of every 64-key block, or null
  long long vm_stride_seq, vm_stride_block, vm_stride_head;
  float *slots;
  long long slot_stride;
  fold_ws_header *hdr;
  int max_slots, max_seqlen, Hq, Hkv, G, stack, R;
  int num_seqs;                                   // KV sequences of the launch (persistent kernels walk them all)
  int chunk_major;                                // tcgen05 row-block kernel: the chunk list's order (1: chunk fastest)
  int paged, page_shift, max_pages, num_pages, box_tok;
  int num_splits, stages, vr;
  int pos_tok, pos_head, pos_seq;                 // which tensor-map coordinate (1..3) each axis is
  int row_groups;                                 // row-block kernels: 16-row groups per (sequence, kv head), each its own CTA
  int box_min;                                    // gated: fetch a whole slice by one TMA box from this many live rows on
  float scale_log2, neg_T;
};

constexpr int kDenseThreads = (kConsumerWarps + 1) * 32;        // 4 consumers + producer
constexpr int kGatedThreads = (2 * kConsumerWarps + 1) * 32;    // 4 scorers + 4 multipliers + producer

// Shared-memory carve-up.  All offsets are from a 1 KB-aligned base.
template <int D, int TK = kTileKeys>
struct DenseLayout {
  static constexpr int kKTile = TK * D * 2;
  static constexpr int kStage = 2 * kKTile;                                    // K tile then V tile
  __host__ __device__ static int off_red(int stages) { return stages * kStage; }
  __host__ __device__ static int off_redl(int stages, int R) { return off_red(stages) + kConsumerWarps * R * D * 4; }
  __host__ __device__ static int off_bar(int stages, int R) { return off_redl(stages, R) + kConsumerWarps * kMaxRows * 4; }
  __host__ __device__ static int total(int stages, int R) { return off_bar(stages, R) + 2 * stages * 8 + 1024; }
};

// Narrow gated kernel: every value slice in the swizzled box layout (no row padding), and a two-warp
// parking area for the chunk-end add.
template <int D, bool TAIL = false, int NT = 1>
struct GatedNarrowLayout {
  static constexpr int kTK = narrow_tile_keys<D>();          // keys per tile
  static constexpr int kU = kTK / 64;                        // 16-key sub-slices per warp slice
  static constexpr int kKTile = kTK * D * 2;
  static constexpr int kVSlice = 16 * kU * D * 2;            // [D/64 halves][16 kU rows][128 B], swizzled
  // per slice: 16 B of B-operand registers per lane and sub-slice; with the block tail each lane's cut mass of its
  // two rows (8 B per lane) and the mean value row of the slice's block (D * 2 <= 256 B); the verdict words
  static constexpr int kPEntry = kU * NT * 512 + (TAIL ? NT * 256 + 256 : 0) + 32;   // NT: 8-row N tiles per warp
  static constexpr int kMeanBytes = (kTK / 64) * D * 2;      // mean rows that ride with a K tile: one per 64-key block
  static constexpr int kKStage = kKTile + (TAIL ? 1024 : 0); // K tile (+ mean rows), 1 KB-aligned for the swizzle
  static constexpr int kPark = D / 16 * 4 * 32 * 4;          // one warp's accumulators, fragment order
  __host__ __device__ static int off_vring(int stages) { return stages * kKStage; }
  __host__ __device__ static int off_pring(int stages, int vr) { return off_vring(stages) + kConsumerWarps * vr * kVSlice; }
  __host__ __device__ static int off_red(int stages, int vr) { return off_pring(stages, vr) + kConsumerWarps * vr * kPEntry; }
  __host__ __device__ static int off_redl(int stages, int vr) { return off_red(stages, vr) + 2 * kPark; }
  __host__ __device__ static int off_bar(int stages, int vr) { return off_redl(stages, vr) + kConsumerWarps * kMaxRows * 4; }
  __host__ __device__ static int total(int stages, int vr) {
    return off_bar(stages, vr) + 2 * stages * 8 + 2 * kConsumerWarps * vr * 8 + 1024;
  }
};

__device__ __forceinline__ void named_bar(int id, int threads = 128) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

// ------------------------------------------------------------------------------------------------
// Geometry of the CTA's work: sequence length, tiles, chunks.
struct SeqWork {
  int n, n_tiles, ctiles, n_chunks;
};
template <int TK = kTileKeys>
__device__ __forceinline__ SeqWork seq_work(const ScanParams &p, int seq) {
  SeqWork w;
  int n = p.seqlens[seq];
  w.n = n < 0 ? 0 : (n > p.max_seqlen ? p.max_seqlen : n);
  w.n_tiles = (w.n + TK - 1) / TK;
  w.ctiles = chunk_keys_of(w.n) / TK;
  w.n_chunks = num_chunks_of(w.n);
  return w;
}

struct TileCursor {            // walks the tiles of chunks split, split + num_splits, ... in order
  int c, t, t_end;
};
__device__ __forceinline__ TileCursor cursor_begin(const SeqWork &w, int split) {
  TileCursor k;
  k.c = split;
  k.t = split * w.ctiles;
  k.t_end = min((split + 1) * w.ctiles, w.n_tiles);
  return k;
}
__device__ __forceinline__ bool cursor_valid(const TileCursor &k, const SeqWork &w) { return k.c < w.n_chunks; }
// returns true if the tile just left was the last of its chunk
__device__ __forceinline__ bool cursor_next(TileCursor &k, const SeqWork &w, int num_splits) {
  if (++k.t < k.t_end) return false;
  k.c += num_splits;
  k.t = k.c * w.ctiles;
  k.t_end = min((k.c + 1) * w.ctiles, w.n_tiles);
  return true;
}

// Producer thread: TMA-stage the tiles of chunks split, split + num_splits, ... in order.
// WITH_MEAN: the mean value rows of the tile's 64-key blocks (block tail) follow the K tile in its stage.
template <int D, bool WITH_V, int STAGE_BYTES, int TK = kTileKeys, bool WITH_MEAN = false>
__device__ __forceinline__ void produce_tiles(const CUtensorMap *tmK, const CUtensorMap *tmV, const ScanParams &p,
                                              const SeqWork &w, int split, int kvh, int seq, uint32_t ring,
                                              uint32_t full0, uint32_t empty0) {
  constexpr int HALVES = D / 64;
  constexpr int KTILE = TK * D * 2;
  tma_prefetch_desc(tmK);
  if (WITH_V) tma_prefetch_desc(tmV);
  const uint64_t pol = policy_evict_first();
  bool dead = false;
  int stage = 0;
  uint32_t wrapped = 0, phase = 0;                 // phase = parity of the ring round being refilled
  const int boxes_per_tile = TK / p.box_tok;
  const int page_mask = (1 << p.page_shift) - 1;
  for (TileCursor k = cursor_begin(w, split); cursor_valid(k, w); cursor_next(k, w, p.num_splits)) {
    if (wrapped && !mbar_wait(empty0 + 8u * stage, phase ^ 1u, dead)) break;
    const int tok0 = k.t * TK;
    const int nbox = min(boxes_per_tile, (w.n - tok0 + p.box_tok - 1) / p.box_tok);
    const uint32_t full = full0 + 8u * stage;
    const int nmean = WITH_MEAN ? min(TK / 64, (w.n - tok0 + 63) / 64) : 0;
    mbar_expect_tx(full, nbox * p.box_tok * D * 2 * (WITH_V ? 2 : 1) + nmean * D * 2);
    const uint32_t kdst = ring + stage * STAGE_BYTES;
    if (WITH_MEAN) {
      const __nv_bfloat16 *m = p.vmean + (long long)seq * p.vm_stride_seq + (long long)(tok0 / 64) * p.vm_stride_block +
                               (long long)kvh * p.vm_stride_head;
      for (int i = 0; i < nmean; ++i)
        bulk_load(kdst + KTILE * (WITH_V ? 2 : 1) + i * (D * 2), m + (long long)i * p.vm_stride_block, D * 2, full);
    }
    const uint32_t vdst = kdst + KTILE;
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
      for (int h = 0; h < HALVES; ++h) {
        const uint32_t o = (h * TK + bx * p.box_tok) * 128;
        tma_load_4d(kdst + o, tmK, full, h * 64, c1, c2, c3, pol);
        if (WITH_V) tma_load_4d(vdst + o, tmV, full, h * 64, c1, c2, c3, pol);
      }
    }
    if (++stage == p.stages) { stage = 0; wrapped = 1u; phase ^= 1u; }
  }
  if (dead) atomicOr(&p.hdr->wait_timeouts, 1u);
}

// Query rows of the block as A-operand fragments, and their references.
template <int D>
struct RowBlock {
  uint32_t qf[D / 16][4];
  float z_lo, z_hi;
  uint32_t dm_lo, dm_hi;       // draft masks of the two rows' requests (all ones without drafts)
  bool rv_lo, rv_hi, two_blocks;
};
template <int D>
__device__ __forceinline__ void load_rows(RowBlock<D> &rb, const ScanParams &p, int seq, int kvh, int lane,
                                          int row0 = 0) {
  const int row_lo = row0 + (lane >> 2), row_hi = row_lo + 8, qcol = (lane & 3) * 2;
  rb.rv_lo = row_lo < p.R;
  rb.rv_hi = row_hi < p.R;
  rb.two_blocks = p.R > row0 + 8;
  const int req_lo = seq * p.stack + row_lo / p.G, head_lo = kvh * p.G + row_lo % p.G;
  const int req_hi = seq * p.stack + row_hi / p.G, head_hi = kvh * p.G + row_hi % p.G;
  const __nv_bfloat16 *ql = p.q + (long long)req_lo * p.q_stride_b + (long long)head_lo * p.q_stride_h;
  const __nv_bfloat16 *qh = p.q + (long long)req_hi * p.q_stride_b + (long long)head_hi * p.q_stride_h;
#pragma unroll
  for (int kk = 0; kk < D / 16; ++kk) {
    const int col = kk * 16 + qcol;
    rb.qf[kk][0] = rb.rv_lo ? *reinterpret_cast<const uint32_t *>(ql + col) : 0u;
    rb.qf[kk][1] = rb.rv_hi ? *reinterpret_cast<const uint32_t *>(qh + col) : 0u;
    rb.qf[kk][2] = rb.rv_lo ? *reinterpret_cast<const uint32_t *>(ql + col + 8) : 0u;
    rb.qf[kk][3] = rb.rv_hi ? *reinterpret_cast<const uint32_t *>(qh + col + 8) : 0u;
  }
  rb.z_lo = rb.rv_lo ? p.z[(long long)req_lo * p.Hq + head_lo] : 0.f;
  rb.z_hi = rb.rv_hi ? p.z[(long long)req_hi * p.Hq + head_hi] : 0.f;
  rb.dm_lo = (p.draft_len && rb.rv_lo) ? p.draft_mask[req_lo] : 0xffffffffu;
  rb.dm_hi = (p.draft_len && rb.rv_hi) ? p.draft_mask[req_hi] : 0xffffffffu;
}

// First draft key of a sequence of n keys (n itself without drafts): keys from here on are masked per request.
__device__ __forceinline__ int draft_start(const ScanParams &p, int n) { return p.draft_len ? n - p.draft_len : n; }
// Is key `key` (>= 0) usable under mask dm, the drafts starting at key dstart?
__device__ __forceinline__ bool draft_ok(uint32_t dm, int key, int dstart) {
  const int t = key - dstart;
  return t < 0 || t > 31 || ((dm >> t) & 1u);
}

// Score one 16-key slice of the K tile at `kt` against the row block and form the weights.
// Returns the slice's fetch mask (bit k: key k is live for some row); ah / al receive the
// two-term BF16 weights as A-operand fragments of the value product; l_lo / l_hi accumulate
// this thread's share of L.
// TAIL: c_lo / c_hi also accumulate the weight of this thread's cut keys for its two rows (block tail).
template <int D, bool GATED, bool TAIL = false>
__device__ __forceinline__ uint32_t score_slice(const RowBlock<D> &rb, uint32_t kt, int warp, int lane, int key0,
                                                int n, float scale_log2, float neg_T, uint32_t (&ah)[4],
                                                uint32_t (&al)[4], float &l_lo, float &l_hi, float *c_lo = nullptr,
                                                float *c_hi = nullptr, int dstart = 0x7fffffff) {
  // S[rows, 16 keys] = Q K^T.  Lane l addresses key row (l>>4)*8 + (l&7), 16-byte chunk 2*kk + ((l>>3)&1)
  // of the tile laid out [half][key][128 B] with the 128-byte swizzle.
  const int k_key = warp * 16 + ((lane >> 4) << 3) + (lane & 7);
  const uint32_t k_row = k_key * 128, k_x = ((lane >> 3) & 1) ^ (k_key & 7);
  float s[2][4];
#pragma unroll
  for (int i = 0; i < 4; ++i) s[0][i] = s[1][i] = 0.f;
#pragma unroll
  for (int kk = 0; kk < D / 16; ++kk) {
    uint32_t b0, b1, b2, b3;
    ldsm_x4(kt + (kk >> 2) * (kTileKeys * 128) + k_row + ((((2 * kk) & 7) ^ k_x) << 4), b0, b1, b2, b3);
    mma_bf16(s[0], rb.qf[kk], b0, b1);
    mma_bf16(s[1], rb.qf[kk], b2, b3);
  }
  const int qcol = (lane & 3) * 2;
  if (key0 + 16 > dstart) {                                  // draft keys: a row only uses the ones its mask names
#pragma unroll
    for (int nt = 0; nt < 2; ++nt)
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const int key = key0 + nt * 8 + qcol + e;
        if (!draft_ok(rb.dm_lo, key, dstart)) s[nt][e] = -INFINITY;
        if (!draft_ok(rb.dm_hi, key, dstart)) s[nt][2 + e] = -INFINITY;
      }
  }
  uint32_t livemask = 0;
  ah[0] = ah[1] = ah[2] = ah[3] = 0u;
  al[0] = al[1] = al[2] = al[3] = 0u;
#pragma unroll
  for (int nt = 0; nt < 2; ++nt) {
#pragma unroll
    for (int blk = 0; blk < 2; ++blk) {
      if (blk == 1 && !rb.two_blocks) continue;
      float pw[2], pm[2];
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const int kk16 = nt * 8 + qcol + e;
        const bool ok = ((key0 + kk16) < n) && (blk ? rb.rv_hi : rb.rv_lo);
        const float x = ok ? fmaf(s[nt][2 * blk + e], scale_log2, blk ? -rb.z_hi : -rb.z_lo) : -INFINITY;
        const bool live = GATED ? (x >= neg_T) : ok;         // dense: every valid key is live
        pw[e] = ex2_approx(x);                               // 2^-inf = 0 for masked keys
        pm[e] = live ? pw[e] : 0.f;
        if (live) livemask |= 1u << kk16;
      }
      // two-term BF16 split of the live weights; L sums the weights the products use, cut keys add p
      const uint32_t hi2 = pack_bf16(pm[0], pm[1]);
      const float h0 = __uint_as_float(hi2 << 16), h1 = __uint_as_float(hi2 & 0xffff0000u);
      const uint32_t lo2 = pack_bf16(pm[0] - h0, pm[1] - h1);
      const float g0 = __uint_as_float(lo2 << 16), g1 = __uint_as_float(lo2 & 0xffff0000u);
      const float add = ((h0 + g0) + (pw[0] - pm[0])) + ((h1 + g1) + (pw[1] - pm[1]));
      if (blk) l_hi += add; else l_lo += add;
      if (TAIL) {
        const float cut = (pw[0] - pm[0]) + (pw[1] - pm[1]);
        if (blk) *c_hi += cut; else *c_lo += cut;
      }
      ah[nt * 2 + blk] = hi2;
      al[nt * 2 + blk] = lo2;
    }
  }
  return __reduce_or_sync(0xffffffffu, livemask);            // verdicts ORed over the row block
}

// A += P_hi V + P_lo V for one slice.  SWIZZLED: V rows sit in a TMA tile ([half][key][128 B], swizzled)
// of HALF_ROWS rows per half, starting at row `row0`; otherwise in padded rows of ROW_BYTES.
template <int D, bool SWIZZLED, int ROW_BYTES, int HALF_ROWS = kTileKeys>
__device__ __forceinline__ void value_product(float (&o)[D / 8][4], uint32_t vbase, int row0, int lane,
                                              const uint32_t (&ah)[4], const uint32_t (&al)[4]) {
  const int v_key = ((lane >> 3) & 1) * 8 + (lane & 7);      // key row this lane addresses (ldmatrix.trans)
  const uint32_t sw_row = (row0 + v_key) * 128, sw_x = (lane >> 4) ^ (v_key & 7);
  const uint32_t pad_off = v_key * ROW_BYTES + (lane >> 4) * 16;
#pragma unroll
  for (int pr = 0; pr < D / 16; ++pr) {
    uint32_t b0, b1, b2, b3;
    if (SWIZZLED) ldsm_x4_trans(vbase + (pr >> 2) * (HALF_ROWS * 128) + sw_row + ((((2 * pr) & 7) ^ sw_x) << 4), b0, b1, b2, b3);
    else ldsm_x4_trans(vbase + pad_off + pr * 32, b0, b1, b2, b3);
    mma_bf16(o[2 * pr], ah, b0, b1);
    mma_bf16(o[2 * pr], al, b0, b1);
    mma_bf16(o[2 * pr + 1], ah, b2, b3);
    mma_bf16(o[2 * pr + 1], al, b2, b3);
  }
}

// Block tail for rows-on-M accumulators: o[nt] holds rows lane/4 (elements 0, 1) and lane/4 + 8 (elements 2, 3),
// channels 8 nt + (lane%4)*2 + {0,1}.  c_lo / c_hi: the two rows' cut mass; mean: the block's mean value row.
template <int D>
__device__ __forceinline__ void tail_update(float (&o)[D / 8][4], float c_lo, float c_hi, const __nv_bfloat16 *mean, int lane) {
  const uint32_t *m2 = reinterpret_cast<const uint32_t *>(mean) + (lane & 3);
#pragma unroll
  for (int nt = 0; nt < D / 8; ++nt) {
    const uint32_t w = m2[nt * 4];
    const float m0 = __uint_as_float(w << 16), m1 = __uint_as_float(w & 0xffff0000u);
    o[nt][0] = fmaf(c_lo, m0, o[nt][0]); o[nt][1] = fmaf(c_lo, m1, o[nt][1]);
    o[nt][2] = fmaf(c_hi, m0, o[nt][2]); o[nt][3] = fmaf(c_hi, m1, o[nt][3]);
  }
}

// ------------------------------------------------------------------------------------------------
// Narrow row blocks (at most 8 query rows per (sequence, kv head): every GQA group up to 8).
// The products are turned round -- keys, then channels, on M and the query rows on N = 8 -- as
// Algorithm 1 has them: half the MMAs and half the accumulator registers of the rows-on-M form.
//   scores   S^T[16 keys, 8 rows] = K[16, D] Q^T            (A = K slice by ldmatrix, B = Q registers)
//   values   A^T[D, 8 rows]      += V^T[D, 16 keys] P^T      (A = V slice by ldmatrix.trans, B = P^T)
// P^T comes out of the score fragment by one movmatrix per 8x8 block.
template <int D>
struct RowBlockN {
  uint32_t qb[D / 16][2];      // B fragments: row lane/4, channels kk*16 + (lane%4)*2 + {0,1} (+8)
  float z0, z1;                // references of the two rows this thread's score fragment holds: (lane%4)*2 + {0,1}
  uint32_t dm0, dm1;           // their requests' draft masks (all ones without drafts)
  bool v0, v1;
};
// `row0`: first row of this 8-row N tile within the (sequence, kv head)'s row block (0, or 8 for the second tile).
template <int D>
__device__ __forceinline__ void load_rows_n(RowBlockN<D> &rb, const ScanParams &p, int seq, int kvh, int lane, int row0 = 0) {
  {
    const int r = row0 + (lane >> 2);                         // the row this lane feeds as B operand
    const bool ok = r < p.R;
    const int req = seq * p.stack + r / p.G, head = kvh * p.G + r % p.G;
    const __nv_bfloat16 *q = p.q + (long long)req * p.q_stride_b + (long long)head * p.q_stride_h + (lane & 3) * 2;
#pragma unroll
    for (int kk = 0; kk < D / 16; ++kk) {
      rb.qb[kk][0] = ok ? *reinterpret_cast<const uint32_t *>(q + kk * 16) : 0u;
      rb.qb[kk][1] = ok ? *reinterpret_cast<const uint32_t *>(q + kk * 16 + 8) : 0u;
    }
  }
  const int r0 = row0 + (lane & 3) * 2;                       // the rows this lane holds scores of
  rb.v0 = r0 < p.R;
  rb.v1 = r0 + 1 < p.R;
  const int req0 = seq * p.stack + r0 / p.G, head0 = kvh * p.G + r0 % p.G;
  const int req1 = seq * p.stack + (r0 + 1) / p.G, head1 = kvh * p.G + (r0 + 1) % p.G;
  rb.z0 = rb.v0 ? p.z[(long long)req0 * p.Hq + head0] : 0.f;
  rb.z1 = rb.v1 ? p.z[(long long)req1 * p.Hq + head1] : 0.f;
  rb.dm0 = (p.draft_len && rb.v0) ? p.draft_mask[req0] : 0xffffffffu;
  rb.dm1 = (p.draft_len && rb.v1) ? p.draft_mask[req1] : 0xffffffffu;
}
// Draft keys of a 16-key sub-slice: scores of keys a row does not use become -inf (weight exactly 0).
template <int D>
__device__ __forceinline__ void mask_drafts_n(const RowBlockN<D> &rb, float (&s)[4], int lane, int key0, int dstart) {
#pragma unroll
  for (int kh = 0; kh < 2; ++kh) {
    const int key = key0 + (lane >> 2) + 8 * kh;
    if (!draft_ok(rb.dm0, key, dstart)) s[2 * kh] = -INFINITY;
    if (!draft_ok(rb.dm1, key, dstart)) s[2 * kh + 1] = -INFINITY;
  }
}

__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a) {
  uint32_t d;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
  return d;
}

// s[0], s[1]: key lane/4, rows (lane%4)*2 + {0,1};  s[2], s[3]: key lane/4 + 8.
template <int D, int TK = kTileKeys>
__device__ __forceinline__ void qk_issue_n(const RowBlockN<D> &rb, uint32_t kt, int slice, int lane, float (&s)[4]) {
  // ldmatrix matrix i = lane/8: keys (i&1)*8 + lane%8 of the slice, 16-byte chunk 2*kk + (i>>1)
  const int k_key = slice * 16 + (((lane >> 3) & 1) << 3) + (lane & 7);
  const uint32_t k_row = k_key * 128, k_x = (lane >> 4) ^ (k_key & 7);
  s[0] = s[1] = s[2] = s[3] = 0.f;
#pragma unroll
  for (int kk = 0; kk < D / 16; ++kk) {
    uint32_t a[4];
    ldsm_x4(kt + (kk >> 2) * (TK * 128) + k_row + ((((2 * kk) & 7) ^ k_x) << 4), a[0], a[1], a[2], a[3]);
    mma_bf16(s, a, rb.qb[kk][0], rb.qb[kk][1]);
  }
}

// The same for NT 8-row N tiles at once: one ldmatrix of the K slice feeds every tile's MMA.
template <int D, int TK, int NT>
__device__ __forceinline__ void qk_issue_nt(const RowBlockN<D> (&rb)[NT], uint32_t kt, int slice, int lane, float (&s)[NT][4]) {
  const int k_key = slice * 16 + (((lane >> 3) & 1) << 3) + (lane & 7);
  const uint32_t k_row = k_key * 128, k_x = (lane >> 4) ^ (k_key & 7);
#pragma unroll
  for (int t = 0; t < NT; ++t) s[t][0] = s[t][1] = s[t][2] = s[t][3] = 0.f;
#pragma unroll
  for (int kk = 0; kk < D / 16; ++kk) {
    uint32_t a[4];
    ldsm_x4(kt + (kk >> 2) * (TK * 128) + k_row + ((((2 * kk) & 7) ^ k_x) << 4), a[0], a[1], a[2], a[3]);
#pragma unroll
    for (int t = 0; t < NT; ++t) mma_bf16(s[t], a, rb[t].qb[kk][0], rb[t].qb[kk][1]);
  }
}

// Final weights of a slice.  Returns the fetch mask; bh / bl receive P_hi^T / P_lo^T as B fragments of the
// value product; l0 / l1 accumulate this thread's share of L for rows (lane%4)*2 + {0,1}.
// TAIL: c0 / c1 also accumulate the weight of this thread's cut keys (the block tail's virtual row, Algorithm 1).
template <int D, bool GATED, bool TAIL = false>
__device__ __forceinline__ uint32_t weights_n(const RowBlockN<D> &rb, const float (&s)[4], int lane, int key0, int n,
                                              float scale_log2, float neg_T, uint32_t (&bh)[2], uint32_t (&bl)[2],
                                              float &l0, float &l1, float *c0 = nullptr, float *c1 = nullptr) {
  const int klo = lane >> 2;
  uint32_t livemask = 0;
#pragma unroll
  for (int kh = 0; kh < 2; ++kh) {                            // key lane/4, then key lane/4 + 8
    const bool kvalid = (key0 + klo + 8 * kh) < n;
    float pw[2], pm[2];
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      const bool ok = kvalid && (e ? rb.v1 : rb.v0);
      const float x = ok ? fmaf(s[2 * kh + e], scale_log2, e ? -rb.z1 : -rb.z0) : -INFINITY;
      const bool live = GATED ? (x >= neg_T) : ok;
      pw[e] = ex2_approx(x);
      pm[e] = live ? pw[e] : 0.f;
      if (live) livemask |= 1u << (klo + 8 * kh);
    }
    const uint32_t hi2 = pack_bf16(pm[0], pm[1]);
    const float h0 = __uint_as_float(hi2 << 16), h1 = __uint_as_float(hi2 & 0xffff0000u);
    const uint32_t lo2 = pack_bf16(pm[0] - h0, pm[1] - h1);
    const float g0 = __uint_as_float(lo2 << 16), g1 = __uint_as_float(lo2 & 0xffff0000u);
    l0 += (h0 + g0) + (pw[0] - pm[0]);
    l1 += (h1 + g1) + (pw[1] - pm[1]);
    if (TAIL) { *c0 += pw[0] - pm[0]; *c1 += pw[1] - pm[1]; }
    bh[kh] = movmatrix_trans(hi2);                            // [key][row] block -> [row][key]: the B fragment
    bl[kh] = movmatrix_trans(lo2);
  }
  return __reduce_or_sync(0xffffffffu, livemask);
}

// A^T += V^T (P_hi^T + P_lo^T) for one slice; o[mt]: channels 16*mt + lane/4 (+8), rows (lane%4)*2 + {0,1}.
template <int D, bool SWIZZLED, int ROW_BYTES, int HALF_ROWS = kTileKeys>
__device__ __forceinline__ void value_product_n(float (&o)[D / 16][4], uint32_t vbase, int row0, int lane,
                                                const uint32_t (&bh)[2], const uint32_t (&bl)[2]) {
  // ldmatrix.trans matrix i = lane/8: keys (i>>1)*8 + lane%8, 16-byte chunk 2*mt + (i&1)
  const int v_key = ((lane >> 4) << 3) + (lane & 7);
  const uint32_t sw_row = (row0 + v_key) * 128, sw_x = ((lane >> 3) & 1) ^ (v_key & 7);
  const uint32_t pad_off = v_key * ROW_BYTES + ((lane >> 3) & 1) * 16;
#pragma unroll
  for (int mt = 0; mt < D / 16; ++mt) {
    uint32_t a[4];
    if (SWIZZLED) ldsm_x4_trans(vbase + (mt >> 2) * (HALF_ROWS * 128) + sw_row + ((((2 * mt) & 7) ^ sw_x) << 4), a[0], a[1], a[2], a[3]);
    else ldsm_x4_trans(vbase + pad_off + mt * 32, a[0], a[1], a[2], a[3]);
    mma_bf16(o[mt], a, bh[0], bh[1]);
    mma_bf16(o[mt], a, bl[0], bl[1]);
  }
}

// The same for NT N tiles: one ldmatrix.trans of the V slice feeds every tile's MMAs.
template <int D, int HALF_ROWS, int NT>
__device__ __forceinline__ void value_product_nt(float (&o)[NT][D / 16][4], uint32_t vbase, int row0, int lane,
                                                 const uint32_t (&bh)[NT][2], const uint32_t (&bl)[NT][2], uint32_t skip) {
  const int v_key = ((lane >> 4) << 3) + (lane & 7);
  const uint32_t sw_row = (row0 + v_key) * 128, sw_x = ((lane >> 3) & 1) ^ (v_key & 7);
#pragma unroll
  for (int mt = 0; mt < D / 16; ++mt) {
    uint32_t a[4];
    ldsm_x4_trans(vbase + (mt >> 2) * (HALF_ROWS * 128) + sw_row + ((((2 * mt) & 7) ^ sw_x) << 4), a[0], a[1], a[2], a[3]);
#pragma unroll
    for (int t = 0; t < NT; ++t) {
      if ((skip >> t) & 1u) continue;                        // no key of the slice is live for this tile's rows
      mma_bf16(o[t][mt], a, bh[t][0], bh[t][1]);
      mma_bf16(o[t][mt], a, bl[t][0], bl[t][1]);
    }
  }
}

// Chunk end for narrow blocks: park the warp's partial as [row][channel], add the warps in order, store.
template <int D, int WARPS>
__device__ __forceinline__ void reduce_store_A_n(float (&o)[D / 16][4], float *red, float *slot, int R, int warp,
                                                 int lane, int tid, int bar_id) {
  const int r0 = (lane & 3) * 2, c0 = lane >> 2;
  float *mine = red + warp * R * D;
#pragma unroll
  for (int mt = 0; mt < D / 16; ++mt) {
    if (r0 < R) { mine[r0 * D + mt * 16 + c0] = o[mt][0]; mine[r0 * D + mt * 16 + c0 + 8] = o[mt][2]; }
    if (r0 + 1 < R) { mine[(r0 + 1) * D + mt * 16 + c0] = o[mt][1]; mine[(r0 + 1) * D + mt * 16 + c0 + 8] = o[mt][3]; }
    o[mt][0] = o[mt][1] = o[mt][2] = o[mt][3] = 0.f;
  }
  named_bar(bar_id, WARPS * 32);
  const int RD = R * D;
  for (int i = tid; i < RD; i += WARPS * 32) {
    float v = red[i];
#pragma unroll
    for (int wv = 1; wv < WARPS; ++wv) v += red[wv * RD + i];
    slot[i] = v;
  }
  named_bar(bar_id, WARPS * 32);
}
// The same for four warps in a quarter of the room: warps 2, 3 park in fragment order, warps 0, 1 take them
// in; warp 1 parks, warp 0 takes it in and stores:  (w0 + w2) + (w1 + w3), always in this order.
template <int D>
__device__ __forceinline__ void tree_store_A_n(float (&o)[D / 16][4], float *park, float *slot, int R, int warp,
                                               int lane, int bar_id) {
  constexpr int kPerWarp = D / 16 * 4 * 32;
  if (warp >= 2) {
#pragma unroll
    for (int mt = 0; mt < D / 16; ++mt)
#pragma unroll
      for (int j = 0; j < 4; ++j) park[(warp - 2) * kPerWarp + (mt * 4 + j) * 32 + lane] = o[mt][j];
  }
  named_bar(bar_id, 128);
  if (warp < 2) {
#pragma unroll
    for (int mt = 0; mt < D / 16; ++mt)
#pragma unroll
      for (int j = 0; j < 4; ++j) o[mt][j] += park[warp * kPerWarp + (mt * 4 + j) * 32 + lane];
  }
  named_bar(bar_id, 128);
  if (warp == 1) {
#pragma unroll
    for (int mt = 0; mt < D / 16; ++mt)
#pragma unroll
      for (int j = 0; j < 4; ++j) park[(mt * 4 + j) * 32 + lane] = o[mt][j];
  }
  named_bar(bar_id, 128);
  if (warp == 0) {
    const int r0 = (lane & 3) * 2, c0 = lane >> 2;
#pragma unroll
    for (int mt = 0; mt < D / 16; ++mt) {
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int r = r0 + (j & 1);
        const float v = o[mt][j] + park[(mt * 4 + j) * 32 + lane];
        if (r < R) slot[r * D + mt * 16 + c0 + (j >> 1) * 8] = v;
      }
    }
  }
#pragma unroll
  for (int mt = 0; mt < D / 16; ++mt) o[mt][0] = o[mt][1] = o[mt][2] = o[mt][3] = 0.f;
  named_bar(bar_id, 128);
}
template <int WARPS>
__device__ __forceinline__ void reduce_store_L_n(float &l0, float &l1, float *redl, float *slot_l, int R, int warp,
                                                 int lane, int tid, int bar_id) {
#pragma unroll
  for (int m = 4; m <= 16; m <<= 1) {
    l0 += __shfl_xor_sync(0xffffffffu, l0, m);
    l1 += __shfl_xor_sync(0xffffffffu, l1, m);
  }
  const int r0 = (lane & 3) * 2;
  if (lane < 4) {
    if (r0 < R) redl[warp * kMaxRows + r0] = l0;
    if (r0 + 1 < R) redl[warp * kMaxRows + r0 + 1] = l1;
  }
  l0 = l1 = 0.f;
  named_bar(bar_id, WARPS * 32);
  if (tid < R) {
    float v = redl[tid];
#pragma unroll
    for (int wv = 1; wv < WARPS; ++wv) v += redl[wv * kMaxRows + tid];
    slot_l[tid] = v;
  }
  named_bar(bar_id, WARPS * 32);
}

// ------------------------------------------------------------------------------------------------
// Dense decode (T = inf)
template <int D>
__global__ void __launch_bounds__(kDenseThreads, 2)
fold_scan_dense_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                       const ScanParams p) {
  constexpr int TK = narrow_tile_keys<D>();                        // keys per tile
  constexpr int U = TK / 64, KS = 16 * U;                          // 16-key sub-slices and keys per warp slice
  using LO = DenseLayout<D, TK>;
  constexpr int C16 = D / 8;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t *gen = smem_raw + (base - raw);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // kv heads fastest: CTAs that run together read the same tokens' rows, which sit side by side in memory
  const int kvh = blockIdx.x, split = blockIdx.y, seq = blockIdx.z;
  const SeqWork w = seq_work<TK>(p, seq);
  if (split >= w.n_chunks) return;
  const int stages = p.stages, R = p.R, n = w.n;
  const int dstart = draft_start(p, n);                     // keys from here on are per-request drafts
  const uint32_t full0 = base + LO::off_bar(stages, R), empty0 = full0 + 8u * stages;

  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) {
      mbar_init(full0 + 8u * s, 1);
      mbar_init(empty0 + 8u * s, kConsumerWarps);
    }
    mbar_fence_init();
  }
  __syncthreads();
  pdl_launch_dependents();
  if (warp == kConsumerWarps) {                              // the tiles depend on nothing the reference kernel writes:
    if (lane == 0) produce_tiles<D, true, LO::kStage, TK>(&tmK, &tmV, p, w, split, kvh, seq, base, full0, empty0);
    return;                                                  // the ring fills while that kernel drains
  }
  pdl_wait();                                                // z comes from the kernel before

  RowBlockN<D> rb;                                           // rows on N: see "Narrow row blocks"
  load_rows_n<D>(rb, p, seq, kvh, lane);
  float o[D / 16][4];
#pragma unroll
  for (int i = 0; i < D / 16; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
  float l_lo = 0.f, l_hi = 0.f;
  float *red = reinterpret_cast<float *>(gen + LO::off_red(stages));
  float *redl = reinterpret_cast<float *>(gen + LO::off_redl(stages, R));

  bool dead = false;
  int stage = 0;
  uint32_t phase = 0;
  unsigned long long st_total = 0;

  for (int c = split; c < w.n_chunks; c += p.num_splits) {
    const int t_end = min((c + 1) * w.ctiles, w.n_tiles);
    for (int t = c * w.ctiles; t < t_end; ++t) {
      const int my_stage = stage;
      const bool ready = mbar_wait(full0 + 8u * my_stage, phase, dead);
      if (++stage == stages) { stage = 0; phase ^= 1u; }
      if (!ready) continue;
      const uint32_t kt = base + my_stage * LO::kStage;
      const int key0 = t * TK + warp * KS;
      st_total += min(KS, max(0, n - key0));
      if (key0 + KS > n) {                                   // ragged tail: value rows past n may hold anything
        for (int r = 0; r < KS; ++r)
          if (key0 + r >= n && lane < C16)
            *reinterpret_cast<uint4 *>(gen + my_stage * LO::kStage + LO::kKTile +
                                       tile_off(warp * KS + r, lane, TK)) = make_uint4(0, 0, 0, 0);
        __syncwarp();
      }
#pragma unroll
      for (int u = 0; u < U; ++u) {
        float s[4];
        uint32_t bh[2], bl[2];
        qk_issue_n<D, TK>(rb, kt, warp * U + u, lane, s);
        if (key0 + 16 * u + 16 > dstart) mask_drafts_n<D>(rb, s, lane, key0 + 16 * u, dstart);
        const uint32_t fetch16 = weights_n<D, false>(rb, s, lane, key0 + 16 * u, n, p.scale_log2, p.neg_T, bh, bl, l_lo, l_hi);
        if (fetch16 != 0) value_product_n<D, true, 0, TK>(o, kt + LO::kKTile, (warp * U + u) * 16, lane, bh, bl);
      }
      if (key0 + KS > n) fence_proxy_async_smem();           // generic writes before the next TMA fill
      __syncwarp();
      if (lane == 0) mbar_arrive(empty0 + 8u * my_stage);
    }
    float *slot = p.slots + (((long long)seq * p.Hkv + kvh) * p.max_slots + c) * p.slot_stride;
    reduce_store_L_n<kConsumerWarps>(l_lo, l_hi, redl, slot + R * D, R, warp, lane, threadIdx.x, 1);
    reduce_store_A_n<D, kConsumerWarps>(o, red, slot, R, warp, lane, threadIdx.x, 1);
  }

  if (lane == 0) {
    if (dead) atomicOr(&p.hdr->wait_timeouts, 2u);
    atomicAdd(reinterpret_cast<unsigned long long *>(&p.hdr->v_rows_fetched), st_total);
    atomicAdd(reinterpret_cast<unsigned long long *>(&p.hdr->v_rows_total), st_total);
  }
}

// ------------------------------------------------------------------------------------------------
// Dense decode for row blocks of 9..16 rows: the rows-on-N form with two 8-row N tiles per warp.  A warp still
// owns slice w of every tile; each ldmatrix of keys or values feeds both tiles' MMAs.
template <int D>
struct DenseWideLayout {
  static constexpr int kTK = narrow_tile_keys<D>();
  static constexpr int kKTile = kTK * D * 2;
  static constexpr int kStage = 2 * kKTile;                    // K tile then V tile
  static constexpr int kPark = D / 16 * 4 * 32 * 4;            // one warp's accumulators of one N tile, fragment order
  __host__ __device__ static int off_park(int stages) { return stages * kStage; }
  __host__ __device__ static int off_redl(int stages) { return off_park(stages) + 2 * kPark; }
  __host__ __device__ static int off_bar(int stages) { return off_redl(stages) + kConsumerWarps * kMaxRows * 4; }
  __host__ __device__ static int total(int stages) { return off_bar(stages) + 2 * stages * 8 + 1024; }
};

template <int D>
__global__ void __launch_bounds__(kDenseThreads, 2)
fold_scan_dense_nt2_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                           const ScanParams p) {
  using LO = DenseWideLayout<D>;
  constexpr int TK = LO::kTK, U = TK / 64, KS = 16 * U, NT = 2, C16 = D / 8;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t *gen = smem_raw + (base - raw);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // x = row group + row_groups * kv head: the 16-row groups of a kv head sit side by side and share its tiles in L2
  const int rg = blockIdx.x % p.row_groups, kvh = blockIdx.x / p.row_groups, split = blockIdx.y, seq = blockIdx.z;
  const int rbase = rg * 16;                                 // first row of this CTA's group
  const SeqWork w = seq_work<TK>(p, seq);
  if (split >= w.n_chunks) return;
  const int stages = p.stages, R = p.R, n = w.n;
  const int dstart = draft_start(p, n);
  const uint32_t full0 = base + LO::off_bar(stages), empty0 = full0 + 8u * stages;

  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) {
      mbar_init(full0 + 8u * s, 1);
      mbar_init(empty0 + 8u * s, kConsumerWarps);
    }
    mbar_fence_init();
  }
  __syncthreads();
  pdl_launch_dependents();
  if (warp == kConsumerWarps) {                              // the tiles depend on nothing the reference kernel writes:
    if (lane == 0) produce_tiles<D, true, LO::kStage, TK>(&tmK, &tmV, p, w, split, kvh, seq, base, full0, empty0);
    return;                                                  // the ring fills while that kernel drains
  }
  pdl_wait();                                                // z comes from the kernel before

  RowBlockN<D> rb[NT];
#pragma unroll
  for (int t = 0; t < NT; ++t) load_rows_n<D>(rb[t], p, seq, kvh, lane, rbase + 8 * t);
  float o[NT][D / 16][4];
#pragma unroll
  for (int t = 0; t < NT; ++t)
#pragma unroll
    for (int i = 0; i < D / 16; ++i) o[t][i][0] = o[t][i][1] = o[t][i][2] = o[t][i][3] = 0.f;
  float l0[NT] = {0.f, 0.f}, l1[NT] = {0.f, 0.f};
  float *park = reinterpret_cast<float *>(gen + LO::off_park(stages));
  float *redl = reinterpret_cast<float *>(gen + LO::off_redl(stages));

  bool dead = false;
  int stage = 0;
  uint32_t phase = 0;
  unsigned long long st_total = 0;

  for (int c = split; c < w.n_chunks; c += p.num_splits) {
    const int t_end = min((c + 1) * w.ctiles, w.n_tiles);
    for (int t = c * w.ctiles; t < t_end; ++t) {
      const int my_stage = stage;
      const bool ready = mbar_wait(full0 + 8u * my_stage, phase, dead);
      if (++stage == stages) { stage = 0; phase ^= 1u; }
      if (!ready) continue;
      const uint32_t kt = base + my_stage * LO::kStage;
      const int key0 = t * TK + warp * KS;
      st_total += min(KS, max(0, n - key0));
      if (key0 + KS > n) {                                   // ragged tail: value rows past n may hold anything
        for (int r = 0; r < KS; ++r)
          if (key0 + r >= n && lane < C16)
            *reinterpret_cast<uint4 *>(gen + my_stage * LO::kStage + LO::kKTile +
                                       tile_off(warp * KS + r, lane, TK)) = make_uint4(0, 0, 0, 0);
        __syncwarp();
      }
#pragma unroll
      for (int u = 0; u < U; ++u) {
        float s[NT][4];
        uint32_t bh[NT][2], bl[NT][2];
        qk_issue_nt<D, TK, NT>(rb, kt, warp * U + u, lane, s);
        uint32_t skip = 0;
#pragma unroll
        for (int q = 0; q < NT; ++q) {
          if (key0 + 16 * u + 16 > dstart) mask_drafts_n<D>(rb[q], s[q], lane, key0 + 16 * u, dstart);
          const uint32_t live = weights_n<D, false>(rb[q], s[q], lane, key0 + 16 * u, n, p.scale_log2, p.neg_T, bh[q], bl[q],
                                                    l0[q], l1[q]);
          skip |= live ? 0u : (1u << q);
        }
        if (skip != (1u << NT) - 1u) value_product_nt<D, TK, NT>(o, kt + LO::kKTile, (warp * U + u) * 16, lane, bh, bl, skip);
      }
      if (key0 + KS > n) fence_proxy_async_smem();           // generic writes before the next TMA fill
      __syncwarp();
      if (lane == 0) mbar_arrive(empty0 + 8u * my_stage);
    }
    float *slot = p.slots + (((long long)seq * p.Hkv + kvh) * p.max_slots + c) * p.slot_stride;
#pragma unroll
    for (int q = 0; q < NT; ++q) {
      const int rows = min(8, R - rbase - 8 * q);            // 8, then what is left (possibly none)
      reduce_store_L_n<kConsumerWarps>(l0[q], l1[q], redl, slot + R * D + rbase + 8 * q, rows, warp, lane, threadIdx.x, 1);
      tree_store_A_n<D>(o[q], park, slot + (rbase + 8 * q) * D, rows, warp, lane, 1);
    }
  }

  if (lane == 0) {
    if (dead) atomicOr(&p.hdr->wait_timeouts, 2u);
    atomicAdd(reinterpret_cast<unsigned long long *>(&p.hdr->v_rows_fetched), st_total);
    atomicAdd(reinterpret_cast<unsigned long long *>(&p.hdr->v_rows_total), st_total);
  }
}

// ------------------------------------------------------------------------------------------------
// Stacked rows (more than 16 query rows per (sequence, kv head): the shared-prefix level of a
// cascade, Section 4 "Value product" / Appendix "Tile layouts").  K and V tiles arrive together by
// TMA as in dense decode -- with this many rows every key is live for some row, so nothing can be
// skipped -- and each of the four consumer warps owns a 16-row block and walks all four slices of
// every tile.  A CTA covers 64 rows; CTAs of the same tile stream share it through L2.  The depth
// gate still applies row by row.  Each warp writes its own rows of the chunk slot: no cross-warp add.
// TAIL (with GATED): the tile's block-mean row rides behind the V tile; a warp sums its rows' cut mass over the tile
// (= one 64-key block) and adds cut mass x mean once per tile.
template <int D, bool GATED, bool TAIL = false>
__global__ void __launch_bounds__(kDenseThreads, 2)
fold_scan_stacked_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                         const ScanParams p) {
  using LO = DenseLayout<D>;
  constexpr int C16 = D / 8;
  constexpr int STAGE = LO::kStage + (TAIL ? 1024 : 0);      // K tile, V tile (, the block's mean row)
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t *gen = smem_raw + (base - raw);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int row_groups = (p.R + 63) / 64;
  const int rg = blockIdx.x % row_groups, split = blockIdx.x / row_groups;
  const int kvh = blockIdx.y, seq = blockIdx.z;
  const SeqWork w = seq_work(p, seq);
  if (split >= w.n_chunks) return;
  const int stages = p.stages, R = p.R, n = w.n;
  const int dstart = draft_start(p, n);                     // keys from here on are per-request drafts
  // the ring's stages are STAGE bytes apart; what follows it keeps its place relative to the ring's end
  const uint32_t full0 = base + stages * (STAGE - LO::kStage) + LO::off_bar(stages, 0), empty0 = full0 + 8u * stages;

  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) {
      mbar_init(full0 + 8u * s, 1);
      mbar_init(empty0 + 8u * s, kConsumerWarps);
    }
    mbar_fence_init();
  }
  __syncthreads();
  pdl_launch_dependents();
  pdl_wait();

  if (warp == kConsumerWarps) {
    if (lane == 0) produce_tiles<D, true, STAGE, kTileKeys, TAIL>(&tmK, &tmV, p, w, split, kvh, seq, base, full0, empty0);
    return;
  }

  const int row0 = rg * 64 + warp * 16;
  RowBlock<D> rb;
  load_rows<D>(rb, p, seq, kvh, lane, row0);
  float o[D / 8][4];
#pragma unroll
  for (int i = 0; i < D / 8; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
  float l_lo = 0.f, l_hi = 0.f;
  bool dead = false;
  int stage = 0;
  uint32_t phase = 0;

  for (TileCursor k = cursor_begin(w, split); cursor_valid(k, w);) {
    const int my_stage = stage;
    const bool ready = mbar_wait(full0 + 8u * my_stage, phase, dead);
    if (++stage == stages) { stage = 0; phase ^= 1u; }
    if (ready) {
      const uint32_t kt = base + my_stage * STAGE;
      if (k.t * kTileKeys + kTileKeys > n) {                 // ragged tail: value rows past n may hold anything
        // every warp reads every row: warp w clears the rows of slice w, then all four meet
        for (int r = 0; r < 16; ++r)
          if (k.t * kTileKeys + warp * 16 + r >= n && lane < C16)
            *reinterpret_cast<uint4 *>(gen + my_stage * STAGE + LO::kKTile +
                                       tile_off(warp * 16 + r, lane, kTileKeys)) = make_uint4(0, 0, 0, 0);
        named_bar(1);
      }
      float c_lo = 0.f, c_hi = 0.f;                          // this tile's cut mass of the thread's two rows
#pragma unroll 1
      for (int sl = 0; sl < 4; ++sl) {
        const int key0 = k.t * kTileKeys + sl * 16;
        if (key0 >= n) break;
        uint32_t ah[4], al[4];
        const uint32_t live16 = score_slice<D, GATED, TAIL>(rb, kt, sl, lane, key0, n, p.scale_log2, p.neg_T, ah, al, l_lo,
                                                              l_hi, &c_lo, &c_hi, dstart);
        if (live16 != 0) value_product<D, true, 0>(o, kt + LO::kKTile, sl * 16, lane, ah, al);
      }
      if (TAIL) {
        c_lo += __shfl_xor_sync(0xffffffffu, c_lo, 1); c_lo += __shfl_xor_sync(0xffffffffu, c_lo, 2);
        c_hi += __shfl_xor_sync(0xffffffffu, c_hi, 1); c_hi += __shfl_xor_sync(0xffffffffu, c_hi, 2);
        if (__any_sync(0xffffffffu, c_lo > 0.f || c_hi > 0.f))
          tail_update<D>(o, c_lo, c_hi, reinterpret_cast<const __nv_bfloat16 *>(gen + my_stage * STAGE + LO::kStage), lane);
      }
      if (k.t * kTileKeys + kTileKeys > n) fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(empty0 + 8u * my_stage);
    }
    const int c_done = k.c;
    if (cursor_next(k, w, p.num_splits)) {
      // this warp owns its rows of the slot outright
      float *slot = p.slots + (((long long)seq * p.Hkv + kvh) * p.max_slots + c_done) * p.slot_stride;
      const int r_lo = row0 + (lane >> 2), r_hi = r_lo + 8, qcol = (lane & 3) * 2;
#pragma unroll
      for (int nt = 0; nt < D / 8; ++nt) {
        if (r_lo < R) *reinterpret_cast<float2 *>(slot + (long long)r_lo * D + nt * 8 + qcol) = make_float2(o[nt][0], o[nt][1]);
        if (r_hi < R) *reinterpret_cast<float2 *>(slot + (long long)r_hi * D + nt * 8 + qcol) = make_float2(o[nt][2], o[nt][3]);
        o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.f;
      }
      l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1);
      l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
      l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1);
      l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
      if ((lane & 3) == 0) {
        if (r_lo < R) slot[(long long)R * D + r_lo] = l_lo;
        if (r_hi < R) slot[(long long)R * D + r_hi] = l_hi;
      }
      l_lo = l_hi = 0.f;
    }
  }
  if (lane == 0 && dead) atomicOr(&p.hdr->wait_timeouts, 2u);
  if (threadIdx.x == 0 && rg == 0) {                          // every value row is read once per row group pass
    unsigned long long keys = 0;
    for (int c = split; c < w.n_chunks; c += p.num_splits)
      keys += min((c + 1) * w.ctiles * kTileKeys, n) - c * w.ctiles * kTileKeys;
    atomicAdd(reinterpret_cast<unsigned long long *>(&p.hdr->v_rows_fetched), keys);
    atomicAdd(reinterpret_cast<unsigned long long *>(&p.hdr->v_rows_total), keys);
  }
}

// ------------------------------------------------------------------------------------------------
// Depth-gated decode for narrow row blocks (at most 8 rows): the same roles with the products turned
// round (rows on N), which halves the MMAs and the accumulator registers.  Value slices always sit in
// the swizzled box layout, whichever way they were fetched.
// TAIL (block tail of Section 4 "Depth as a dial", mean only): a row's cut keys add their summed weight times
// the mean value row of their 64-key block.  The mean rows ride with the K tiles (256 bytes per tile).  A slice lies
// inside one block; its scorer publishes every lane's cut mass and a copy of the block's mean row with the slice;
// the multiplier sums the cut mass per row and adds cut mass x mean after the slice's products.  A slice with no
// live key still does that part.
// NT = 2: row blocks of 9..16 rows as two 8-row N tiles per warp (one ldmatrix feeds both tiles' MMAs; the verdict is
// ORed over all 16 rows).
template <int D, bool TAIL, int NT>
__global__ void __launch_bounds__(kGatedThreads, 2)
fold_scan_gated_narrow_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmVs,
                              const ScanParams p) {
  using LO = GatedNarrowLayout<D, TAIL, NT>;
  constexpr int TK = LO::kTK, U = LO::kU, KS = 16 * U;       // keys per tile, sub-slices and keys per warp slice
  constexpr int C16 = D / 8;                                 // 16-byte chunks per value row
  constexpr int RPI = 32 / C16;                              // rows one warp-wide async copy covers
  constexpr int SW = kConsumerWarps;                         // scorer warps
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t *gen = smem_raw + (base - raw);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // kv heads fastest: CTAs that run together read the same tokens' rows, which sit side by side in memory
  // x = row group + row_groups * kv head (row groups only with NT = 2: more than 16 rows)
  const int rg = blockIdx.x % p.row_groups, kvh = blockIdx.x / p.row_groups, split = blockIdx.y, seq = blockIdx.z;
  const int rbase = rg * 16;                                 // first row of this CTA's group
  const SeqWork w = seq_work<TK>(p, seq);
  if (split >= w.n_chunks) return;
  const int stages = p.stages, vr = p.vr, R = p.R, n = w.n;
  const int dstart = draft_start(p, n);                     // keys from here on are per-request drafts
  const uint32_t full0 = base + LO::off_bar(stages, vr), empty0 = full0 + 8u * stages;
  const uint32_t vfull0 = empty0 + 8u * stages, vempty0 = vfull0 + 8u * kConsumerWarps * vr;

  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) {
      mbar_init(full0 + 8u * s, 1);
      mbar_init(empty0 + 8u * s, kConsumerWarps);
    }
    for (int s = 0; s < kConsumerWarps * vr; ++s) {
      mbar_init(vfull0 + 8u * s, 1);
      mbar_init(vempty0 + 8u * s, 1);
    }
    mbar_fence_init();
  }
  __syncthreads();
  pdl_launch_dependents();
  if (warp == SW + kConsumerWarps) {                         // the key tiles depend on nothing the reference kernel writes
    if (lane == 0) produce_tiles<D, false, LO::kKStage, TK, TAIL>(&tmK, &tmK, p, w, split, kvh, seq, base, full0, empty0);
    return;
  }
  pdl_wait();                                                // z comes from the kernel before

  const bool scorer = warp < SW;
  const int sl = warp & 3;                                   // the slice of every tile this warp owns
  constexpr int pentry = LO::kPEntry, pcut = U * NT * 512, pmean = pcut + NT * 256, pmask = pentry - 32;
  uint8_t *pring = gen + LO::off_pring(stages, vr) + sl * vr * pentry;
  const uint32_t vring = base + LO::off_vring(stages) + sl * vr * LO::kVSlice;
  const uint32_t vfull = vfull0 + 8u * sl * vr, vempty = vempty0 + 8u * sl * vr;
  bool dead = false;
  int vs = 0;
  uint32_t vphase = 0, vwrapped = 0;

  if (scorer) {
    RowBlockN<D> rb[NT];
    float l0[NT], l1[NT];
#pragma unroll
    for (int q = 0; q < NT; ++q) {
      load_rows_n<D>(rb[q], p, seq, kvh, lane, rbase + 8 * q);
      l0[q] = l1[q] = 0.f;
    }
    float *redl = reinterpret_cast<float *>(gen + LO::off_redl(stages, vr));
    const int page_mask = (1 << p.page_shift) - 1;
    const uint64_t vpol = policy_evict_first();
    // row-by-row fetch: lane covers 16-byte chunk (lane % C16) of rows (lane / C16) + RPI * i, swizzled as a box is
    const uint32_t rdst0 = ((lane % C16) >> 3) * (KS * 128) + (lane / C16) * 128;
    const long long rsrc0 = (long long)(lane / C16) * p.v_stride_tok + (lane % C16) * 8;
    int stage = 0;
    uint32_t phase = 0;
    unsigned long long st_fetched = 0, st_total = 0, st_skipped = 0;

    for (TileCursor k = cursor_begin(w, split); cursor_valid(k, w);) {
      const int my_stage = stage, my_vs = vs;
      const uint32_t my_phase = phase, my_vphase = vphase, my_wrapped = vwrapped;
      if (++stage == stages) { stage = 0; phase ^= 1u; }
      if (++vs == vr) { vs = 0; vwrapped = 1u; vphase ^= 1u; }
      {
        const bool ready = mbar_wait(full0 + 8u * my_stage, my_phase, dead);
        const int key0 = k.t * TK + sl * KS;
        uint32_t bh[U][NT][2], bl[U][NT][2];
        float cm0[NT], cm1[NT];                              // this lane's keys' cut mass for rows 8 q + (lane%4)*2 + {0,1}
        uint2 mean8 = make_uint2(0u, 0u);
        uint32_t fetch = 0;                                  // bit 16 u + k: key k of sub-slice u is live for some row
        uint32_t tile_live = 0;                              // bit NT u + q: some key of sub-slice u is live for N tile q
#pragma unroll
        for (int q = 0; q < NT; ++q) {
          cm0[q] = cm1[q] = 0.f;
#pragma unroll
          for (int u = 0; u < U; ++u) bh[u][q][0] = bh[u][q][1] = bl[u][q][0] = bl[u][q][1] = 0u;
        }
        if (ready) {
          float s[U][NT][4];
#pragma unroll
          for (int u = 0; u < U; ++u) {
            qk_issue_nt<D, TK, NT>(rb, base + my_stage * LO::kKStage, sl * U + u, lane, s[u]);
            if (key0 + 16 * u + 16 > dstart) {
#pragma unroll
              for (int q = 0; q < NT; ++q) mask_drafts_n<D>(rb[q], s[u][q], lane, key0 + 16 * u, dstart);
            }
          }
          if (TAIL && lane * 8 < D * 2)                      // this lane's 8 bytes of the slice's block mean row
            mean8 = *reinterpret_cast<const uint2 *>(gen + my_stage * LO::kKStage + LO::kKTile +
                                                     ((sl * KS) / 64) * (D * 2) + lane * 8);
          __syncwarp();
          if (lane == 0) mbar_arrive(empty0 + 8u * my_stage); // the K slice is consumed: release the tile
#pragma unroll
          for (int u = 0; u < U; ++u)
#pragma unroll
            for (int q = 0; q < NT; ++q) {
              const uint32_t live = weights_n<D, true, TAIL>(rb[q], s[u][q], lane, key0 + 16 * u, n, p.scale_log2, p.neg_T,
                                                             bh[u][q], bl[u][q], l0[q], l1[q], &cm0[q], &cm1[q]);
              fetch |= live << (16 * u);
              tile_live |= live ? (1u << (NT * u + q)) : 0u;
            }
        }
        bool any_cut = false;
#pragma unroll
        for (int q = 0; q < NT; ++q) any_cut |= cm0[q] > 0.f || cm1[q] > 0.f;
        const bool tail = TAIL && __any_sync(0xffffffffu, any_cut);
        // a mostly-live sub-slice is cheaper to fetch whole (one TMA box per 64 channels) than row by row; rows nobody
        // keeps then ride along under a zero weight.  Never past the sequence end: those rows may hold anything.
        uint32_t whole = 0;
#pragma unroll
        for (int u = 0; u < U; ++u) {
          const uint32_t m = (fetch >> (16 * u)) & 0xffffu;
          const bool wh = (key0 + 16 * u + 16 <= n) && (__popc(m) >= p.box_min);
          whole |= wh ? (1u << u) : 0u;
          st_fetched += wh ? 16 : __popc(m);
        }
        {
          const int nvalid = min(KS, max(0, n - key0));
          st_total += nvalid;
          st_skipped += (fetch == 0 && nvalid > 0) ? 1 : 0;
        }
        if (!my_wrapped || mbar_wait(vempty + 8u * my_vs, my_vphase ^ 1u, dead)) {
          // publish the slice: weights as the value product's B-operand registers, and the verdict
          uint8_t *pe = pring + my_vs * pentry;
#pragma unroll
          for (int u = 0; u < U; ++u)
#pragma unroll
            for (int q = 0; q < NT; ++q)
              *reinterpret_cast<uint4 *>(pe + (u * NT + q) * 512 + lane * 16) =
                  make_uint4(bh[u][q][0], bh[u][q][1], bl[u][q][0], bl[u][q][1]);
          if (TAIL && tail) {
#pragma unroll
            for (int q = 0; q < NT; ++q) *reinterpret_cast<float2 *>(pe + pcut + q * 256 + lane * 8) = make_float2(cm0[q], cm1[q]);
            if (lane * 8 < D * 2) *reinterpret_cast<uint2 *>(pe + pmean + lane * 8) = mean8;
          }
          // verdict words: the fetch mask; bit 0 = block tail present, bits 8.. = which N tiles have a live key per sub-slice
          if (lane == 0) *reinterpret_cast<uint2 *>(pe + pmask) = make_uint2(fetch, (tail ? 1u : 0u) | (tile_live << 8));
          const uint32_t bar = vfull + 8u * my_vs;
          const uint32_t vdst = vring + my_vs * LO::kVSlice;
          if (whole) {
            fence_proxy_async_smem();                        // the slot's earlier generic-proxy traffic, then TMA writes
            __syncwarp();
          }
          bool rows = false;
#pragma unroll
          for (int u = 0; u < U; ++u) {
            const uint32_t m = (fetch >> (16 * u)) & 0xffffu;
            if (m == 0u) continue;
            int c_seq = seq, c_tok = key0 + 16 * u;
            if (p.paged) {
              const int pg = p.page_table[(long long)seq * p.max_pages + (c_tok >> p.page_shift)];
              c_seq = min(max(pg, 0), p.num_pages - 1);
              c_tok &= page_mask;
            }
            if ((whole >> u) & 1u) {
              if (lane == 0) {
                mbar_expect_tx_only(bar, 16 * D * 2);
                const int c1 = p.pos_tok == 1 ? c_tok : (p.pos_head == 1 ? kvh : c_seq);
                const int c2 = p.pos_tok == 2 ? c_tok : (p.pos_head == 2 ? kvh : c_seq);
                const int c3 = p.pos_tok == 3 ? c_tok : (p.pos_head == 3 ? kvh : c_seq);
#pragma unroll
                for (int h = 0; h < D / 64; ++h)
                  tma_load_4d(vdst + (h * KS + 16 * u) * 128, &tmVs, bar, h * 64, c1, c2, c3, vpol);
              }
            } else {
              rows = true;
              const __nv_bfloat16 *src = p.v + (long long)c_seq * p.v_stride_seq + (long long)c_tok * p.v_stride_tok +
                                         (long long)kvh * p.v_stride_head + rsrc0;
#pragma unroll
              for (int i = 0; i < 16 / RPI; ++i) {
                const int row = i * RPI + lane / C16;        // row & 7 is the same within the sub-slice and the slice
                const bool f = (m >> row) & 1u;
                cp_async_16(vdst + rdst0 + (16 * u + i * RPI) * 128 + ((((lane % C16) ^ row) & 7) << 4), f ? src : p.v,
                            f ? 16u : 0u);
                src += (long long)RPI * p.v_stride_tok;
              }
            }
          }
          if (rows) cp_async_mbar_arrive(bar);               // this lane's copies hold the phase open
          __syncwarp();
          if (lane == 0) mbar_arrive(bar);
        }
      }
      const int c_done = k.c;
      if (cursor_next(k, w, p.num_splits)) {
        float *slot = p.slots + (((long long)seq * p.Hkv + kvh) * p.max_slots + c_done) * p.slot_stride;
#pragma unroll
        for (int q = 0; q < NT; ++q)
          reduce_store_L_n<SW>(l0[q], l1[q], redl, slot + R * D + rbase + 8 * q, min(8, R - rbase - 8 * q), warp, lane,
                               threadIdx.x, 1);
      }
    }
    if (lane == 0) {
      if (dead) atomicOr(&p.hdr->wait_timeouts, 2u);
      atomicAdd(reinterpret_cast<unsigned long long *>(&p.hdr->v_rows_fetched), st_fetched);
      atomicAdd(reinterpret_cast<unsigned long long *>(&p.hdr->v_rows_total), st_total);
      if (st_skipped) atomicAdd(reinterpret_cast<unsigned long long *>(&p.hdr->v_slices_skipped), st_skipped);
    }
  } else {
    float o[NT][D / 16][4];
#pragma unroll
    for (int q = 0; q < NT; ++q)
#pragma unroll
      for (int i = 0; i < D / 16; ++i) o[q][i][0] = o[q][i][1] = o[q][i][2] = o[q][i][3] = 0.f;
    float *red = reinterpret_cast<float *>(gen + LO::off_red(stages, vr));
    for (TileCursor k = cursor_begin(w, split); cursor_valid(k, w);) {
      const int my = vs;
      const bool landed = mbar_wait(vfull + 8u * my, vphase, dead);
      if (++vs == vr) { vs = 0; vphase ^= 1u; }
      if (landed) {
        const uint8_t *pe = pring + my * pentry;
        const uint2 vw = *reinterpret_cast<const uint2 *>(pe + pmask);
        const uint32_t verdict = vw.x;
#pragma unroll
        for (int u = 0; u < U; ++u) {
          if (((verdict >> (16 * u)) & 0xffffu) == 0u) continue;   // nobody keeps a key of this sub-slice
          uint32_t bh[NT][2], bl[NT][2];
#pragma unroll
          for (int q = 0; q < NT; ++q) {
            const uint4 a = *reinterpret_cast<const uint4 *>(pe + (u * NT + q) * 512 + lane * 16);
            bh[q][0] = a.x; bh[q][1] = a.y; bl[q][0] = a.z; bl[q][1] = a.w;
          }
          const uint32_t skip = ~(vw.y >> (8 + NT * u)) & ((1u << NT) - 1u);
          value_product_nt<D, KS, NT>(o, vring + my * LO::kVSlice, 16 * u, lane, bh, bl, skip);
        }
        if (TAIL && (vw.y & 1u)) {                           // o[q][mt]: channels 16 mt + lane/4 (+8), rows 8 q + (lane%4)*2 + {0,1}
          const __nv_bfloat16 *mrow = reinterpret_cast<const __nv_bfloat16 *>(pe + pmean) + (lane >> 2);
#pragma unroll
          for (int q = 0; q < NT; ++q) {
            float2 c = make_float2(0.f, 0.f);                // the rows' cut mass: over the 8 lanes that scored their keys
#pragma unroll
            for (int gsrc = 0; gsrc < 8; ++gsrc) {
              const float2 t = *reinterpret_cast<const float2 *>(pe + pcut + q * 256 + (gsrc * 4 + (lane & 3)) * 8);
              c.x += t.x; c.y += t.y;
            }
#pragma unroll
            for (int mt = 0; mt < D / 16; ++mt) {
              const float m0 = __bfloat162float(mrow[mt * 16]), m1 = __bfloat162float(mrow[mt * 16 + 8]);
              o[q][mt][0] = fmaf(c.x, m0, o[q][mt][0]); o[q][mt][1] = fmaf(c.y, m0, o[q][mt][1]);
              o[q][mt][2] = fmaf(c.x, m1, o[q][mt][2]); o[q][mt][3] = fmaf(c.y, m1, o[q][mt][3]);
            }
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(vempty + 8u * my);
      }
      const int c_done = k.c;
      if (cursor_next(k, w, p.num_splits)) {
        float *slot = p.slots + (((long long)seq * p.Hkv + kvh) * p.max_slots + c_done) * p.slot_stride;
#pragma unroll
        for (int q = 0; q < NT; ++q) tree_store_A_n<D>(o[q], red, slot + (rbase + 8 * q) * D, min(8, R - rbase - 8 * q), sl, lane, 2);
      }
    }
    if (lane == 0 && dead) atomicOr(&p.hdr->wait_timeouts, 4u);
  }
}

}  // namespace fold
