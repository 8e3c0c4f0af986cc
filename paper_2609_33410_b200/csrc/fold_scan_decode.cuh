// Row-block decode scan on the 5th-generation tensor cores (tcgen05 + TMEM), head_dim 128, up to 16 query
// rows per (sequence, kv head), dense or depth-gated.
//
// Algorithm 1 puts the keys on the M side of its score product and the group's rows on N, and reads the
// verdicts of a tile off the accumulator.  On sm_100a that shape is native: one tcgen05.mma covers 128 keys,
// the scores S^T[128 keys x 16 rows] land in tensor memory with ONE KEY PER LANE, and a tcgen05.ld hands every
// thread of the weight warps all the rows' scores of one key.  The verdict "some row keeps this key" is then a
// thread-local OR, the weights need no shuffles, and the per-key cost in warp instructions is a fraction of the
// mma.sync form's (no ldmatrix, no movmatrix, no warp-wide reduction per 16 keys).
//
//   scores   S^T[128 keys, 16]  = K tile [128 keys, D] (A, shared memory, K-major)  x  Q^T (B, shared memory)
//   weights  thread-per-key: p = 2^(s - Z) per row, depth gate, two-term BF16 split, L in registers;
//            P_hi / P_lo written to shared memory as the B operand [16 rows, 128 keys] of the value product
//   values   A^T[D, 16] += V^T[D, 128 keys] (A, the value tile as it lies in shared memory, MN-major) x P^T
//            accumulated in tensor memory over the tiles of a canonical chunk, read out once per chunk
//
// Depth-gated: only K is streamed ahead by the producer; after the verdicts the weight warps request the value
// rows some row of the group keeps -- a 16-key group that is mostly live as one tensor-map box, otherwise row by
// row with 16-byte async copies issued for live rows only.  Rows nobody keeps cost no traffic and no
// instruction; their weights are exactly zero and the shared-memory rows they would occupy hold zeros or
// earlier rows of the same cache (finite), so the product is unaffected.
//
// Scheduling: a persistent grid.  The canonical chunks of the whole launch form one list, ordered kv head
// fastest, then chunk, then sequence; a CTA hosts two WORKERS (worker v takes chunks v, v + W, v + 2 W, ...,
// W = 2 x CTAs), each a set of four weight warps with its own score / weight / accumulator buffers.  The two
// workers' tiles alternate in the CTA's key ring and on the tensor pipe, so one worker's weight phase hides
// behind the other's products, and the ring never drains between chunks or (sequence, kv head) units.  A chunk's
// (A, L) is formed by the same instruction sequence whichever worker runs it: the slot's bits do not depend on
// the grid, the batch or the split hint.
#pragma once

#include <cooperative_groups.h>

#include "fold_estimate.cuh"
#include "fold_merge.cuh"
#include "fold_scan_umma.cuh"

namespace fold {


constexpr int kDecKeys = 128;                        // keys per tile (MMA M of the score product)
constexpr int kDecKS = 3, kDecVS = 3;                // key / value ring depths (32 KB stages)
constexpr int kDecThreads = 12 * 32;                 // key producer, score issuer, value-product issuer, value producer (dense), 2 workers x 4 weight warps
constexpr int kDecTmemCols = 128;                    // S[worker][2]: 16 columns each from 0;  A[worker][chunk parity]: 16 columns each from 64
constexpr int kDecMaxRows = 8;                       // rows per (sequence, kv head) the host sends here (the kernel itself takes 16)

struct DecLayout {                                   // byte offsets from a 1 KB-aligned base
  static constexpr int kTile = kDecKeys * 256;       // one key or value tile: [2 halves][128 keys][128 B], swizzled
  static constexpr int kK = 0;
  static constexpr int kV = kK + kDecKS * kTile;
  static constexpr int kP = kV + kDecVS * kTile;     // weights, 8 KB per worker: two 4 KB buffers (up to 8 rows) or one of 8 KB
  static constexpr int kQ = kP + 4 * 4096;           // query rows [worker][parity]: [2 halves][8 rows][128 B] = 2 KB each
  static constexpr int kQZero = kQ + 4 * 2048;       // [2 halves][8 rows][128 B] of zeros: rows 8..15 of every query operand
  static constexpr int kCut = kQZero + 2048;         // block tail: cut mass [worker][chunk parity][8 tiles][4 warps][8 rows] floats
  static constexpr int kLpart = kCut + 4096;         // [worker][chunk parity][4 warps][16] floats (kQ .. kLpart is 16 KB)
  static constexpr int kBar = kLpart + 1024;
  static constexpr int kTotal = kBar + 512 + 1024;   // + alignment slack
};
// barrier indices (8 bytes each, from kBar)
constexpr int kDecBarKFull = 40, kDecBarKEmpty = 0, kDecBarVFull = 4, kDecBarPvDone = 8, kDecBarSEmpty = 12,
              kDecBarPFull = 16, kDecBarQFull = 20, kDecBarLFull = 24, kDecBarSFull = 28, kDecBarPFree = 32, kDecBarTmemSlot = 38;
constexpr int kDecLiveFlags = 384;                   // byte offset from kBar: [worker][weight buffer][warp] words: a key of the warp's 32 is live
constexpr int kDecTimeouts = 448;                    // byte offset from kBar: which roles of this CTA gave up a wait (one word)
constexpr int kDecStats = 456;                       // byte offset from kBar: value rows fetched, value rows in all, groups skipped (64-bit each)

// A problem of one wave -- every worker has at most one canonical chunk -- runs the whole decode in ONE cooperative
// launch of the scan kernel: the weight warps form their (sequence, kv head)'s reference from the 192 sampled keys
// themselves while the key tiles travel (mode 1; mode 2 reads a given z), the chunks are scanned, and after a grid-wide
// barrier the CTAs share out the rows of the order-free partial add.  Every step is the separate kernels' own device
// code, so the three-launch path and this one agree bit for bit.
struct FusedParams {
  int mode;                                          // 0: the scan alone
  EstParams est;
  MergeParams mrg;
};

// D[tmem] (+)= A * B with both operands in shared memory (64-bit matrix descriptors as two words each).
template <bool ACC>
__device__ __forceinline__ void umma_bf16_ss(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi,
                                             uint32_t idesc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 ad, bd;\n\t"
      "setp.ne.b32 p, %6, 0;\n\t"
      "mov.b64 ad, {%1, %2};\n\t"
      "mov.b64 bd, {%3, %4};\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], ad, bd, %5, p;\n\t}"
      ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "n"(ACC ? 1 : 0)
      : "memory");
}
// Instruction descriptor: FP32 accumulate, BF16 operands, M = 128, N = n; a_mn: the A operand is MN-major.
__host__ __device__ constexpr uint32_t dec_idesc(int n, int a_mn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a_mn << 15) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
}
// N consecutive FP32 columns of this thread's TMEM lane.
template <int N>
__device__ __forceinline__ void tmem_ld_cols(uint32_t taddr, float (&v)[N]) {
  static_assert(N == 1 || N == 4 || N == 8 || N == 16 || N == 32, "column counts the decode scan uses");
  if constexpr (N == 32) {
    tmem_ld32(taddr, v);
    return;
  }
  uint32_t r[N];
  if constexpr (N == 1) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x1.b32 {%0}, [%1];" : "=r"(r[0]) : "r"(taddr) : "memory");
  } else if constexpr (N == 4) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(taddr) : "memory");
  } else if constexpr (N == 8) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(taddr) : "memory");
  } else {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr) : "memory");
  }
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < N; ++i) v[i] = __uint_as_float(r[i]);
}

// Barrier `id` (1..15) among `threads` threads of the CTA (whole warps); barrier 0 is __syncthreads'.
__device__ __forceinline__ void named_bar_sync(int id, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

// ------------------------------------------------------------------------------------------------
// A worker's walk over its canonical chunks: entries g = first, first + step, ... of the launch's chunk list
// (kv head fastest, then chunk, then sequence); entries past a sequence's own chunk count are skipped.
struct DecWorker {
  int g, step, n_entries;        // next list entry to look at
  int g_a, g_b, g_seq;           // that entry in the list's mixed radix (fastest digit first): kept in step with g, no divisions per chunk
  int d_a, d_b, d_seq;           // the step in the same mixed radix
  int ra, rb;                    // the radices: (kv heads, slots), or chunk-major (slots rounded up to even, kv heads)
  int len_seq, len_n;            // the sequence whose length was read last (entries of a worker mostly stay in one)
  int seq, kvh, c, n;            // the current chunk: sequence, kv head, chunk index, the sequence's length
  int t, t_end;                  // tile cursor: 128-key tiles [t, t_end) of the sequence remain in the chunk
  int t_first;                   // first tile of the chunk
};
__device__ __forceinline__ int dec_seqlen(const ScanParams &p, int seq) {
  const int n = p.seqlens[seq];
  return n < 0 ? 0 : (n > p.max_seqlen ? p.max_seqlen : n);
}
// The list's two orders.  Ordinarily kv head fastest, then chunk, then sequence.  Chunk-major (a decode that runs in one
// launch, every worker with one chunk at most): chunk fastest, a (sequence, kv head)'s chunks padded to an even count,
// so that the two workers of a CTA always scan chunks of the same (sequence, kv head) and share its reference.
__device__ __forceinline__ int dec_radix_a(const ScanParams &p) { return p.chunk_major ? ((p.max_slots + 1) & ~1) : p.Hkv; }
__device__ __forceinline__ int dec_radix_b(const ScanParams &p) { return p.chunk_major ? p.Hkv : p.max_slots; }
__device__ __forceinline__ void dec_worker_init(DecWorker &w, const ScanParams &p, int first, int step) {
  w.g = first; w.step = step;
  w.ra = dec_radix_a(p); w.rb = dec_radix_b(p);
  w.n_entries = p.num_seqs * w.ra * w.rb;
  w.g_a = first % w.ra; w.g_b = (first / w.ra) % w.rb; w.g_seq = first / w.ra / w.rb;
  w.d_a = step % w.ra; w.d_b = (step / w.ra) % w.rb; w.d_seq = step / w.ra / w.rb;
  w.len_seq = -1; w.len_n = 0;
  w.seq = w.kvh = w.c = w.n = 0;
  w.t = w.t_end = w.t_first = 0;
}
// Move to the worker's next non-empty chunk.  False when its list is exhausted.
__device__ __forceinline__ bool dec_worker_next_chunk(DecWorker &w, const ScanParams &p) {
  while (w.g < w.n_entries) {
    const int kvh = p.chunk_major ? w.g_b : w.g_a, c = p.chunk_major ? w.g_a : w.g_b, seq = w.g_seq;
    w.g += w.step;                                           // and the same step in the mixed radix, with carries
    w.g_a += w.d_a;
    if (w.g_a >= w.ra) { w.g_a -= w.ra; ++w.g_b; }
    w.g_b += w.d_b;
    if (w.g_b >= w.rb) { w.g_b -= w.rb; ++w.g_seq; }
    w.g_seq += w.d_seq;
    if (seq != w.len_seq) { w.len_seq = seq; w.len_n = dec_seqlen(p, seq); }
    const int n = w.len_n;
    if (c < num_chunks_of(n)) {
      const int ctiles = chunk_keys_of(n) / kDecKeys;
      w.seq = seq; w.kvh = kvh; w.c = c; w.n = n;
      w.t_first = w.t = c * ctiles;
      w.t_end = min((c + 1) * ctiles, (n + kDecKeys - 1) / kDecKeys);
      return true;
    }
  }
  return false;
}
// Tiles of list entry g (0 for an entry past its sequence's chunks).
__device__ __forceinline__ int dec_entry_tiles(const ScanParams &p, int g) {
  const int ra = dec_radix_a(p), rb = dec_radix_b(p);
  const int c = p.chunk_major ? g % ra : (g / ra) % rb, seq = g / ra / rb;
  const int n = dec_seqlen(p, seq);
  if (c >= num_chunks_of(n)) return 0;
  const int ctiles = chunk_keys_of(n) / kDecKeys;
  return min((c + 1) * ctiles, (n + kDecKeys - 1) / kDecKeys) - c * ctiles;
}
// Position in the CTA's tile order of the i-th tile of worker `set`, the workers having ta and tb tiles in all:
// the two alternate (a first) while both have tiles left, then the longer one runs on alone.
__device__ __forceinline__ int dec_global_index(int set, int i, int ta, int tb) {
  return set == 0 ? i + min(i, tb) : i + min(i + 1, ta);
}
// The CTA's tile order as seen by the roles that serve both workers (producer, MMA issuer): both walks are kept in
// named registers, never indexed.
struct DecPairWalk {
  DecWorker a, b;
  bool alive_a, alive_b;
  int cnt_a, cnt_b, ent_a, ent_b;                            // tiles and chunks each worker has been through
  int s, it;                                                 // whose tile is next; its position in the order
};
__device__ __forceinline__ void dec_pair_init(DecPairWalk &x, const ScanParams &p, int cta, int workers) {
  dec_worker_init(x.a, p, 2 * cta, workers);
  dec_worker_init(x.b, p, 2 * cta + 1, workers);
  x.alive_a = dec_worker_next_chunk(x.a, p);
  x.alive_b = dec_worker_next_chunk(x.b, p);
  x.cnt_a = x.cnt_b = x.ent_a = x.ent_b = 0;
  x.it = 0;
  x.s = x.alive_a ? 0 : 1;
}
__device__ __forceinline__ bool dec_pair_valid(const DecPairWalk &x) { return x.alive_a || x.alive_b; }
__device__ __forceinline__ void dec_pair_next(DecPairWalk &x, const ScanParams &p) {
  if (x.s == 0) {
    ++x.cnt_a;
    if (++x.a.t == x.a.t_end) { x.alive_a = dec_worker_next_chunk(x.a, p); ++x.ent_a; }
    x.s = x.alive_b ? 1 : 0;
  } else {
    ++x.cnt_b;
    if (++x.b.t == x.b.t_end) { x.alive_b = dec_worker_next_chunk(x.b, p); ++x.ent_b; }
    x.s = x.alive_a ? 0 : 1;
  }
  ++x.it;
}

// NC: score columns a weight thread reads (query rows, rounded up; at most 8).  The two weight terms share one N = 16
// operand (P_hi in rows 0..7, P_lo in rows 8..15: the value tile is read once per tile, not twice), double-buffered.
// The score product's B operand needs 16 rows too: rows 8..15 of every query buffer are one shared group of zeros
// (the descriptor's stride between 8-row groups points there).
// TAIL (with GATED; Section 4 "Depth as a dial", the block model's mean): a row's cut keys add their summed weight times
// the mean value row of their 64-key block.  Each weight warp sums its 32 keys' cut weights per row and tile (a tile
// is two blocks, a block two warps); at the chunk's end every thread -- one channel -- adds cut mass x mean for the
// chunk's blocks in block order, in FP32.
// KEYS: the key ring's depth (the value ring takes the rest of the six stages).
template <bool GATED, int NC, bool TAIL = false, int KEYS = (GATED ? 3 : 2)>
__global__ void __launch_bounds__(kDecThreads, 1)
fold_scan_decode_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                        const ScanParams p, const FusedParams f) {
  constexpr int D = 128;
  static_assert(NC <= 8 && (!TAIL || GATED), "up to 8 rows; the tail belongs to finite depth");
  constexpr int NPV = 16;                                    // N of the value product; P_lo sits NPV / 2 rows after P_hi
  constexpr int PB = 2;                                      // weight buffers per worker
  constexpr int PBYTES = NPV * 256;                          // [2 key halves][NPV rows][128 B]
  // Six 32 KB stages in all.  Dense: a key stage is free as soon as its scores are issued, a value stage waits for the
  // weights, so two key stages feed four value stages (5 % over three and three).  Depth-gated, the best split depends on
  // how much of the cache is live (and on the chunk length): a cache that is all live wants dense decode's two and four
  // (C2 at T=16: 321 us against 332 with three and three), a half-live one three and three (C3: 273 against 278 and
  // 301 us), one nobody keeps a value row of four and two where chunks are long (4-5 % over three and three).  The host
  // picks KEYS from the caller's fold_args.live_hint; three and three without a hint.  The split only schedules: every
  // one gives the same bits.
  static_assert(KEYS >= 2 && KEYS <= 4, "two to four key stages");
  constexpr int KS = KEYS, VS = 6 - KS;
  using LO = DecLayout;
  constexpr int OFF_V = KS * LO::kTile;                      // the value ring follows the key ring
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t *gen = smem_raw + (base - raw);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t bar0 = base + LO::kBar;
  auto bar = [&](int idx) { return bar0 + 8u * idx; };

  if (threadIdx.x == 0) {
    // "key tile landed": twice as many barriers as stages, so that a barrier only ever serves one worker's tiles (the
    // workers alternate) and its waiter, who takes them in order, is never more than one phase ahead of it
    for (int s = 0; s < 2 * KS; ++s) mbar_init(bar(kDecBarKFull + s), 1);
    for (int s = 0; s < KS; ++s) mbar_init(bar(kDecBarKEmpty + s), 1);
    for (int s = 0; s < VS; ++s) { mbar_init(bar(kDecBarVFull + s), GATED ? 4 : 1); mbar_init(bar(kDecBarPvDone + s), 1); }
    for (int s = 0; s < 4; ++s) {                            // one arrival per weight warp of the worker
      mbar_init(bar(kDecBarSEmpty + s), 4);
      mbar_init(bar(kDecBarPFull + s), 4);
      mbar_init(bar(kDecBarQFull + s), 4);
      mbar_init(bar(kDecBarLFull + s), 4);
      mbar_init(bar(kDecBarSFull + s), 1);
      mbar_init(bar(kDecBarPFree + s), 1);
    }
    mbar_fence_init();
    for (int i = 0; i < 8; ++i) reinterpret_cast<uint32_t *>(gen + LO::kBar + kDecTimeouts)[i] = 0u;   // timeouts, statistics
  }
  // one launch for the whole decode: nothing before this kernel has cleared the workspace header
  if (f.mode && blockIdx.x == 0 && threadIdx.x >= 32 && threadIdx.x < 48) reinterpret_cast<uint32_t *>(p.hdr)[threadIdx.x - 32] = 0u;
  if (warp == 1) tmem_alloc(bar(kDecBarTmemSlot), kDecTmemCols);
  // value ring, weight buffers and query tiles start as zeros: a row or column nobody writes must hold finite data
  for (int i = threadIdx.x; i < (LO::kLpart - OFF_V) / 16; i += kDecThreads)
    *reinterpret_cast<uint4 *>(gen + OFF_V + i * 16) = make_uint4(0, 0, 0, 0);
  fence_proxy_async_smem();
  pdl_launch_dependents();
  tc_fence_before();
  __syncthreads();                                           // barriers initialised, TMEM allocated, buffers cleared
  tc_fence_after();
  const uint32_t tmem = *reinterpret_cast<volatile uint32_t *>(gen + LO::kBar + 8 * kDecBarTmemSlot);

  // the CTA's two workers and how many tiles each will walk (every warp computes both counts, a lane per entry)
  const int W = 2 * gridDim.x;
  const int n_entries = p.num_seqs * dec_radix_a(p) * dec_radix_b(p);
  int TA = 0, TB = 0;
  {
    int ca = 0, cb = 0;
    for (int g = 2 * blockIdx.x + lane * W; g < n_entries; g += 32 * W) {
      ca += dec_entry_tiles(p, g);
      if (g + 1 < n_entries) cb += dec_entry_tiles(p, g + 1);
    }
    TA = __reduce_add_sync(0xffffffffu, ca);
    TB = __reduce_add_sync(0xffffffffu, cb);
  }
  const int page_mask = (1 << p.page_shift) - 1;
  uint32_t *s_timeouts = reinterpret_cast<uint32_t *>(gen + LO::kBar + kDecTimeouts);
  unsigned long long *s_stats = reinterpret_cast<unsigned long long *>(gen + LO::kBar + kDecStats);
  bool dead = false;
  // warp-uniform bounded wait: the warp goes on together or gives up together
  auto wait_u = [&](uint32_t b, uint32_t parity) {
    const bool ok = __all_sync(0xffffffffu, mbar_wait(b, parity, dead));
    if (!ok) dead = true;
    return ok;
  };

  if (warp == 0 || (!GATED && warp == 3)) {
    // ------------------------------------------------------------ producers: warp 0 streams the key tiles; dense decode
    // reads every value row, so there warp 3 streams the value tiles the same way (its ring is freed by the value
    // products, the key ring by the score products: neither waits for the other)
    const bool keys = warp == 0;
    if (lane < 2 && TA + TB > 0) {                           // one lane per 64-channel half of a tile
      const CUtensorMap *tm_ = keys ? &tmK : &tmV;
      tma_prefetch_desc(tm_);
      const uint64_t pol = policy_evict_first();
      DecPairWalk x;
      dec_pair_init(x, p, blockIdx.x, W);
      const int boxes_per_tile = kDecKeys / p.box_tok;
      const int full0 = keys ? kDecBarKFull : kDecBarVFull, empty0 = keys ? kDecBarKEmpty : kDecBarPvDone;
      const int depth = keys ? KS : VS;
      for (; dec_pair_valid(x); dec_pair_next(x, p)) {
        const int it = x.it, st = it % depth;
        const int seq = x.s ? x.b.seq : x.a.seq, kvh = x.s ? x.b.kvh : x.a.kvh, n = x.s ? x.b.n : x.a.n;
        const int tok0 = (x.s ? x.b.t : x.a.t) * kDecKeys;
        const int nbox = min(boxes_per_tile, (n - tok0 + p.box_tok - 1) / p.box_tok);
        int pg[8];                                           // the boxes' pages, looked up before the stage is waited for
        if (p.paged) {
#pragma unroll
          for (int bx = 0; bx < 8; ++bx)
            if (bx < nbox) pg[bx] = p.page_table[(long long)seq * p.max_pages + ((tok0 + bx * p.box_tok) >> p.page_shift)];
        }
        if (it >= depth && !mbar_wait_spin(bar(empty0 + st), (uint32_t)((it / depth - 1) & 1), dead)) break;
        const uint32_t full = bar(keys ? kDecBarKFull + it % (2 * KS) : full0 + st);
        const uint32_t dst = base + (keys ? LO::kK : OFF_V) + st * LO::kTile;
        if (lane == 0) mbar_expect_tx(full, nbox * p.box_tok * D * 2);
#pragma unroll
        for (int bx = 0; bx < 8; ++bx) {
          if (bx >= nbox) break;
          const int j0 = tok0 + bx * p.box_tok;
          int c_seq = seq, c_tok = j0;
          if (p.paged) {
            c_seq = min(max(pg[bx], 0), p.num_pages - 1);
            c_tok = j0 & page_mask;
          }
          const int c1 = p.pos_tok == 1 ? c_tok : (p.pos_head == 1 ? kvh : c_seq);
          const int c2 = p.pos_tok == 2 ? c_tok : (p.pos_head == 2 ? kvh : c_seq);
          const int c3 = p.pos_tok == 3 ? c_tok : (p.pos_head == 3 ? kvh : c_seq);
          tma_load_4d(dst + (lane * kDecKeys + bx * p.box_tok) * 128, tm_, full, lane * 64, c1, c2, c3, pol);
        }
      }
      if (dead && lane == 0) {
        // gave up: the copies already requested must still land before the CTA may leave (bounded waits again)
        atomicOr(s_timeouts, 1u);
        bool d2 = false;
        for (int back = 1; back <= depth && x.it - back >= 0; ++back) {
          const int it = x.it - back;
          if (keys) mbar_wait(bar(kDecBarKFull + it % (2 * KS)), (uint32_t)((it / (2 * KS)) & 1), d2);
          else mbar_wait(bar(full0 + it % depth), (uint32_t)((it / depth) & 1), d2);
        }
      }
    }
  } else if (warp == 1 || warp == 2) {
    // ------------------------------------------------------------ MMA issuers, one thread per worker
    // One thread can start a tcgen05.mma about every 72 cycles while the pipe takes an M128 N16 K16 product about every
    // 40, so each worker has its own issuing thread.  It keeps two walks over the worker's tiles -- value products, and
    // scores up to two tiles ahead (the worker has two score buffers) -- and issues whichever is ready, value products
    // first (they free a value stage and a weight buffer), probing the barriers without suspending.  The worker thus
    // forms the weights of its next tile, and requests that tile's value rows, while those of its current tile travel.
    const int set = warp - 1;
    const int my_tiles = set == 0 ? TA : TB;
    if (lane == 0 && my_tiles > 0) {
      constexpr uint32_t idesc_qk = dec_idesc(16, 0), idesc_pv = dec_idesc(NPV, 1);
      constexpr uint32_t desc_hi = umma_desc_hi(1024);
      DecWorker wq, wp;
      dec_worker_init(wq, p, 2 * blockIdx.x + set, W);
      dec_worker_init(wp, p, 2 * blockIdx.x + set, W);
      bool q_alive = dec_worker_next_chunk(wq, p);
      bool p_alive = dec_worker_next_chunk(wp, p);
      int iq = 0, eq = 0;                                    // tiles / chunks the score walk has been through
      int ip = 0, ep = 0;                                    // the same for the value products
      uint32_t idle = 0;
      while (p_alive) {
        // ---- value product of tile ip, if its weights and value rows are in
        {
          const int it = dec_global_index(set, ip, TA, TB), vs = it % VS;
          const bool pf = mbar_test_wait(bar(kDecBarPFull + 2 * set + (ip % PB)), (uint32_t)((ip / PB) & 1));
          const bool vf = mbar_test_wait(bar(kDecBarVFull + vs), (uint32_t)((it / VS) & 1));
          if (pf && vf) {
            const bool first = wp.t == wp.t_first;
            bool some = true;                                // depth-gated: a tile nobody keeps a key of adds nothing
            if (GATED && !first) {                           // (a chunk's first tile always runs: it initialises the accumulator)
              const volatile uint32_t *f = reinterpret_cast<const volatile uint32_t *>(gen + LO::kBar + kDecLiveFlags) + (set * 2 + (ip % PB)) * 4;
              some = (f[0] | f[1] | f[2] | f[3]) != 0u;
            }
            fence_proxy_async_smem();                        // value rows written by plain async copies, read by the tensor pipe
            tc_fence_after();
            // value tile [2 channel halves][128 keys][128 B] as the MN-major A operand: 16 keys = 2048 B per K step,
            // the halves 16 KB apart (leading-dimension offset); weights [2 key halves][NPV rows][128 B], K-major
            const uint32_t a_lo = umma_desc_lo(base + OFF_V + vs * LO::kTile, kDecKeys * 128);
            const uint32_t b_lo = umma_desc_lo(base + LO::kP + set * 8192 + (ip % PB) * PBYTES, 16);
            const uint32_t d = tmem + 64 + set * 32 + (ep & 1) * 16;   // the accumulators alternate with the chunk's parity
            if (some) {
#pragma unroll
              for (int j = 0; j < kDecKeys / 16; ++j) {
                const uint32_t bo = ((j >> 2) * (NPV * 128) + (j & 3) * 32) >> 4;
                if (j == 0) {
                  if (first) umma_bf16_ss<false>(d, a_lo, desc_hi, b_lo, desc_hi, idesc_pv);
                  else umma_bf16_ss<true>(d, a_lo, desc_hi, b_lo, desc_hi, idesc_pv);
                } else {
                  umma_bf16_ss<true>(d, a_lo + j * (2048 >> 4), desc_hi, b_lo + bo, desc_hi, idesc_pv);
                }
              }
            }
            tc_commit(bar(kDecBarPvDone + vs));              // the value stage is free
            tc_commit(bar(kDecBarPFree + 2 * set + (ip % PB)));   // so is the worker's weight buffer (and, at a chunk's end, A is final)
            ++ip;
            if (++wp.t == wp.t_end) { p_alive = dec_worker_next_chunk(wp, p); ++ep; }
            idle = 0;
            continue;
          }
        }
        // ---- scores of tile iq: at most two tiles ahead of the value products, and at most one chunk ahead (a chunk's
        // query rows are staged while the worker is on the chunk before)
        if (q_alive && iq <= ip + 2 && eq <= ep + 1) {
          const int it = dec_global_index(set, iq, TA, TB), ks = it % KS;
          const bool first = wq.t == wq.t_first;
          bool ok = mbar_test_wait(bar(kDecBarKFull + it % (2 * KS)), (uint32_t)((it / (2 * KS)) & 1));
          if (iq >= 2) ok &= mbar_test_wait(bar(kDecBarSEmpty + 2 * set + (iq & 1)), (uint32_t)(((iq >> 1) - 1) & 1));
          if (first) ok &= mbar_test_wait(bar(kDecBarQFull + 2 * set + (eq & 1)), (uint32_t)((eq >> 1) & 1));
          if (ok) {
            tc_fence_after();
            const uint32_t a_lo = umma_desc_lo(base + LO::kK + ks * LO::kTile, 16);
            // query rows 0..7 of each 64-channel half in the worker's buffer, rows 8..15 in the shared zero group: the
            // descriptor's stride between 8-row groups is the distance from the one to the other
            const uint32_t qoff = LO::kQ + (2 * set + (eq & 1)) * 2048;
            const uint32_t b_lo = umma_desc_lo(base + qoff, 16);
            const uint32_t b_hi = umma_desc_hi(LO::kQZero - qoff);
            const uint32_t d = tmem + set * 32 + (iq & 1) * 16;
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) {
              const uint32_t ao = ((kk >> 2) * (kDecKeys * 128) + (kk & 3) * 32) >> 4;
              const uint32_t bo = ((kk >> 2) * 1024 + (kk & 3) * 32) >> 4;
              if (kk == 0) umma_bf16_ss<false>(d, a_lo + ao, desc_hi, b_lo + bo, b_hi, idesc_qk);
              else umma_bf16_ss<true>(d, a_lo + ao, desc_hi, b_lo + bo, b_hi, idesc_qk);
            }
            tc_commit(bar(kDecBarSFull + 2 * set + (iq & 1)));   // the worker's scores are ready
            tc_commit(bar(kDecBarKEmpty + ks));              // the key stage is free
            ++iq;
            if (++wq.t == wq.t_end) { q_alive = dec_worker_next_chunk(wq, p); ++eq; }
            idle = 0;
            continue;
          }
        }
        if (++idle > 8u * kWaitLimit) { dead = true; break; }   // bounded: give up, flag, fall through
      }
      if (dead) atomicOr(s_timeouts, 8u);
    }
  } else if (warp >= 4) {
    // ------------------------------------------------------------ weight warps: one key per thread
    const int set = (warp - 4) >> 2, qd = warp & 3;          // worker; TMEM lane quarter this warp may touch
    const int my_tiles = set == 0 ? TA : TB;
    const uint32_t lane_addr = tmem + ((uint32_t)(qd * 32) << 16);
    const int wtid = (warp - 4 - 4 * set) * 32 + lane;       // 0..127 within the worker
    const int krow = qd * 32 + lane;                         // this thread's key row within a tile
    float *lpart = reinterpret_cast<float *>(gen + LO::kLpart) + set * 128;
    float *cutp = reinterpret_cast<float *>(gen + LO::kCut) + set * 512;   // [chunk parity][8 tiles][4 warps][8 rows]
    DecWorker cur, nxt;
    dec_worker_init(nxt, p, 2 * blockIdx.x + set, W);
    bool have_next = my_tiles > 0 && dec_worker_next_chunk(nxt, p);
    float z_next[NC], z_own[NC];                             // z_own: references this worker formed itself (one launch for the whole decode)
#pragma unroll
    for (int r = 0; r < NC; ++r) z_own[r] = 0.f;
    const bool own_z = f.mode == 1;
    pdl_wait();                                              // z comes from the kernel before
    // Staging the query rows (and the references) of chunk `w`, the worker's e-th, into query buffer e & 1, in two
    // steps so that the global loads are not waited for: stage_load requests them (one 16-byte piece of a row per
    // thread: at most 8 rows), stage_store puts them into shared memory a tile later.
    uint4 q_piece = make_uint4(0, 0, 0, 0);
    auto stage_load = [&](const DecWorker &w) {
      if (wtid < p.R * 16) {                                 // 16-byte chunk wtid % 16 of row wtid / 16
        const int r = wtid >> 4, c16 = wtid & 15;
        const int req = w.seq * p.stack + r / p.G, head = w.kvh * p.G + r % p.G;
        q_piece = *reinterpret_cast<const uint4 *>(p.q + (long long)req * p.q_stride_b + (long long)head * p.q_stride_h + c16 * 8);
      }
#pragma unroll
      for (int r = 0; r < NC; ++r) {
        const int req = w.seq * p.stack + r / p.G, head = w.kvh * p.G + r % p.G;
        z_next[r] = own_z ? z_own[r] : (r < p.R ? p.z[(long long)req * p.Hq + head] : INFINITY);   // rows past R: weight 0 by themselves
      }
    };
    auto stage_store = [&](int e) {
      uint8_t *qb = gen + LO::kQ + (2 * set + (e & 1)) * 2048;
      if (wtid < p.R * 16) {
        const int r = wtid >> 4, c16 = wtid & 15;
        *reinterpret_cast<uint4 *>(qb + (c16 >> 3) * 1024 + r * 128 + (((c16 & 7) ^ (r & 7)) << 4)) = q_piece;
      }
      fence_proxy_async_smem();                              // generic writes, then tensor-core (async proxy) reads
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(kDecBarQFull + 2 * set + (e & 1)));
    };
    bool stage_open = false;                                 // loads requested, not yet stored
    if (have_next) { stage_load(nxt); stage_store(0); }
    if (own_z) {
      // The reference of the CTA's (sequence, kv head) -- in this mode both workers scan chunks of the same one --
      // formed here while the key tiles travel: the 192 sampled keys' scores in blocks of 16 over the eight weight
      // warps, then a warp per row.  The scores sit in the first worker's weight buffers, which nothing else touches
      // before the first weights are handed over, and which are cleared again afterwards (a weight row nobody writes
      // must read as zero).
      const int ra = dec_radix_a(p), first = 2 * blockIdx.x;
      const int e_c = first % ra, e_kvh = (first / ra) % p.Hkv, e_seq = first / ra / p.Hkv;
      const int e_n = e_seq < p.num_seqs ? dec_seqlen(p, e_seq) : 0;
      if (e_c < num_chunks_of(e_n)) {                        // the CTA has a chunk (the same test in all eight warps)
        float (*sc)[kEstSamples] = reinterpret_cast<float (*)[kEstSamples]>(gen + LO::kP);
        float *zs = reinterpret_cast<float *>(gen + LO::kP + kMaxRows / 2 * kEstSamples * 4);
        const int ew = warp - 4;                             // 0..7
        const int lens[kMaxLevels] = {e_n, 0, 0, 0};
        const int n_samples = e_n < kEstSamples ? e_n : kEstSamples;
#pragma unroll 1
        for (int blk = ew; blk < kEstWarps; blk += 8)        // (one block at a time: two at once cost the whole kernel registers)
          est_score_blocks<D, 1>(f.est, e_seq, e_kvh, blk, 1, lane, e_n, lens, sc);   // one request per sequence in this mode
        named_bar_sync(1, 256);
        for (int g = ew; g < p.G; g += 8) {
          const float zval = est_reduce_row(sc[g], e_n, n_samples, lane);
          if (lane == 0) {
            zs[g] = zval;
            if (e_c == 0) f.est.z[(long long)e_seq * p.Hq + e_kvh * p.G + g] = zval;   // the first chunk's CTA publishes it
          }
        }
        named_bar_sync(1, 256);
#pragma unroll
        for (int r = 0; r < NC; ++r) z_next[r] = z_own[r] = r < p.R ? zs[r] : INFINITY;
        named_bar_sync(1, 256);                              // everybody has read the references
        *reinterpret_cast<uint4 *>(gen + LO::kP + (threadIdx.x - 128) * 32) = make_uint4(0, 0, 0, 0);
        *reinterpret_cast<uint4 *>(gen + LO::kP + (threadIdx.x - 128) * 32 + 16) = make_uint4(0, 0, 0, 0);
        fence_proxy_async_smem();
        named_bar_sync(1, 256);                              // cleared before the first weights are written
      }
    }
    unsigned long long st_fetched = 0, st_total = 0, st_skipped = 0;
    const int cut_exp = 24 + min(max((int)floorf(-p.neg_T), 0), 96);   // block tail: the cut mass's integer grid
    const float cut_scale = __int_as_float((127 + cut_exp) << 23), cut_unscale = __int_as_float((127 - cut_exp) << 23);
    const uint64_t vpol = policy_evict_first();
    const int vbox = p.vr;                                   // tokens per value box (16 or 32)
    const uint32_t gmask = vbox == 32 ? 0xffffffffu : 0xffffu;
    int i = 0;                                               // tiles this worker has been through
    DecWorker pend;                                          // the chunk whose slot is being written
    int pend_e = 0, pend_i = 0;
    // Chunk end, second half: the row sums from the four warps, the accumulator out of tensor memory, the block tail,
    // the slot.  A warp can only reach the chunk after next once every warp has been here (each tile's value product
    // needs all four warps' weights), so the parity-indexed buffers are free again when they are rewritten.
    auto flush_chunk = [&]() {
      const int pe = pend_e, par = pe & 1;
      float *slot = p.slots + (((long long)pend.seq * p.Hkv + pend.kvh) * p.max_slots + pend.c) * p.slot_stride;
      const float *lp = lpart + par * 64;
      if (TAIL || wtid < 32) {                               // the worker's first warp (block tail: every warp reads the cut mass)
        if (!wait_u(bar(kDecBarLFull + 2 * set + par), (uint32_t)((pe >> 1) & 1))) return;
      }
      if (wtid < 32) {
        // in the order of the key rows: lane quarters 0, 1, 2, 3
        if (lane < p.R) slot[(long long)p.R * D + lane] = ((lp[lane] + lp[16 + lane]) + lp[32 + lane]) + lp[48 + lane];
      }
      // block tail: this channel of the chunk's block means (up to 16 blocks), requested before the waits below -- as raw
      // bits from clamped block indices, converted and masked only where they are used: a select or a conversion right
      // behind each load would wait for it, sixteen memory latencies in a row
      unsigned short mraw[16];
      const int nblocks = TAIL ? (pend.n + 63) >> 6 : 1;
      if (TAIL) {
        const unsigned short *mrow = reinterpret_cast<const unsigned short *>(p.vmean) + (long long)pend.seq * p.vm_stride_seq +
                                     (long long)pend.kvh * p.vm_stride_head + krow;
#pragma unroll
        for (int j = 0; j < 16; ++j) mraw[j] = mrow[(long long)min(pend.t_first * 2 + j, nblocks - 1) * p.vm_stride_block];
      }
      if (!wait_u(bar(kDecBarPFree + 2 * set + (pend_i % PB)), (uint32_t)((pend_i / PB) & 1))) return;   // the chunk's last product
      tc_fence_after();
      float o[NPV];
      tmem_ld_cols<NPV>(lane_addr + 64 + set * 32 + par * 16, o);   // this thread's channel: every row's P_hi part, then the P_lo parts
      tc_fence_before();
      float tl[NC];
#pragma unroll
      for (int r = 0; r < NC; ++r) tl[r] = 0.f;
      if (TAIL) {
        // cut mass x block mean, the chunk's blocks in order (a tile is two 64-key blocks, a block two warps' keys; tiles
        // and blocks the chunk does not have carry zero cut mass and a zero mean)
        const float *cp = cutp + par * 256;
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const bool there = j < 2 * (pend.t_end - pend.t_first) && pend.t_first * 2 + j < nblocks;
          const float mean = there ? __uint_as_float((uint32_t)mraw[j] << 16) : 0.f;
#pragma unroll
          for (int r = 0; r < NC; ++r)
            tl[r] = fmaf(cp[(j * 2) * 8 + r] + cp[(j * 2 + 1) * 8 + r], mean, tl[r]);
        }
      }
#pragma unroll
      for (int r = 0; r < NC; ++r)
        if (r < p.R) slot[(long long)r * D + krow] = (o[r] + o[NPV / 2 + r]) + tl[r];
    };
    for (int e = 0; have_next && !dead; ++e) {
      cur = nxt;
      float z[NC];
#pragma unroll
      for (int r = 0; r < NC; ++r) z[r] = z_next[r];
      have_next = dec_worker_next_chunk(nxt, p);
      if (have_next) { stage_load(nxt); stage_open = true; } // one chunk ahead: the score products never wait for rows
      const int n = cur.n, dstart = draft_start(p, n);
      float L[NC];
#pragma unroll
      for (int r = 0; r < NC; ++r) L[r] = 0.f;
      int it = 0;
      for (; cur.t < cur.t_end; ++cur.t, ++i) {
        it = dec_global_index(set, i, TA, TB);
        const int vs = it % VS;
        const int key = cur.t * kDecKeys + krow;
        const int tok_w = cur.t * kDecKeys + qd * 32;        // first key of this warp's 32
        int pg0 = 0, pg1 = 0;                                // pages of the warp's value groups, fetched ahead of their use
        if (GATED && p.paged) {
          const int *pt = p.page_table + (long long)cur.seq * p.max_pages;
          if (tok_w < n) pg0 = pt[tok_w >> p.page_shift];
          if (tok_w + 16 < n) pg1 = pt[(tok_w + 16) >> p.page_shift];
        }
        // the tcgen05 loads are warp-wide: the warp takes them together or not at all
        if (!wait_u(bar(kDecBarSFull + 2 * set + (i & 1)), (uint32_t)((i >> 1) & 1))) break;
        tc_fence_after();
        float s[NC];
        tmem_ld_cols<NC>(lane_addr + set * 32 + (i & 1) * 16, s);
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(kDecBarSEmpty + 2 * set + (i & 1)));   // this score buffer may be rewritten
        const bool valid = key < n;
        const bool drafts = p.draft_len > 0 && key >= dstart;
        // final scores s - Z in binades, and the verdict: does some row keep this key?
        float x[NC];
        bool any_live = false;
#pragma unroll
        for (int r = 0; r < NC; ++r) {
          x[r] = valid ? fmaf(s[r], p.scale_log2, -z[r]) : -INFINITY;   // select: rows past n may hold anything
          if (drafts && r < p.R && !draft_ok(p.draft_mask[cur.seq * p.stack + r / p.G], key, dstart)) x[r] = -INFINITY;
          any_live |= GATED ? (x[r] >= p.neg_T) : true;
        }
        // this tile's value stage is free once the value product of the tile VS back in the CTA's order is over (the
        // other worker's, while the two alternate)
        if (it >= VS && !wait_u(bar(kDecBarPvDone + vs), (uint32_t)((it / VS - 1) & 1))) break;
        const uint32_t vfull = bar(kDecBarVFull + vs);
        uint32_t live32 = 0xffffffffu;                       // which of the warp's 32 keys some row keeps
        if (GATED) {
          // requests for the value rows some row keeps, before anything else is done with the scores, per group of vbox
          // keys: a mostly-live group whole as one tensor-map box per 64 channels (never past the sequence end),
          // otherwise its live rows one by one
          const uint32_t fetch = __ballot_sync(0xffffffffu, any_live);
          live32 = fetch;
          const uint32_t vdst = base + OFF_V + vs * LO::kTile;
          bool rows = false;
          for (int gq = 0; gq * vbox < 32; ++gq) {
            uint32_t m = (fetch >> (gq * vbox)) & gmask;
            const int tok = tok_w + gq * vbox;
            const int nvalid = min(vbox, max(0, n - tok));
            st_total += nvalid;
            if (m == 0u) { st_skipped += nvalid > 0 ? 1 : 0; continue; }
            int c_seq = cur.seq, c_tok = tok;
            if (p.paged) {
              c_seq = min(max(gq ? pg1 : pg0, 0), p.num_pages - 1);
              c_tok = tok & page_mask;
            }
            const int row0 = qd * 32 + gq * vbox;            // the group's first row within the tile
            if (__popc(m) >= p.box_min && tok + vbox <= n) {
              st_fetched += vbox;
              if (lane == 0) {
                mbar_expect_tx_only(vfull, vbox * D * 2);
                const int c1 = p.pos_tok == 1 ? c_tok : (p.pos_head == 1 ? cur.kvh : c_seq);
                const int c2 = p.pos_tok == 2 ? c_tok : (p.pos_head == 2 ? cur.kvh : c_seq);
                const int c3 = p.pos_tok == 3 ? c_tok : (p.pos_head == 3 ? cur.kvh : c_seq);
#pragma unroll
                for (int h = 0; h < 2; ++h) tma_load_4d(vdst + (h * kDecKeys + row0) * 128, &tmV, vfull, h * 64, c1, c2, c3, vpol);
              }
            } else {
              st_fetched += __popc(m);
              rows = true;
              const __nv_bfloat16 *src = p.v + (long long)c_seq * p.v_stride_seq + (long long)c_tok * p.v_stride_tok +
                                         (long long)cur.kvh * p.v_stride_head + (lane & 15) * 8;
              const uint32_t dst = vdst + ((lane & 15) >> 3) * (kDecKeys * 128);
              while (m) {                                    // two live rows per warp-wide copy: lanes 0..15, 16..31
                const int r0 = __ffs(m) - 1;
                m &= m - 1;
                const int r1 = m ? __ffs(m) - 1 : -1;
                m &= m - 1;
                const int row = lane < 16 ? r0 : r1;
                if (row >= 0)
                  cp_async_16(dst + (row0 + row) * 128 + ((((lane & 15) ^ row) & 7) << 4), src + (long long)row * p.v_stride_tok, 16u);
              }
            }
          }
          if (rows) cp_async_mbar_arrive(vfull);             // this lane's copies hold the phase open
          __syncwarp();
          if (lane == 0) mbar_arrive(vfull);                 // this warp's requests are out
        } else {
          st_total += min(32, max(0, n - tok_w));
          if (cur.t * kDecKeys + kDecKeys > n) {             // ragged tail: value rows past n may hold anything
            if (!wait_u(vfull, (uint32_t)((it / VS) & 1))) break;
            if (!valid) {
#pragma unroll
              for (int c16 = 0; c16 < 16; ++c16)
                *reinterpret_cast<uint4 *>(gen + OFF_V + vs * LO::kTile + tile_off(krow, c16, kDecKeys)) = make_uint4(0, 0, 0, 0);
            }
          }
        }
        // final weights 2^(s - Z), their two-term BF16 split, and this thread's share of L
        uint32_t hi16[NC], lo16[NC];
#pragma unroll
        for (int r = 0; r < NC; ++r) {
          const float pw = ex2_approx(x[r]);                 // 2^-inf = 0
          const bool live = GATED ? (x[r] >= p.neg_T) : true;
          const float pm = live ? pw : 0.f;
          const float h = __bfloat162float(__float2bfloat16_rn(pm));
          const float g = __bfloat162float(__float2bfloat16_rn(pm - h));
          L[r] += (h + g) + (pw - pm);                       // L sums the weights the products use; cut keys add p
          hi16[r] = __float_as_uint(h) >> 16;
          lo16[r] = __float_as_uint(g) >> 16;
          if (TAIL) {
            // the warp's cut mass of row r in this tile: a cut weight is below 2^-T, so on the grid 2^-(24 + floor T) it is
            // an integer under 2^24 and the warp's 32 add up in ONE order-free integer reduction (five dependent shuffles
            // per row and tile sat on the weight warps' critical chain); weights under half a grid step count as zero
            const int ci = __reduce_add_sync(0xffffffffu, __float2int_rn((pw - pm) * cut_scale));
            if (lane == 0) cutp[(((e & 1) * 8 + (cur.t - cur.t_first)) * 4 + qd) * 8 + r] = (float)ci * cut_unscale;
          }
        }
        // the worker's weight buffer is free once its own value product PB tiles back is over
        if (i >= PB && !wait_u(bar(kDecBarPFree + 2 * set + (i % PB)), (uint32_t)((i / PB - 1) & 1))) break;
        // (the verdict word travels with the weight buffer: the issuing thread skips the product of a tile nobody keeps a key of)
        if (GATED && lane == 0) reinterpret_cast<uint32_t *>(gen + LO::kBar + kDecLiveFlags)[(set * 2 + (i % PB)) * 4 + qd] = live32;
        // weights: B operand [2 key halves][NPV rows][128 B], K-major, swizzled like a tensor-map box; P_hi of row r in
        // row r, P_lo in row NPV / 2 + r (the same swizzle phase: NPV / 2 is a multiple of 8)
        {
          uint8_t *ph = gen + LO::kP + set * 8192 + (i % PB) * PBYTES + (krow >> 6) * (NPV * 128) + (krow & 7) * 2;
          const int kc = (krow >> 3) & 7;
#pragma unroll
          for (int r = 0; r < NC; ++r) {
            const int off = r * 128 + ((kc ^ (r & 7)) << 4);
            *reinterpret_cast<uint16_t *>(ph + off) = (uint16_t)hi16[r];
            *reinterpret_cast<uint16_t *>(ph + (NPV / 2) * 128 + off) = (uint16_t)lo16[r];
          }
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(kDecBarPFull + 2 * set + (i % PB)));
        if (stage_open) { stage_store(e + 1); stage_open = false; }   // the next chunk's rows, requested a tile ago
        if (dead) break;
      }
      if (dead) break;
      // chunk end: L over the warp in a fixed shuffle order, handed to the worker's first warp through shared memory (the
      // buffer alternates with the chunk's parity), then the accumulator out of tensor memory and the slot (flush_chunk).
      // (Putting the second half off behind the next chunk's first tile was measured: no gain on 256-key chunks, 2 % lost
      // on long ones.)
#pragma unroll
      for (int r = 0; r < NC; ++r) {
#pragma unroll
        for (int m = 16; m >= 1; m >>= 1) L[r] += __shfl_xor_sync(0xffffffffu, L[r], m);
        if (lane == 0) lpart[(e & 1) * 64 + qd * 16 + r] = L[r];
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(kDecBarLFull + 2 * set + (e & 1)));
      pend = cur; pend_e = e; pend_i = i - 1;
      flush_chunk();
    }
    if (lane == 0) {
      if (dead) atomicOr(s_timeouts, 16u);
      if (st_total) {
        atomicAdd(s_stats, GATED ? st_fetched : st_total);
        atomicAdd(s_stats + 1, st_total);
      }
      if (st_skipped) atomicAdd(s_stats + 2, st_skipped);
    }
  }

  // every warp meets here; the allocating warp returns the tensor memory
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, kDecTmemCols);
  }
  if (f.mode) {
    // the whole decode in this launch: every CTA's slots (and the cleared header) are out before any row is added
    __threadfence();
    cooperative_groups::this_grid().sync();
  }
  if (threadIdx.x == 0) {
    // what the roles of this CTA recorded, into the workspace header (cleared by the kernel before, or above)
    pdl_wait();
    if (*s_timeouts) atomicOr(&p.hdr->wait_timeouts, *s_timeouts);
    if (s_stats[1]) {
      atomicAdd(reinterpret_cast<unsigned long long *>(&p.hdr->v_rows_fetched), s_stats[0]);
      atomicAdd(reinterpret_cast<unsigned long long *>(&p.hdr->v_rows_total), s_stats[1]);
    }
    if (s_stats[2]) atomicAdd(reinterpret_cast<unsigned long long *>(&p.hdr->v_slices_skipped), s_stats[2]);
  }
  if (f.mode && warp < 8) {
    // the order-free partial add, a row at a time per CTA: eight warps share the row's slots (the key ring is free now)
    unsigned (*s_max)[D + 1] = reinterpret_cast<unsigned (*)[D + 1]>(gen);
    long long (*s_sum)[D + 1] = reinterpret_cast<long long (*)[D + 1]>(gen + 8 * (D + 1) * 4 + 8);
    const long long n_rows = (long long)p.num_seqs * p.Hq;
    for (long long row = blockIdx.x; row < n_rows; row += gridDim.x) {
      // a sequence without keys has no worker: its rows' references are written here (the estimate of no key is 0)
      if (f.mode == 1 && threadIdx.x == 0 && dec_seqlen(p, (int)(row / p.Hq)) == 0) f.est.z[row] = 0.f;
      if (p.max_slots <= 8 * kMergeResident)                 // a warp's share of the slots stays in registers
        merge_row<D / 32, true>(f.mrg, 8, row, true, warp, warp, lane, s_max, s_sum, [] { named_bar_sync(3, 256); });
      else
        merge_row<D / 32, false>(f.mrg, 8, row, true, warp, warp, lane, s_max, s_sum, [] { named_bar_sync(3, 256); });
      named_bar_sync(3, 256);                                // the staging arrays are reused by the next row
    }
  }
}

}  // namespace fold
