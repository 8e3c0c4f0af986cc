// Stacked-row scan on the 5th-generation tensor cores (tcgen05 + TMEM), head_dim 128.
//
// The shared-prefix level of a cascade stacks the query rows of every request that holds the
// prefix (Section 4, "Value product"; Appendix "Tile layouts"): with hundreds of rows per
// (sequence, kv head) the scan is a dense contraction, not a stream, so it runs on tcgen05.mma
// with the accumulators in tensor memory.  One CTA owns 128 query rows (M = 128) of one
// (sequence, kv head) and walks the 64-key tiles of its canonical chunks:
//
//   producer warp   TMA: K and V tiles -> 6-stage shared-memory ring (same tiles as dense decode); the tiles come
//                   from L2 (every row tile of a kv head reads them) and the ring has to cover that latency
//   MMA warp        S = Q K^T        (A = Q in tensor memory;  B = K tile, K-major;  N = 64 keys)
//                   O += P_hi V + P_lo V   (A = P in tensor memory;  B = V tile, MN-major;  N = 128)
//   8 weight warps  two threads per query row (the row's TMEM lane; each takes 32 of the tile's 64 keys and
//                   64 of the 128 channels): tcgen05.ld S, final weights 2^(s - Z) with the depth gate,
//                   L in a register, two-term BF16 P -> tensor memory by tcgen05.st
//
// Both A operands live in tensor memory (a row of A is a TMEM lane, two BF16 per 32-bit column), so the only
// shared-memory traffic is the K and V tiles: with Q and P in shared memory the operand reads alone (112 KB per
// tile) exceeded what the SM's shared memory delivers in the time the products take.  S is double-buffered, so
// the scores of tile t+1 are computed while the weights of tile t are formed; P has one buffer (the value
// product of tile t is over long before the weights of t+1 are ready).  No maximum is tracked and nothing is
// rescaled: the accumulator O is only ever added to.  At a chunk's end each thread reads its row of O from
// TMEM and writes it, with its L, to the chunk's slot.
#pragma once

#include "fold_scan.cuh"

namespace fold {

constexpr int kUmmaThreads = 10 * 32;                // producer, MMA, 8 weight warps
constexpr int kUmmaWeightThreads = 8 * 32;
constexpr int kUmmaRows = 128;                       // query rows per CTA (MMA M)
constexpr int kUmmaStages = 6;
constexpr int kUmmaTmemCols = 512;                   // S0 [0,64)  S1 [64,128)  O [128,256)  Q [256,320)  P_hi [320,352)  P_lo [352,384)  cut mass hi [384,400) lo [400,416)
constexpr int kUmmaColQ = 256, kUmmaColPhi = 320, kUmmaColPlo = 352, kUmmaColCutHi = 384, kUmmaColCutLo = 400;

struct UmmaLayout {                                  // byte offsets from a 1 KB-aligned base
  static constexpr int kRing = 0;                                // stages x (K tile 16 KB + V tile 16 KB)
  static constexpr int kStage = 32768;
  static constexpr int kBar = kRing + kUmmaStages * kStage;
  static constexpr int kLbuf = kBar + 256;                       // 128 floats: the second half-row's share of L
  static constexpr int kMean = kBar + 1024;                      // block tail: the chunk's block means [2 halves][16 blocks][128 B], swizzled
  static constexpr int kTotal = kMean + 4096 + 1024;             // + alignment slack
};

// ---------------------------------------------------------------- tcgen05 wrappers
__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(cols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A * B, BF16 inputs, FP32 accumulate, issued by one thread, with the A operand in tensor memory (row r of A = TMEM lane r, K elements packed two per column).
// The B descriptor comes as two 32-bit words: the issuing thread's instruction stream is the critical path of
// the whole CTA, and stepping a descriptor is then one 32-bit add on the low word.
template <bool ACC>
__device__ __forceinline__ void umma_bf16_ta(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t b_hi, uint32_t idesc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 bd;\n\t"
      "setp.ne.b32 p, %5, 0;\n\t"
      "mov.b64 bd, {%2, %3};\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], bd, %4, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(b_hi), "r"(idesc), "n"(ACC ? 1 : 0)
      : "memory");
}
__device__ __forceinline__ void umma_bf16_ta(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t b_hi, uint32_t idesc,
                                             bool accumulate) {
  if (accumulate) umma_bf16_ta<true>(d_tmem, a_tmem, b_lo, b_hi, idesc);
  else umma_bf16_ta<false>(d_tmem, a_tmem, b_lo, b_hi, idesc);
}
// Low and high words of a shared-memory matrix descriptor (128-byte swizzle, version 1); offsets in bytes.
__device__ __forceinline__ uint32_t umma_desc_lo(uint32_t smem_addr, uint32_t lbo) {
  return ((smem_addr >> 4) & 0x3fffu) | (((lbo >> 4) & 0x3fffu) << 16);
}
__host__ __device__ constexpr uint32_t umma_desc_hi(uint32_t sbo) {
  return ((sbo >> 4) & 0x3fffu) | (1u << 14) | (2u << 29);
}
// 16 / 32 consecutive 32-bit columns of this thread's TMEM lane, written from registers.
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
        "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}
__device__ __forceinline__ void tmem_st8(uint32_t taddr, const uint32_t (&r)[8]) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
               ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
               : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
// 32 consecutive FP32 columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

// Instruction descriptor: FP32 accumulate, BF16 A and B, M = 128.
__host__ __device__ constexpr uint32_t umma_idesc(int n, int b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)b_mn_major << 16) | ((uint32_t)(n >> 3) << 17) |
         ((uint32_t)(kUmmaRows >> 4) << 24);
}

// TAIL (with GATED; Section 4 "Depth as a dial", the block model's mean): a row's cut keys add their summed weight
// times the mean value row of their 64-key block -- a tile here.  Each thread keeps the cut mass of its 32 keys per tile
// of the chunk; with the chunk's last weights it writes them, split into two BF16 terms like the weights, to 16 more
// columns of its lane (the two threads of a row own 16 K slots each: slot 16 half + block), the chunk's block means
// go to shared memory as a [16 blocks x 128 channels] MN-major tile, and four more products
// O += cut_hi M + cut_lo M (K = 16 each, the same tile for both halves' slots) follow the chunk's last value product.
template <bool GATED, bool TAIL = false>
__global__ void __launch_bounds__(kUmmaThreads, 1)
fold_scan_stacked_umma_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                              const ScanParams p) {
  constexpr int D = 128;
  using LO = UmmaLayout;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t *gen = smem_raw + (base - raw);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int row_tiles = (p.R + kUmmaRows - 1) / kUmmaRows;
  const int rt = blockIdx.x % row_tiles, split = blockIdx.x / row_tiles;
  const int kvh = blockIdx.y, seq = blockIdx.z;
  const SeqWork w = seq_work(p, seq);
  if (split >= w.n_chunks) return;
  const int R = p.R, n = w.n;
  const int dstart = draft_start(p, n);

  // barriers (8 bytes each): kv_full[stages] pv_done[stages] s_full[2] s_empty[2] p_full o_empty.
  // pv_done[stage] completes when the value product of the tile in `stage` has: it frees the stage for the producer,
  // P for the weight warps, and at a chunk's end says that O is final -- one commit per tile serves all three (a
  // commit holds the issuing thread for on the order of a hundred cycles).
  const uint32_t bar = base + LO::kBar;
  const uint32_t kv_full = bar, pv_done = bar + 8 * kUmmaStages, s_full = bar + 16 * kUmmaStages, s_empty = s_full + 16,
                 p_full = s_full + 32, o_empty = s_full + 40, tmem_slot = bar + 192;
  if (threadIdx.x == 0) {
    for (int s = 0; s < kUmmaStages; ++s) { mbar_init(kv_full + 8u * s, 1); mbar_init(pv_done + 8u * s, 1); }
    for (int b = 0; b < 2; ++b) {
      mbar_init(s_full + 8u * b, 1);
      mbar_init(s_empty + 8u * b, kUmmaWeightThreads / 32);      // one arrival per weight warp
    }
    mbar_init(p_full, kUmmaWeightThreads / 32);
    mbar_init(o_empty, kUmmaWeightThreads / 32);
    mbar_fence_init();
  }
  if (warp == 1) tmem_alloc(tmem_slot, kUmmaTmemCols);
  pdl_launch_dependents();
  pdl_wait();                                                // q and z come from earlier work

  tc_fence_before();
  __syncthreads();                                           // barriers initialised, TMEM allocated
  tc_fence_after();
  const uint32_t tmem = *reinterpret_cast<volatile uint32_t *>(gen + LO::kBar + 192);

  // the weight warps put their query rows into tensor memory: row r of the tile = lane r, channel pairs = columns
  const int row = (warp & 3) * 32 + lane;                    // TMEM lane == query row of the tile
  const int ch = warp >= 6 ? 1 : 0;                          // which half of the tile's keys / of the channels
  const int r_glob = rt * kUmmaRows + row;
  const uint32_t lane_addr = tmem + ((uint32_t)((warp & 3) * 32) << 16);
  float z_row = 0.f;
  uint32_t dm_row = 0xffffffffu;                             // the row's request's draft mask
  if (warp >= 2) {
    const bool valid_row = r_glob < R;
    const int req = seq * p.stack + r_glob / p.G, head = kvh * p.G + r_glob % p.G;
    const uint4 *qrow = reinterpret_cast<const uint4 *>(p.q + (long long)req * p.q_stride_b + (long long)head * p.q_stride_h);
#pragma unroll
    for (int c = 0; c < 2; ++c) {                            // 16 columns = 32 channels at a time
      uint32_t qw[16];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const uint4 v = valid_row ? qrow[ch * 8 + c * 4 + i] : make_uint4(0, 0, 0, 0);
        qw[4 * i] = v.x; qw[4 * i + 1] = v.y; qw[4 * i + 2] = v.z; qw[4 * i + 3] = v.w;
      }
      tmem_st16(lane_addr + kUmmaColQ + ch * 32 + c * 16, qw);
    }
    tmem_st_wait();
    z_row = valid_row ? p.z[(long long)req * p.Hq + head] : INFINITY;
    if (p.draft_len && valid_row) dm_row = p.draft_mask[req];
  }
  tc_fence_before();
  __syncthreads();                                           // Q is in tensor memory
  tc_fence_after();

  bool dead = false;
  if (warp == 0) {
    // ------------------------------------------------------------ producer
    if (lane == 0) {
      ScanParams pp = p;
      pp.stages = kUmmaStages;
      produce_tiles<D, true, LO::kStage>(&tmK, &tmV, pp, w, split, kvh, seq, base + LO::kRing, kv_full, pv_done);
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    // The whole warp walks the loop and its waits in step; one lane issues.  Everything an MMA takes as operand
    // (tensor-memory addresses, descriptor words) is then the same in every lane, which lets it be kept in
    // uniform registers instead of being moved there before every instruction.
    {
      const bool leader = lane == 0;
      const uint32_t tm = __shfl_sync(0xffffffffu, tmem, 0);
      SeqWork wu;
      wu.n = __shfl_sync(0xffffffffu, w.n, 0); wu.n_tiles = __shfl_sync(0xffffffffu, w.n_tiles, 0);
      wu.ctiles = __shfl_sync(0xffffffffu, w.ctiles, 0); wu.n_chunks = __shfl_sync(0xffffffffu, w.n_chunks, 0);
      constexpr uint32_t idesc_qk = umma_idesc(64, 0), idesc_pv = umma_idesc(128, 1);
      const uint32_t ring_lo = umma_desc_lo(base + LO::kRing, 0);
      auto issue_qk = [&](int it, int stage) {               // S[it & 1] = Q K^T for the tile in `stage`
        const int b = it & 1;
        if (!mbar_wait(kv_full + 8u * stage, (uint32_t)((it / kUmmaStages) & 1), dead)) return;
        if (it >= 2 && !mbar_wait(s_empty + 8u * b, (uint32_t)(((it >> 1) - 1) & 1), dead)) return;
        tc_fence_after();
        // K tile [2 halves][64 keys][128 B]: K step kk = 32 bytes along the row, half kk / 4; LBO 16
        const uint32_t k_lo = ring_lo + ((uint32_t)(stage * LO::kStage) >> 4) + (1u << 16);
        const uint32_t s_t = tm + b * 64;
        if (leader) {
          umma_bf16_ta<false>(s_t, tm + kUmmaColQ, k_lo, umma_desc_hi(1024), idesc_qk);
#pragma unroll
          for (int kk = 1; kk < D / 16; ++kk)
            umma_bf16_ta<true>(s_t, tm + kUmmaColQ + kk * 8, k_lo + (((kk >> 2) * (kTileKeys * 128) + (kk & 3) * 32) >> 4),
                               umma_desc_hi(1024), idesc_qk);
          tc_commit(s_full + 8u * b);
        }
        __syncwarp();
      };
      int it = 0, chunk_i = 0;
      TileCursor k = cursor_begin(wu, split);
      if (cursor_valid(k, wu)) issue_qk(0, 0);
      bool first_of_chunk = true;
      while (cursor_valid(k, wu) && !dead) {
        const int stage = it % kUmmaStages;
        TileCursor kn = k;
        const bool chunk_ends = cursor_next(kn, wu, p.num_splits);
        if (cursor_valid(kn, wu)) issue_qk(it + 1, (it + 1) % kUmmaStages);
        // O += P V for tile `it`
        if (first_of_chunk && chunk_i > 0 && !mbar_wait(o_empty, (uint32_t)((chunk_i - 1) & 1), dead)) break;
        if (!mbar_wait(p_full, (uint32_t)(it & 1), dead)) break;
        tc_fence_after();
        // V tile [2 halves][64 keys][128 B], MN-major: 16 keys = 2048 bytes per K step, halves 8192 bytes apart (LBO)
        const uint32_t v_lo = ring_lo + ((uint32_t)(stage * LO::kStage + 16384) >> 4) + ((8192u >> 4) << 16);
        if (leader) {
          umma_bf16_ta(tm + 128, tm + kUmmaColPhi, v_lo, umma_desc_hi(1024), idesc_pv, !first_of_chunk);
#pragma unroll
          for (int i = 1; i < 2 * (kTileKeys / 16); ++i) {
            const int term = i / (kTileKeys / 16), j = i % (kTileKeys / 16);
            umma_bf16_ta<true>(tm + 128, tm + (term ? kUmmaColPlo : kUmmaColPhi) + j * 8, v_lo + j * (2048 >> 4),
                               umma_desc_hi(1024), idesc_pv);
          }
          if (TAIL && chunk_ends) {
            // the chunk's tail: cut mass [128 rows, 2 x 16 slots] x block means [16, 128], the means for both slot groups
            const uint32_t m_lo = umma_desc_lo(base + LO::kMean, 2048);
#pragma unroll
            for (int i = 0; i < 4; ++i)
              umma_bf16_ta<true>(tm + 128, tm + ((i & 2) ? kUmmaColCutLo : kUmmaColCutHi) + (i & 1) * 8, m_lo,
                                 umma_desc_hi(1024), idesc_pv);
          }
          tc_commit(pv_done + 8u * stage);
        }
        __syncwarp();
        if (chunk_ends) ++chunk_i;
        first_of_chunk = chunk_ends;
        k = kn;
        ++it;
      }
      if (dead && leader) atomicOr(&p.hdr->wait_timeouts, 8u);
    }
  } else {
    // ------------------------------------------------------------ weight warps: one query row per thread
    const bool valid_row = r_glob < R;
    float l_row = 0.f;
    float cut[TAIL ? 16 : 1];                                // this thread's cut mass per tile (= 64-key block) of the chunk
#pragma unroll
    for (int i = 0; i < (TAIL ? 16 : 1); ++i) cut[i] = 0.f;
    int it = 0, chunk_i = 0;
    for (TileCursor k = cursor_begin(w, split); cursor_valid(k, w); ++it) {
      const int b = it & 1, stage = it % kUmmaStages;
      const int key_base = k.t * kTileKeys;
      TileCursor k_after = k;
      const bool last_of_chunk = cursor_next(k_after, w, p.num_splits);
      uint4 mean_piece = make_uint4(0, 0, 0, 0);             // block tail: this thread's 16 bytes of the chunk's means, requested early
      if (TAIL && last_of_chunk) {
        const int tw = threadIdx.x - 64, blk = k.c * w.ctiles + (tw >> 4);
        if ((tw >> 4) < w.ctiles && blk * 64 < n)
          mean_piece = *reinterpret_cast<const uint4 *>(p.vmean + (long long)seq * p.vm_stride_seq + (long long)blk * p.vm_stride_block +
                                                        (long long)kvh * p.vm_stride_head + (tw & 15) * 8);
      }
      float cm = 0.f;
      uint32_t ph[16], pl[16];                               // this thread's 32 weights, BF16 pairs: hi and lo terms
      // the tcgen05 loads and stores below are warp-wide: the warp takes them together or not at all
      const bool have_s = __all_sync(0xffffffffu, mbar_wait(s_full + 8u * b, (uint32_t)((it >> 1) & 1), dead));
      if (have_s) {
        tc_fence_after();
        float s[32];
        tmem_ld32(lane_addr + b * 64 + ch * 32, s);
        // rows beyond R carry z = +inf, so their weights vanish by themselves; keys beyond n only occur in a tail tile
        const int key_lim = n - (key_base + ch * 32);        // this thread's keys j < key_lim exist
        if (key_base + kTileKeys > dstart) {                 // draft keys: the row only uses the ones its mask names
#pragma unroll
          for (int j = 0; j < 32; ++j)
            if (!draft_ok(dm_row, key_base + ch * 32 + j, dstart)) s[j] = -INFINITY;
        }
        auto weights = [&](auto tail) {
#pragma unroll
          for (int j = 0; j < 32; j += 2) {
            float pw[2], pm[2];
#pragma unroll
            for (int e = 0; e < 2; ++e) {
              float x = fmaf(s[j + e], p.scale_log2, -z_row);
              if (decltype(tail)::value) x = (j + e) < key_lim ? x : -INFINITY;
              pw[e] = ex2_approx(x);
              pm[e] = (!GATED || x >= p.neg_T) ? pw[e] : 0.f;
            }
            const uint32_t hi2 = pack_bf16(pm[0], pm[1]);
            const float h0 = __uint_as_float(hi2 << 16), h1 = __uint_as_float(hi2 & 0xffff0000u);
            const uint32_t lo2 = pack_bf16(pm[0] - h0, pm[1] - h1);
            const float g0 = __uint_as_float(lo2 << 16), g1 = __uint_as_float(lo2 & 0xffff0000u);
            l_row += ((h0 + g0) + (pw[0] - pm[0])) + ((h1 + g1) + (pw[1] - pm[1]));
            if (TAIL) cm += (pw[0] - pm[0]) + (pw[1] - pm[1]);
            ph[j / 2] = hi2;
            pl[j / 2] = lo2;
          }
        };
        if (key_lim >= 32) weights(std::false_type{}); else weights(std::true_type{});
        tc_fence_before();
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(s_empty + 8u * b);          // S[b] may be overwritten
      // P is free once the value product of the tile before has completed
      if (__all_sync(0xffffffffu, it < 1 || mbar_wait(pv_done + 8u * ((it - 1) % kUmmaStages),
                                                        (uint32_t)(((it - 1) / kUmmaStages) & 1), dead))) {
        tmem_st16(lane_addr + kUmmaColPhi + ch * 16, ph);    // this thread's 32 keys = 16 columns of its lane
        tmem_st16(lane_addr + kUmmaColPlo + ch * 16, pl);
        if (TAIL) {
          cut[k.t - k.c * w.ctiles] = cm;
          if (last_of_chunk) {
            // the chunk's cut mass in two BF16 terms, this thread's 16 slots = 8 columns of each term; and the means
            uint32_t chi[8], clo[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const float c0 = cut[2 * i], c1 = cut[2 * i + 1];
              chi[i] = pack_bf16(c0, c1);
              clo[i] = pack_bf16(c0 - __uint_as_float(chi[i] << 16), c1 - __uint_as_float(chi[i] & 0xffff0000u));
              cut[2 * i] = cut[2 * i + 1] = 0.f;
            }
            tmem_st8(lane_addr + kUmmaColCutHi + ch * 8, chi);
            tmem_st8(lane_addr + kUmmaColCutLo + ch * 8, clo);
            const int tw = threadIdx.x - 64;
            *reinterpret_cast<uint4 *>(gen + LO::kMean + tile_off(tw >> 4, tw & 15, 16)) = mean_piece;
            fence_proxy_async_smem();                        // generic writes, then tensor-core (async proxy) reads
          }
        }
        tmem_st_wait();
        if (key_base + kTileKeys > n) {                      // ragged tail: value rows past n may hold anything
          const int tw = threadIdx.x - 64;
          for (int i = tw; i < kTileKeys * 16; i += kUmmaWeightThreads) {
            const int vr_ = i >> 4, c16 = i & 15;
            if (key_base + vr_ >= n)
              *reinterpret_cast<uint4 *>(gen + LO::kRing + stage * LO::kStage + 16384 + tile_off(vr_, c16, kTileKeys)) =
                  make_uint4(0, 0, 0, 0);
          }
          fence_proxy_async_smem();                          // generic writes, then tensor-core (async proxy) reads
        }
        tc_fence_before();
      }
      __syncwarp();                                          // every lane's writes and proxy fence are done
      if (lane == 0) mbar_arrive(p_full);
      const int c_done = k.c;
      if (cursor_next(k, w, p.num_splits)) {
        // chunk end: this thread's half of its row of O, and the row's L, go to the chunk's slot
        float *slot = p.slots + (((long long)seq * p.Hkv + kvh) * p.max_slots + c_done) * p.slot_stride;
        float *lbuf = reinterpret_cast<float *>(gen + LO::kLbuf);
        if (ch == 1) lbuf[row] = l_row;
        if (__all_sync(0xffffffffu, mbar_wait(pv_done + 8u * stage, (uint32_t)((it / kUmmaStages) & 1), dead))) {
          tc_fence_after();
#pragma unroll 1
          for (int q4 = ch * 2; q4 < ch * 2 + 2; ++q4) {
            float o[32];
            tmem_ld32(lane_addr + 128 + q4 * 32, o);
            if (valid_row) {
              float4 *dst = reinterpret_cast<float4 *>(slot + (long long)r_glob * D + q4 * 32);
#pragma unroll
              for (int i = 0; i < 8; ++i) dst[i] = make_float4(o[4 * i], o[4 * i + 1], o[4 * i + 2], o[4 * i + 3]);
            }
          }
          tc_fence_before();
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(o_empty);
        asm volatile("bar.sync 1, %0;" ::"n"(kUmmaWeightThreads) : "memory");   // both halves of every row are in
        if (ch == 0 && valid_row) slot[(long long)R * D + r_glob] = l_row + lbuf[row];
        asm volatile("bar.sync 1, %0;" ::"n"(kUmmaWeightThreads) : "memory");   // lbuf may be rewritten
        l_row = 0.f;
        ++chunk_i;
      }
    }
    if (dead && lane == 0) atomicOr(&p.hdr->wait_timeouts, 16u);
    if (threadIdx.x == 64 && rt == 0) {                      // every value row is read once per row-tile pass
      unsigned long long keys = 0;
      for (int c = split; c < w.n_chunks; c += p.num_splits)
        keys += min((c + 1) * w.ctiles * kTileKeys, n) - c * w.ctiles * kTileKeys;
      atomicAdd(reinterpret_cast<unsigned long long *>(&p.hdr->v_rows_fetched), keys);
      atomicAdd(reinterpret_cast<unsigned long long *>(&p.hdr->v_rows_total), keys);
    }
  }

  // every warp meets here; the allocating warp returns the tensor memory
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, kUmmaTmemCols);
  }
}

// ------------------------------------------------------------------------------------------------
// Two row tiles per CTA (more than 128 stacked rows).  Both tiles (groups a and b, 128 rows each) share the CTA's
// K and V tiles, and their products alternate on the tensor pipe: while the weight warps of one group turn S into P,
// the pipe runs the other group's value product and next scores.  Per group S (64 columns) is overwritten in place
// by P (each thread writes P_hi and P_lo over the 32 score columns it has just read), so no buffer is ever waited
// for: the in-order pipe runs the scores of tile t+1 only after the value product of tile t has read P.
//   tensor memory (512 columns): S/P_a [0,64)  S/P_b [64,128)  O_a [128,256)  O_b [256,384)  Q_a [384,448)  Q_b [448,512)
constexpr int kPairThreads = (2 + 16) * 32;          // producer, MMA, 2 x 8 weight warps
constexpr int kPairRows = 2 * kUmmaRows;
constexpr int kPairStages = 6;

struct PairLayout {                                  // byte offsets from a 1 KB-aligned base
  static constexpr int kRing = 0;
  static constexpr int kStage = 32768;
  static constexpr int kBar = kRing + kPairStages * kStage;
  static constexpr int kLbuf = kBar + 256;                       // 2 x 128 floats: the second half-row's share of L
  static constexpr int kTotal = kLbuf + 1024 + 1024;
};

template <bool GATED>
__global__ void __launch_bounds__(kPairThreads, 1)
fold_scan_stacked_pair_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                              const ScanParams p) {
  constexpr int D = 128;
  using LO = PairLayout;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t *gen = smem_raw + (base - raw);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int row_pairs = (p.R + kPairRows - 1) / kPairRows;
  const int rp = blockIdx.x % row_pairs, split = blockIdx.x / row_pairs;
  const int kvh = blockIdx.y, seq = blockIdx.z;
  const SeqWork w = seq_work(p, seq);
  if (split >= w.n_chunks) return;
  const int R = p.R, n = w.n;
  const int dstart = draft_start(p, n);

  // barriers (8 bytes each): kv_full[stages]  xa[stages]  xb[stages]  s0[2]  p_full[2]  o_empty[2]
  // One commit per group and tile: x{a,b}[stage] completes when that group's value product of the tile in `stage` AND
  // its scores of the next tile have (the pipe runs in order), so it tells the group's weight warps both that S of the
  // next tile is ready and, at a chunk's end, that O is final.  xb (`pv_done` below) is committed after everything
  // issued for the tile and also frees the stage for the producer.  s0[g] (`s_full`): the very first scores.
  const uint32_t bar = base + LO::kBar;
  const uint32_t kv_full = bar, xa = bar + 8 * kPairStages, pv_done = bar + 16 * kPairStages, s_full = bar + 24 * kPairStages,
                 p_full = s_full + 16, o_empty = s_full + 32, tmem_slot = bar + 224;
  if (threadIdx.x == 0) {
    for (int s = 0; s < kPairStages; ++s) { mbar_init(kv_full + 8u * s, 1); mbar_init(xa + 8u * s, 1); mbar_init(pv_done + 8u * s, 1); }
    for (int g = 0; g < 2; ++g) {
      mbar_init(s_full + 8u * g, 1);
      mbar_init(p_full + 8u * g, 8);                         // one arrival per weight warp of the group
      mbar_init(o_empty + 8u * g, 8);
    }
    mbar_fence_init();
  }
  if (warp == 1) tmem_alloc(tmem_slot, 512);
  pdl_launch_dependents();
  pdl_wait();                                                // q and z come from earlier work
  tc_fence_before();
  __syncthreads();                                           // barriers initialised, TMEM allocated
  tc_fence_after();
  const uint32_t tmem = *reinterpret_cast<volatile uint32_t *>(gen + LO::kBar + 224);

  // weight warps 2..17: group g, key/channel half ch, TMEM lane quarter warp % 4
  const int wg = warp - 2;
  const int g = wg >> 3, ch = (wg >> 2) & 1;
  const int row = (warp & 3) * 32 + lane;                    // TMEM lane == query row of the group's tile
  const int r_glob = rp * kPairRows + g * kUmmaRows + row;
  const uint32_t lane_addr = tmem + ((uint32_t)((warp & 3) * 32) << 16);
  const uint32_t col_s = g * 64, col_o = 128 + g * 128, col_q = 384 + g * 64;
  float z_row = 0.f;
  uint32_t dm_row = 0xffffffffu;                             // the row's request's draft mask
  if (warp >= 2) {
    const bool valid_row = r_glob < R;
    const int req = seq * p.stack + r_glob / p.G, head = kvh * p.G + r_glob % p.G;
    const uint4 *qrow = reinterpret_cast<const uint4 *>(p.q + (long long)req * p.q_stride_b + (long long)head * p.q_stride_h);
#pragma unroll
    for (int c = 0; c < 2; ++c) {                            // 16 columns = 32 channels at a time
      uint32_t qw[16];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const uint4 v = valid_row ? qrow[ch * 8 + c * 4 + i] : make_uint4(0, 0, 0, 0);
        qw[4 * i] = v.x; qw[4 * i + 1] = v.y; qw[4 * i + 2] = v.z; qw[4 * i + 3] = v.w;
      }
      tmem_st16(lane_addr + col_q + ch * 32 + c * 16, qw);
    }
    tmem_st_wait();
    z_row = valid_row ? p.z[(long long)req * p.Hq + head] : INFINITY;
    if (p.draft_len && valid_row) dm_row = p.draft_mask[req];
  }
  tc_fence_before();
  __syncthreads();                                           // Q is in tensor memory
  tc_fence_after();

  bool dead = false;
  if (warp == 0) {
    // ------------------------------------------------------------ producer
    if (lane == 0) {
      ScanParams pp = p;
      pp.stages = kPairStages;
      produce_tiles<D, true, LO::kStage>(&tmK, &tmV, pp, w, split, kvh, seq, base + LO::kRing, kv_full, pv_done);
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (the warp walks in step, one lane issues)
    const bool leader = lane == 0;
    const uint32_t tm = __shfl_sync(0xffffffffu, tmem, 0);
    constexpr uint32_t idesc_qk = umma_idesc(64, 0), idesc_pv = umma_idesc(128, 1);
    const uint32_t ring_lo = umma_desc_lo(base + LO::kRing, 0);
    // S_g = Q_g K^T for the tile in `stage` (K tile [2 halves][64 keys][128 B]: K step kk = 32 bytes along the row)
    auto issue_qk = [&](int gg, int stage, bool first) {
      const uint32_t k_lo = ring_lo + ((uint32_t)(stage * LO::kStage) >> 4) + (1u << 16);
      if (leader) {
        umma_bf16_ta<false>(tm + gg * 64, tm + 384 + gg * 64, k_lo, umma_desc_hi(1024), idesc_qk);
#pragma unroll
        for (int kk = 1; kk < D / 16; ++kk)
          umma_bf16_ta<true>(tm + gg * 64, tm + 384 + gg * 64 + kk * 8,
                             k_lo + (((kk >> 2) * (kTileKeys * 128) + (kk & 3) * 32) >> 4), umma_desc_hi(1024), idesc_qk);
        if (first) tc_commit(s_full + 8u * gg);               // later scores are announced by the group's x barrier
      }
      __syncwarp();
    };
    // O_g += P_g V for the tile in `stage`; thread ch of a row holds keys ch*32.. : P_hi at its columns +0, P_lo at +16
    auto issue_pv = [&](int gg, int stage, bool accumulate) {
      const uint32_t v_lo = ring_lo + ((uint32_t)(stage * LO::kStage + 16384) >> 4) + ((8192u >> 4) << 16);
      if (leader) {
#pragma unroll
        for (int i = 0; i < 2 * (kTileKeys / 16); ++i) {
          const int term = i / (kTileKeys / 16), j = i % (kTileKeys / 16);       // keys 16 j ..: thread half j / 2
          const uint32_t a = tm + gg * 64 + (j >> 1) * 32 + term * 16 + (j & 1) * 8;
          if (i == 0) umma_bf16_ta(tm + 128 + gg * 128, a, v_lo, umma_desc_hi(1024), idesc_pv, accumulate);
          else umma_bf16_ta<true>(tm + 128 + gg * 128, a, v_lo + j * (2048 >> 4), umma_desc_hi(1024), idesc_pv);
        }
      }
      __syncwarp();
    };
    int it = 0, chunk_i = 0;
    TileCursor k = cursor_begin(w, split);
    if (cursor_valid(k, w) && mbar_wait(kv_full, 0u, dead)) {
      tc_fence_after();
      issue_qk(0, 0, true);
      issue_qk(1, 0, true);
    }
    bool first_of_chunk = true;
    while (cursor_valid(k, w) && !dead) {
      const int stage = it % kPairStages, nstage = (it + 1) % kPairStages;
      TileCursor kn = k;
      const bool chunk_ends = cursor_next(kn, w, p.num_splits);
      const bool more = cursor_valid(kn, w);
      if (more && !mbar_wait(kv_full + 8u * nstage, (uint32_t)(((it + 1) / kPairStages) & 1), dead)) break;
#pragma unroll
      for (int gg = 0; gg < 2; ++gg) {
        if (first_of_chunk && chunk_i > 0 && !mbar_wait(o_empty + 8u * gg, (uint32_t)((chunk_i - 1) & 1), dead)) break;
        if (!mbar_wait(p_full + 8u * gg, (uint32_t)(it & 1), dead)) break;
        tc_fence_after();
        issue_pv(gg, stage, !first_of_chunk);
        if (more) issue_qk(gg, nstage, false);
        if (leader) tc_commit((gg == 0 ? xa : pv_done) + 8u * stage);
        __syncwarp();
      }
      if (chunk_ends) ++chunk_i;
      first_of_chunk = chunk_ends;
      k = kn;
      ++it;
    }
    if (dead && leader) atomicOr(&p.hdr->wait_timeouts, 8u);
  } else {
    // ------------------------------------------------------------ weight warps: two threads per query row
    const bool valid_row = r_glob < R;
    float l_row = 0.f;
    int it = 0;
    for (TileCursor k = cursor_begin(w, split); cursor_valid(k, w); ++it) {
      const int stage = it % kPairStages;
      const int key_base = k.t * kTileKeys;
      // the tcgen05 loads and stores below are warp-wide: the warp takes them together or not at all
      const uint32_t xg = g == 0 ? xa : pv_done;             // this group's per-stage barrier
      const bool have_s = it == 0 ? mbar_wait(s_full + 8u * g, 0u, dead)
                                  : mbar_wait(xg + 8u * ((it - 1) % kPairStages), (uint32_t)(((it - 1) / kPairStages) & 1), dead);
      if (__all_sync(0xffffffffu, have_s)) {
        tc_fence_after();
        float s[32];
        uint32_t ph[16], pl[16];                             // this thread's 32 weights, BF16 pairs: hi and lo terms
        tmem_ld32(lane_addr + col_s + ch * 32, s);
        // rows beyond R carry z = +inf, so their weights vanish by themselves; keys beyond n only occur in a tail tile
        const int key_lim = n - (key_base + ch * 32);        // this thread's keys j < key_lim exist
        if (key_base + kTileKeys > dstart) {                 // draft keys: the row only uses the ones its mask names
#pragma unroll
          for (int j = 0; j < 32; ++j)
            if (!draft_ok(dm_row, key_base + ch * 32 + j, dstart)) s[j] = -INFINITY;
        }
        auto weights = [&](auto tail) {
#pragma unroll
          for (int j = 0; j < 32; j += 2) {
            float pw[2], pm[2];
#pragma unroll
            for (int e = 0; e < 2; ++e) {
              float x = fmaf(s[j + e], p.scale_log2, -z_row);
              if (decltype(tail)::value) x = (j + e) < key_lim ? x : -INFINITY;
              pw[e] = ex2_approx(x);
              pm[e] = (!GATED || x >= p.neg_T) ? pw[e] : 0.f;
            }
            const uint32_t hi2 = pack_bf16(pm[0], pm[1]);
            const float h0 = __uint_as_float(hi2 << 16), h1 = __uint_as_float(hi2 & 0xffff0000u);
            const uint32_t lo2 = pack_bf16(pm[0] - h0, pm[1] - h1);
            const float g0 = __uint_as_float(lo2 << 16), g1 = __uint_as_float(lo2 & 0xffff0000u);
            l_row += ((h0 + g0) + (pw[0] - pm[0])) + ((h1 + g1) + (pw[1] - pm[1]));
            ph[j / 2] = hi2;
            pl[j / 2] = lo2;
          }
        };
        if (key_lim >= 32) weights(std::false_type{}); else weights(std::true_type{});
        // P over the scores this thread has just read: P_hi in the first 16 of its 32 columns, P_lo in the rest
        tmem_st16(lane_addr + col_s + ch * 32, ph);
        tmem_st16(lane_addr + col_s + ch * 32 + 16, pl);
        tmem_st_wait();
        if (g == 0 && key_base + kTileKeys > n) {            // ragged tail: value rows past n may hold anything
          const int tw = threadIdx.x - 64;                   // group a's 256 threads clear them for both groups
          for (int i = tw; i < kTileKeys * 16; i += 256) {
            const int vr_ = i >> 4, c16 = i & 15;
            if (key_base + vr_ >= n)
              *reinterpret_cast<uint4 *>(gen + LO::kRing + stage * LO::kStage + 16384 + tile_off(vr_, c16, kTileKeys)) =
                  make_uint4(0, 0, 0, 0);
          }
          fence_proxy_async_smem();                          // generic writes, then tensor-core (async proxy) reads
        }
        tc_fence_before();
      }
      __syncwarp();                                          // every lane's stores and fences are done
      if (lane == 0) mbar_arrive(p_full + 8u * g);
      const int c_done = k.c;
      if (cursor_next(k, w, p.num_splits)) {
        // chunk end: this thread's half of its row of O, and the row's L, go to the chunk's slot
        float *slot = p.slots + (((long long)seq * p.Hkv + kvh) * p.max_slots + c_done) * p.slot_stride;
        float *lbuf = reinterpret_cast<float *>(gen + LO::kLbuf) + g * kUmmaRows;
        if (ch == 1) lbuf[row] = l_row;
        if (__all_sync(0xffffffffu, mbar_wait(xg + 8u * stage, (uint32_t)((it / kPairStages) & 1), dead))) {
          tc_fence_after();
#pragma unroll 1
          for (int q4 = ch * 2; q4 < ch * 2 + 2; ++q4) {
            float o[32];
            tmem_ld32(lane_addr + col_o + q4 * 32, o);
            if (valid_row) {
              float4 *dst = reinterpret_cast<float4 *>(slot + (long long)r_glob * D + q4 * 32);
#pragma unroll
              for (int i = 0; i < 8; ++i) dst[i] = make_float4(o[4 * i], o[4 * i + 1], o[4 * i + 2], o[4 * i + 3]);
            }
          }
          tc_fence_before();
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(o_empty + 8u * g);
        named_bar(1 + g, 256);                               // both halves of every row of the group are in
        if (ch == 0 && valid_row) slot[(long long)R * D + r_glob] = l_row + lbuf[row];
        named_bar(1 + g, 256);                               // lbuf may be rewritten
        l_row = 0.f;
      }
    }
    if (dead && lane == 0) atomicOr(&p.hdr->wait_timeouts, 16u);
    if (threadIdx.x == 64 && rp == 0) {                      // every value row is read once per row-pair pass
      unsigned long long keys = 0;
      for (int c = split; c < w.n_chunks; c += p.num_splits)
        keys += min((c + 1) * w.ctiles * kTileKeys, n) - c * w.ctiles * kTileKeys;
      atomicAdd(reinterpret_cast<unsigned long long *>(&p.hdr->v_rows_fetched), keys);
      atomicAdd(reinterpret_cast<unsigned long long *>(&p.hdr->v_rows_total), keys);
    }
  }

  // every warp meets here; the allocating warp returns the tensor memory
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
}

}  // namespace fold
