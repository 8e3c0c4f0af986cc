// Stacked-row scan on the 5th-generation tensor cores (tcgen05 + TMEM), head_dim 128.
//
// The shared-prefix level of a cascade stacks the query rows of every request that holds the
// prefix (Section 4, "Value product"; Appendix "Tile layouts"): with hundreds of rows per
// (sequence, kv head) the scan is a dense contraction, not a stream, so it runs on tcgen05.mma
// with the accumulators in tensor memory.  One CTA owns 128 query rows (M = 128) of one
// (sequence, kv head) and walks the 64-key tiles of its canonical chunks:
//
//   producer warp   TMA: K and V tiles -> 3-stage shared-memory ring (same tiles as dense decode)
//   MMA warp        S = Q K^T        (A = Q in smem, K-major;  B = K tile, K-major;  N = 64 keys)
//                   O += P_hi V + P_lo V   (A = P in smem, K-major;  B = V tile, MN-major;  N = 128)
//   8 weight warps  two threads per query row (the row's TMEM lane; each takes 32 of the tile's 64 keys and
//                   64 of the 128 channels): tcgen05.ld S, final weights 2^(s - Z) with the depth gate,
//                   L in a register, two-term BF16 P -> smem
//
// S is double-buffered in TMEM and P in shared memory, so the scores of tile t+1 are computed
// while the weights of tile t are formed.  No maximum is tracked and nothing is rescaled: the
// accumulator O is only ever added to.  At a chunk's end each thread reads its row of O from
// TMEM and writes it, with its L, to the chunk's slot.
#pragma once

#include "fold_scan.cuh"

namespace fold {

constexpr int kUmmaThreads = 10 * 32;                // producer, MMA, 8 weight warps
constexpr int kUmmaWeightThreads = 8 * 32;
constexpr int kUmmaRows = 128;                       // query rows per CTA (MMA M)
constexpr int kUmmaStages = 3;
constexpr int kUmmaTmemCols = 256;                   // S0 [0,64)  S1 [64,128)  O [128,256)

struct UmmaLayout {                                  // byte offsets from a 1 KB-aligned base
  static constexpr int kQ = 0;                                   // [2 halves][128 rows][128 B], swizzled
  static constexpr int kRing = 32768;                            // stages x (K tile 16 KB + V tile 16 KB)
  static constexpr int kStage = 32768;
  static constexpr int kP = kRing + kUmmaStages * kStage;        // 2 buffers x (hi 16 KB + lo 16 KB)
  static constexpr int kBar = kP + 2 * 32768;
  static constexpr int kLbuf = kBar + 256;                       // 128 floats: the second half-row's share of L
  static constexpr int kTotal = kLbuf + 512 + 1024;              // + alignment slack
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
// D[tmem] (+)= A[smem] * B[smem], BF16 inputs, FP32 accumulate; issued by one thread.
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(0u)
      : "memory");
}
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

// Shared-memory matrix descriptor (128-byte swizzle, descriptor version 1).  Offsets in bytes.
__device__ __forceinline__ uint64_t umma_desc(uint32_t smem_addr, uint32_t lbo, uint32_t sbo) {
  return (uint64_t)((smem_addr >> 4) & 0x3fffu) | ((uint64_t)((lbo >> 4) & 0x3fffu) << 16) |
         ((uint64_t)((sbo >> 4) & 0x3fffu) << 32) | (1ull << 46) | (2ull << 61);
}
// Instruction descriptor: FP32 accumulate, BF16 A and B, M = 128.
__host__ __device__ constexpr uint32_t umma_idesc(int n, int b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)b_mn_major << 16) | ((uint32_t)(n >> 3) << 17) |
         ((uint32_t)(kUmmaRows >> 4) << 24);
}

template <bool GATED>
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

  // barriers (8 bytes each): kv_full[3] kv_empty[3] s_full[2] s_empty[2] p_full[2] p_empty[2] o_full o_empty
  const uint32_t bar = base + LO::kBar;
  const uint32_t kv_full = bar, kv_empty = bar + 24, s_full = bar + 48, s_empty = bar + 64, p_full = bar + 80,
                 p_empty = bar + 96, o_full = bar + 112, o_empty = bar + 120, tmem_slot = bar + 128;
  if (threadIdx.x == 0) {
    for (int s = 0; s < kUmmaStages; ++s) { mbar_init(kv_full + 8u * s, 1); mbar_init(kv_empty + 8u * s, 1); }
    for (int b = 0; b < 2; ++b) {
      mbar_init(s_full + 8u * b, 1);
      mbar_init(s_empty + 8u * b, kUmmaWeightThreads);
      mbar_init(p_full + 8u * b, kUmmaWeightThreads);
      mbar_init(p_empty + 8u * b, 1);
    }
    mbar_init(o_full, 1);
    mbar_init(o_empty, kUmmaWeightThreads);
    mbar_fence_init();
  }
  if (warp == 1) tmem_alloc(tmem_slot, kUmmaTmemCols);
  pdl_launch_dependents();
  pdl_wait();                                                // q and z come from earlier work

  // the weight warps stage their query rows: row r of the tile -> [half][r][128 B], 128-byte swizzle
  const int row = (warp & 3) * 32 + lane;                    // TMEM lane == query row of the tile
  const int ch = warp >= 6 ? 1 : 0;                          // which half of the tile's keys / of the channels
  const int r_glob = rt * kUmmaRows + row;
  float z_row = 0.f;
  if (warp >= 2) {
    const bool valid_row = r_glob < R;
    const int req = seq * p.stack + r_glob / p.G, head = kvh * p.G + r_glob % p.G;
    const uint4 *qrow = reinterpret_cast<const uint4 *>(p.q + (long long)req * p.q_stride_b + (long long)head * p.q_stride_h);
#pragma unroll
    for (int c = ch * 8; c < ch * 8 + 8; ++c) {
      const uint4 v = valid_row ? qrow[c] : make_uint4(0, 0, 0, 0);
      *reinterpret_cast<uint4 *>(gen + LO::kQ + tile_off(row, c, kUmmaRows)) = v;
    }
    if (valid_row) z_row = p.z[(long long)req * p.Hq + head];
    fence_proxy_async_smem();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *reinterpret_cast<volatile uint32_t *>(gen + LO::kBar + 128);

  bool dead = false;
  if (warp == 0) {
    // ------------------------------------------------------------ producer
    if (lane == 0) {
      ScanParams pp = p;
      pp.stages = kUmmaStages;
      produce_tiles<D, true, LO::kStage>(&tmK, &tmV, pp, w, split, kvh, seq, base + LO::kRing, kv_full, kv_empty);
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc_qk = umma_idesc(64, 0), idesc_pv = umma_idesc(128, 1);
      const uint32_t q_s = base + LO::kQ;
      auto issue_qk = [&](int it, int stage) {               // S[it & 1] = Q K^T for the tile in `stage`
        const int b = it & 1;
        if (!mbar_wait(kv_full + 8u * stage, (uint32_t)((it / kUmmaStages) & 1), dead)) return;
        if (it >= 2 && !mbar_wait(s_empty + 8u * b, (uint32_t)(((it >> 1) - 1) & 1), dead)) return;
        tc_fence_after();
        const uint32_t k_s = base + LO::kRing + stage * LO::kStage;
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          const uint32_t off = (kk >> 2), sub = (kk & 3) * 32;
          umma_bf16(tmem + b * 64, umma_desc(q_s + off * (kUmmaRows * 128) + sub, 16, 1024),
                    umma_desc(k_s + off * (kTileKeys * 128) + sub, 16, 1024), idesc_qk, kk > 0 ? 1u : 0u);
        }
        tc_commit(s_full + 8u * b);
      };
      int it = 0, chunk_i = 0;
      TileCursor k = cursor_begin(w, split);
      if (cursor_valid(k, w)) issue_qk(0, 0);
      bool first_of_chunk = true;
      while (cursor_valid(k, w) && !dead) {
        const int stage = it % kUmmaStages, b = it & 1;
        TileCursor kn = k;
        const bool chunk_ends = cursor_next(kn, w, p.num_splits);
        if (cursor_valid(kn, w)) issue_qk(it + 1, (it + 1) % kUmmaStages);
        // O += P V for tile `it`
        if (first_of_chunk && chunk_i > 0 && !mbar_wait(o_empty, (uint32_t)((chunk_i - 1) & 1), dead)) break;
        if (!mbar_wait(p_full + 8u * b, (uint32_t)((it >> 1) & 1), dead)) break;
        tc_fence_after();
        const uint32_t v_s = base + LO::kRing + stage * LO::kStage + 16384;
        const uint32_t p_s = base + LO::kP + b * 32768;
#pragma unroll
        for (int term = 0; term < 2; ++term)
#pragma unroll
          for (int j = 0; j < kTileKeys / 16; ++j)
            umma_bf16(tmem + 128, umma_desc(p_s + term * 16384 + j * 32, 16, 1024),
                      umma_desc(v_s + j * 2048, 8192, 1024), idesc_pv, (first_of_chunk && term == 0 && j == 0) ? 0u : 1u);
        tc_commit(p_empty + 8u * b);
        tc_commit(kv_empty + 8u * stage);
        if (chunk_ends) { tc_commit(o_full); ++chunk_i; }
        first_of_chunk = chunk_ends;
        k = kn;
        ++it;
      }
      if (dead) atomicOr(&p.hdr->wait_timeouts, 8u);
    }
  } else {
    // ------------------------------------------------------------ weight warps: one query row per thread
    const bool valid_row = r_glob < R;
    const uint32_t lane_addr = tmem + ((uint32_t)((warp & 3) * 32) << 16);
    float l_row = 0.f;
    int it = 0, chunk_i = 0;
    for (TileCursor k = cursor_begin(w, split); cursor_valid(k, w); ++it) {
      const int b = it & 1, stage = it % kUmmaStages;
      const int key_base = k.t * kTileKeys;
      uint32_t ph[16], pl[16];                               // this thread's 32 weights, BF16 pairs: hi and lo terms
      const bool have_s = mbar_wait(s_full + 8u * b, (uint32_t)((it >> 1) & 1), dead);
      if (have_s) {
        tc_fence_after();
        float s[32];
        tmem_ld32(lane_addr + b * 64 + ch * 32, s);
#pragma unroll
        for (int j = 0; j < 32; j += 2) {
          float pw[2], pm[2];
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            const bool ok = valid_row && (key_base + ch * 32 + j + e) < n;
            const float x = ok ? fmaf(s[j + e], p.scale_log2, -z_row) : -INFINITY;
            const bool live = GATED ? (x >= p.neg_T) : ok;
            pw[e] = ex2_approx(x);
            pm[e] = live ? pw[e] : 0.f;
          }
          const uint32_t hi2 = pack_bf16(pm[0], pm[1]);
          const float h0 = __uint_as_float(hi2 << 16), h1 = __uint_as_float(hi2 & 0xffff0000u);
          const uint32_t lo2 = pack_bf16(pm[0] - h0, pm[1] - h1);
          const float g0 = __uint_as_float(lo2 << 16), g1 = __uint_as_float(lo2 & 0xffff0000u);
          l_row += ((h0 + g0) + (pw[0] - pm[0])) + ((h1 + g1) + (pw[1] - pm[1]));
          ph[j / 2] = hi2;
          pl[j / 2] = lo2;
        }
        tc_fence_before();
      }
      mbar_arrive(s_empty + 8u * b);                         // S[b] may be overwritten
      if (it < 2 || mbar_wait(p_empty + 8u * b, (uint32_t)(((it >> 1) - 1) & 1), dead)) {
        uint8_t *p_hi = gen + LO::kP + b * 32768, *p_lo = p_hi + 16384;
#pragma unroll
        for (int c = 0; c < 4; ++c) {                        // 8 keys = one 16-byte chunk, swizzled by the row
          const uint32_t off = row * 128 + (((ch * 4 + c) ^ (row & 7)) << 4);
          *reinterpret_cast<uint4 *>(p_hi + off) = make_uint4(ph[4 * c], ph[4 * c + 1], ph[4 * c + 2], ph[4 * c + 3]);
          *reinterpret_cast<uint4 *>(p_lo + off) = make_uint4(pl[4 * c], pl[4 * c + 1], pl[4 * c + 2], pl[4 * c + 3]);
        }
        if (key_base + kTileKeys > n) {                      // ragged tail: value rows past n may hold anything
          const int tw = threadIdx.x - 64;
          for (int i = tw; i < kTileKeys * 16; i += kUmmaWeightThreads) {
            const int vr_ = i >> 4, c16 = i & 15;
            if (key_base + vr_ >= n)
              *reinterpret_cast<uint4 *>(gen + LO::kRing + stage * LO::kStage + 16384 + tile_off(vr_, c16, kTileKeys)) =
                  make_uint4(0, 0, 0, 0);
          }
        }
        fence_proxy_async_smem();                            // generic writes, then tensor-core (async proxy) reads
      }
      mbar_arrive(p_full + 8u * b);
      const int c_done = k.c;
      if (cursor_next(k, w, p.num_splits)) {
        // chunk end: this thread's half of its row of O, and the row's L, go to the chunk's slot
        float *slot = p.slots + (((long long)seq * p.Hkv + kvh) * p.max_slots + c_done) * p.slot_stride;
        float *lbuf = reinterpret_cast<float *>(gen + LO::kLbuf);
        if (ch == 1) lbuf[row] = l_row;
        if (mbar_wait(o_full, (uint32_t)(chunk_i & 1), dead)) {
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
        mbar_arrive(o_empty);
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

}  // namespace fold
