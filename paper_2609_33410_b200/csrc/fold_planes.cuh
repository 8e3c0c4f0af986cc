// Two-plane INT8 keys (Section 4, "Cache format" and "Weight-gated reads"; Algorithm 1).
//
//   cache write   fold_quantize_keys_kernel: rotate a BF16 key row by the orthonormal Hadamard matrix, split
//                 it into two INT8 planes and a BF16 scale rounded up:  H k = e (a + b / 256)
//   front         fold_planes_front_kernel: split every query row the same way (into the workspace) and
//                 form the 192-key reference estimate on two-plane scores
//   scan          fold_scan_planes_kernel: every key is scored against plane A alone (INT8 products, keys
//                 on M, the group's rows on N); the verdict bits live / refine are ORed over the group, and
//                 only then are plane B rows (refined keys) and value rows (live keys) requested; a second
//                 INT8 product adds plane B; final FP32 weights feed the BF16 value product.
#pragma once

#include <cuda_fp8.h>
#include <cuda_fp16.h>

#include "fold_common.cuh"
#include "fold_estimate.cuh"
#include "fold_scan.cuh"

namespace fold {

// The key planes as the kernels see them.
struct PlaneView {
  const int8_t *a, *b;
  long long stride_seq, stride_tok, stride_head;              // bytes
  const __nv_bfloat16 *scale;
  long long sc_stride_seq, sc_stride_head;                    // elements; tokens are contiguous
  const int *page_table;
  const int *seqlens;
  int paged, page_shift, max_pages, num_pages, max_seqlen;
  const uint8_t *v1, *v2;                                     // E4M3 value planes (strides as a / b), or null
  float v_scale;                                              // 2^v_scale_log2
};

// (sequence-or-page, token-in-it) of logical token j
__device__ __forceinline__ void plane_locate(const PlaneView &kv, int seq, int j, long long &s, long long &t) {
  s = seq; t = j;
  if (kv.paged) {
    int pg = kv.page_table[(long long)seq * kv.max_pages + (j >> kv.page_shift)];
    s = min(max(pg, 0), kv.num_pages - 1);
    t = j & ((1 << kv.page_shift) - 1);
  }
}

// ------------------------------------------------------------------------------------------------
// Rotation and split of one row held by a warp: lane l has channels l * D/32 .. + D/32 - 1 in x[].
// FP32, one rounding per step, in this order (the codes are integers decided by this arithmetic, so the order
// is part of the format): butterfly stages with strides 1, 2, 4, ..., D/2, each (lo, hi) -> (lo + hi, lo - hi);
// one multiply by fp32(1 / sqrt(D)); e = the smallest BF16 >= max|y| / 127 (1 for an all-zero row);
// t = y / e; a = rint(t) within +-127; b = rint((t - a) * 256) within [-128, 127].  Returns e.
template <int D>
__device__ __forceinline__ float rotate_split(float (&x)[D / 32], int lane, int (&a)[D / 32], int (&b)[D / 32]) {
  constexpr int EPL = D / 32;
#pragma unroll
  for (int h = 1; h < EPL; h <<= 1)
#pragma unroll
    for (int i = 0; i < EPL; ++i)
      if (!(i & h)) {
        const float lo = x[i], hi = x[i + h];
        x[i] = __fadd_rn(lo, hi);
        x[i + h] = __fsub_rn(lo, hi);
      }
#pragma unroll
  for (int m = 1; m < 32; m <<= 1)
#pragma unroll
    for (int i = 0; i < EPL; ++i) {
      const float other = __shfl_xor_sync(0xffffffffu, x[i], m);
      x[i] = (lane & m) ? __fsub_rn(other, x[i]) : __fadd_rn(x[i], other);
    }
  const float r_sqrt_d = D == 64 ? 0.125f : __uint_as_float(0x3db504f3u);      // fp32(1 / sqrt(D))
  float mx = 0.f;
#pragma unroll
  for (int i = 0; i < EPL; ++i) {
    x[i] = __fmul_rn(x[i], r_sqrt_d);
    mx = fmaxf(mx, fabsf(x[i]));
  }
#pragma unroll
  for (int m = 16; m > 0; m >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, m));
  float e = 1.f;
  if (mx > 0.f) {
    const uint32_t u = __float_as_uint(__fdiv_rn(mx, 127.f));
    e = __uint_as_float((u & 0xffffu) ? ((u >> 16) + 1u) << 16 : u);
    if (!(e > 0.f)) e = 1.f;
  }
#pragma unroll
  for (int i = 0; i < EPL; ++i) {
    const float t = __fdiv_rn(x[i], e);
    const float af = fminf(fmaxf(rintf(t), -127.f), 127.f);
    const float bf = fminf(fmaxf(rintf(__fmul_rn(__fsub_rn(t, af), 256.f)), -128.f), 127.f);
    a[i] = (int)af;
    b[i] = (int)bf;
  }
  return e;
}

template <int EPL>
__device__ __forceinline__ void load_bf16_row(const __nv_bfloat16 *row, float (&x)[EPL]) {
  if (EPL == 4) {
    const uint2 w = *reinterpret_cast<const uint2 *>(row);
    x[0] = __uint_as_float(w.x << 16); x[1] = __uint_as_float(w.x & 0xffff0000u);
    x[EPL - 2] = __uint_as_float(w.y << 16); x[EPL - 1] = __uint_as_float(w.y & 0xffff0000u);
  } else {
    const uint32_t w = *reinterpret_cast<const uint32_t *>(row);
    x[0] = __uint_as_float(w << 16); x[1] = __uint_as_float(w & 0xffff0000u);
  }
}
template <int EPL>
__device__ __forceinline__ void store_codes(int8_t *dst, const int (&c)[EPL]) {       // EPL consecutive bytes
  if (EPL == 4) {
    *reinterpret_cast<uint32_t *>(dst) = (uint32_t)(c[0] & 0xff) | ((uint32_t)(c[1] & 0xff) << 8) |
                                         ((uint32_t)(c[EPL - 2] & 0xff) << 16) | ((uint32_t)(c[EPL - 1] & 0xff) << 24);
  } else {
    *reinterpret_cast<uint16_t *>(dst) = (uint16_t)((c[0] & 0xff) | ((c[1] & 0xff) << 8));
  }
}

// ------------------------------------------------------------------------------------------------
// Cache write: one warp per (sequence, token, kv head) row.
struct QuantParams {
  const __nv_bfloat16 *k;
  long long k_stride_seq, k_stride_tok, k_stride_head;
  PlaneView kv;                                               // destinations (written)
  const int *first_token;                                     // per sequence, or null: from token 0
};
constexpr int kQuantWarps = 8;                                  // warps per CTA
constexpr int kQuantRowsPerWarp = 4;                            // rows a warp loads before it works on any (bytes in flight)
constexpr int kQuantRowsPerCta = kQuantWarps * kQuantRowsPerWarp;

template <int D>
__global__ void __launch_bounds__(32 * kQuantWarps) fold_quantize_keys_kernel(const QuantParams p) {
  constexpr int EPL = D / 32, RW = kQuantRowsPerWarp;
  const int lane = threadIdx.x, kvh = blockIdx.y, seq = blockIdx.z;
  int n = p.kv.seqlens[seq];
  n = n < 0 ? 0 : (n > p.kv.max_seqlen ? p.kv.max_seqlen : n);
  const int first = p.first_token ? max(p.first_token[seq], 0) : 0;
  const int j0 = first + (blockIdx.x * kQuantWarps + threadIdx.y) * RW;
  if (j0 >= n) return;
  long long s[RW], t[RW];
  float x[RW][EPL];
#pragma unroll
  for (int r = 0; r < RW; ++r) {
    s[r] = t[r] = 0;
    if (j0 + r < n) {
      plane_locate(p.kv, seq, j0 + r, s[r], t[r]);
      load_bf16_row<EPL>(p.k + s[r] * p.k_stride_seq + t[r] * p.k_stride_tok + (long long)kvh * p.k_stride_head + lane * EPL, x[r]);
    }
  }
#pragma unroll
  for (int r = 0; r < RW; ++r) {
    if (j0 + r >= n) break;
    int a[EPL], b[EPL];
    const float e = rotate_split<D>(x[r], lane, a, b);
    const long long off = s[r] * p.kv.stride_seq + t[r] * p.kv.stride_tok + (long long)kvh * p.kv.stride_head + lane * EPL;
    store_codes<EPL>(const_cast<int8_t *>(p.kv.a) + off, a);
    store_codes<EPL>(const_cast<int8_t *>(p.kv.b) + off, b);
    if (lane == 0)
      const_cast<__nv_bfloat16 *>(p.kv.scale)[s[r] * p.kv.sc_stride_seq + (long long)kvh * p.kv.sc_stride_head + t[r]] =
          __float2bfloat16_rn(e);                            // exact: e is a BF16 value
  }
}

// Cache write of the E4M3 value planes: p1 = e4m3(v / scale), p2 = e4m3(v / scale - p1), a warp per four rows.
struct QuantValueParams {
  const __nv_bfloat16 *v;
  long long v_stride_seq, v_stride_tok, v_stride_head;
  PlaneView kv;                                               // destinations v1 / v2 (written)
  const int *first_token;
  float inv_scale;                                            // 2^-v_scale_log2
};
template <int D>
__global__ void __launch_bounds__(32 * kQuantWarps) fold_quantize_values_kernel(const QuantValueParams p) {
  constexpr int EPL = D / 32, RW = kQuantRowsPerWarp;
  const int lane = threadIdx.x, kvh = blockIdx.y, seq = blockIdx.z;
  int n = p.kv.seqlens[seq];
  n = n < 0 ? 0 : (n > p.kv.max_seqlen ? p.kv.max_seqlen : n);
  const int first = p.first_token ? max(p.first_token[seq], 0) : 0;
  const int j0 = first + (blockIdx.x * kQuantWarps + threadIdx.y) * RW;
  if (j0 >= n) return;
  long long s[RW], t[RW];
  float x[RW][EPL];
#pragma unroll
  for (int r = 0; r < RW; ++r) {
    s[r] = t[r] = 0;
    if (j0 + r < n) {
      plane_locate(p.kv, seq, j0 + r, s[r], t[r]);
      load_bf16_row<EPL>(p.v + s[r] * p.v_stride_seq + t[r] * p.v_stride_tok + (long long)kvh * p.v_stride_head + lane * EPL, x[r]);
    }
  }
#pragma unroll
  for (int r = 0; r < RW; ++r) {
    if (j0 + r >= n) break;
    int c1[EPL], c2[EPL];
#pragma unroll
    for (int i = 0; i < EPL; ++i) {
      const float y = __fmul_rn(x[r][i], p.inv_scale);        // exact: a power of two
      const __nv_fp8_storage_t a = __nv_cvt_float_to_fp8(y, __NV_SATFINITE, __NV_E4M3);
      const float ya = __half2float(__half(__nv_cvt_fp8_to_halfraw(a, __NV_E4M3)));
      const __nv_fp8_storage_t b = __nv_cvt_float_to_fp8(__fsub_rn(y, ya), __NV_SATFINITE, __NV_E4M3);   // exact difference
      c1[i] = (int)a;
      c2[i] = (int)b;
    }
    const long long off = s[r] * p.kv.stride_seq + t[r] * p.kv.stride_tok + (long long)kvh * p.kv.stride_head + lane * EPL;
    store_codes<EPL>(reinterpret_cast<int8_t *>(const_cast<uint8_t *>(p.kv.v1)) + off, c1);
    store_codes<EPL>(reinterpret_cast<int8_t *>(const_cast<uint8_t *>(p.kv.v2)) + off, c2);
  }
}

// ------------------------------------------------------------------------------------------------
// Front kernel: one CTA per (kv head, request).  Splits the group's query rows (rows of the workspace:
// [request * Hq + head][2][D] codes and one eta = e_q * scale_log2 per row), then, if the reference is to be
// estimated, thread i scores sampled key i with both planes (exact integer dot products) and warp g
// reduces row g.  A cascade's levels are one logical sequence, level after level: the samples are taken over the
// concatenation, and every level's workspace gets the split rows (and a cleared header).
struct FrontLevel {
  PlaneView kv;
  int stack;                                                   // requests per sequence of this level
  int8_t *qplanes;
  float *qeta;
  fold_ws_header *hdr;                                         // not null: also zero this level's workspace header
};
struct FrontParams {
  const __nv_bfloat16 *q;
  long long q_stride_b, q_stride_h;
  float *z;
  FrontLevel lv[kMaxLevels];
  int n_levels;
  int write_z, Hq, Hkv, G;
  float scale_log2;
  const uint32_t *draft_mask;                                  // drafts: the last draft_len keys are used by request req only
  int draft_len;                                               // where its mask has the bit
};
constexpr int kFrontThreads = kEstSamples;                    // 192

template <int D>
__global__ void __launch_bounds__(kFrontThreads) fold_planes_front_kernel(const FrontParams p) {
  constexpr int EPL = D / 32, W = D / 4;                      // W: 32-bit words per plane row
  __shared__ uint32_t sq[kMaxRows][2][W];
  __shared__ float seta[kMaxRows];
  __shared__ float sc[kMaxRows][kEstSamples];
  const int kvh = blockIdx.x, req = blockIdx.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int G = p.G;
  pdl_launch_dependents();

  // Everything up to the dependency wait below reads only the caller's inputs and writes shared memory: launched
  // early behind the partial add of a call before this one, it overlaps it.
  for (int g = warp; g < G; g += kFrontThreads / 32) {
    const int head = kvh * G + g;
    float x[EPL];
    load_bf16_row<EPL>(p.q + (long long)req * p.q_stride_b + (long long)head * p.q_stride_h + lane * EPL, x);
    int a[EPL], b[EPL];
    const float e = rotate_split<D>(x, lane, a, b);
    store_codes<EPL>(reinterpret_cast<int8_t *>(&sq[g][0][0]) + lane * EPL, a);
    store_codes<EPL>(reinterpret_cast<int8_t *>(&sq[g][1][0]) + lane * EPL, b);
    if (lane == 0) seta[g] = __fmul_rn(e, p.scale_log2);
  }
  __syncthreads();
  // the workspace (split rows, header) may still be read by the scan of a call before this one, z by its partial add
  auto publish = [&]() {
    pdl_wait();
#pragma unroll
    for (int l = 0; l < kMaxLevels; ++l) {                     // (constant indices: the parameter block stays where it is)
      if (l >= p.n_levels) break;
      const FrontLevel &lv = p.lv[l];
      if (lv.hdr && blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x < 16) reinterpret_cast<uint32_t *>(lv.hdr)[threadIdx.x] = 0u;
      for (int i = threadIdx.x; i < G * 2 * W; i += kFrontThreads) {          // rows kvh * G .. + G - 1 are contiguous
        const int g = i / (2 * W), w = i % (2 * W);
        reinterpret_cast<uint32_t *>(lv.qplanes + ((long long)req * p.Hq + kvh * G + g) * (2 * D))[w] = sq[g][w / W][w % W];
      }
      if (threadIdx.x < G) lv.qeta[(long long)req * p.Hq + kvh * G + threadIdx.x] = seta[threadIdx.x];
    }
  };
  if (!p.write_z) { publish(); return; }

  // the request's keys: its sequence of every level, one after the other
  int nl[kMaxLevels], n = 0;
#pragma unroll
  for (int l = 0; l < kMaxLevels; ++l) {
    nl[l] = 0;
    if (l < p.n_levels) {
      const int v = p.lv[l].kv.seqlens[req / p.lv[l].stack];
      nl[l] = v < 0 ? 0 : (v > p.lv[l].kv.max_seqlen ? p.lv[l].kv.max_seqlen : v);
    }
    n += nl[l];
  }
  const int n_samples = n < kEstSamples ? n : kEstSamples;
  const int i = threadIdx.x;
  if (i < n_samples) {
    int j = est_sample_key(i, n);
    float e = 0.f;
    uint32_t ka[W], kb[W];
    bool found = false;
#pragma unroll
    for (int l = 0; l < kMaxLevels; ++l) {
      if (l >= p.n_levels || found) continue;
      if (j >= nl[l]) { j -= nl[l]; continue; }
      found = true;
      const PlaneView &kv = p.lv[l].kv;
      long long s, t;
      plane_locate(kv, req / p.lv[l].stack, j, s, t);
      const long long off = s * kv.stride_seq + t * kv.stride_tok + (long long)kvh * kv.stride_head;
      e = __bfloat162float(kv.scale[s * kv.sc_stride_seq + (long long)kvh * kv.sc_stride_head + t]);
#pragma unroll
      for (int w4 = 0; w4 < W / 4; ++w4) {
        const uint4 va = *reinterpret_cast<const uint4 *>(kv.a + off + w4 * 16);
        const uint4 vb = *reinterpret_cast<const uint4 *>(kv.b + off + w4 * 16);
        ka[4 * w4] = va.x; ka[4 * w4 + 1] = va.y; ka[4 * w4 + 2] = va.z; ka[4 * w4 + 3] = va.w;
        kb[4 * w4] = vb.x; kb[4 * w4 + 1] = vb.y; kb[4 * w4 + 2] = vb.z; kb[4 * w4 + 3] = vb.w;
      }
    }
    if (!found) {                                              // (cannot happen: the sample index is below n)
#pragma unroll
      for (int w = 0; w < W; ++w) ka[w] = kb[w] = 0u;
    }
    for (int g = 0; g < G; ++g) {
      int caa = 0, cab = 0, cba = 0, cbb = 0;
#pragma unroll
      for (int w = 0; w < W; ++w) {
        const int qa = (int)sq[g][0][w], qb = (int)sq[g][1][w];
        caa = __dp4a((int)ka[w], qa, caa); cab = __dp4a((int)ka[w], qb, cab);
        cba = __dp4a((int)kb[w], qa, cba); cbb = __dp4a((int)kb[w], qb, cbb);
      }
      const float f = ((float)caa + (float)cab * 0.00390625f) + ((float)cba + (float)cbb * 0.00390625f) * 0.00390625f;
      sc[g][i] = f * (seta[g] * e);
    }
    if (p.draft_len) {                                         // a draft key the request does not use weighs nothing
      const int t = est_sample_key(i, n) - (n - p.draft_len);
      if (t >= 0 && t < 32 && !((p.draft_mask[req] >> t) & 1u))
        for (int g = 0; g < G; ++g) sc[g][i] = -INFINITY;
    }
  }
  __syncthreads();
  publish();
  for (int g = warp; g < G; g += kFrontThreads / 32) {
    const float zval = est_reduce_row(sc[g], n, n_samples, lane);
    if (lane == 0) p.z[(long long)req * p.Hq + kvh * G + g] = zval;
  }
}

// ------------------------------------------------------------------------------------------------
// Scan.
struct PlaneScanParams {
  ScanParams s;                                               // rows, references, value cache, slots, geometry
  PlaneView kv;
  const int8_t *qplanes;
  const float *qeta;
  int vpos_tok, vpos_head, vpos_seq;                          // coordinate order of the value tensor map
  int box_min;                                                // value rows of a sub-slice come as one box from this many live keys on
  float neg_tau;                                              // -tau_K; -inf: refine every live key; +inf: none
  float neg_tau_v;                                            // the same for the refine-V gate (E4M3 value planes)
  int auto_tau_v;                                             // tau_V = max(log2(n) + 1, 4)
  int auto_tau;                                               // tau_K = max(log2(n) - 2, 4) from the sequence's own length
  // E4M3 value planes, finite depth: the sequences' mean value rows (the 8-bit format's cut model), or null
  const __nv_bfloat16 *vrun;
  long long vrun_stride_seq, vrun_stride_head;
};

// 64-key plane-A tiles (Algorithm 1's tile), two gather buffers per warp, three CTAs per SM: the kernel is bound by
// its warps' instruction latencies, so more resident warps beat deeper rings (measured: 2 CTAs/SM 321 us, 3 CTAs/SM
// 285 us on 16 x 8 x 32768 keys; a third gather buffer or 128-key tiles gain nothing).
constexpr int kPlaneTileKeys = 64;                            // keys per plane-A tile
constexpr int kPlaneCtasPerSm = 3;

// TAIL: the block tail's mean value rows (one per 64-key tile = block) ride along in a ring of stages + 1 slots.
template <int D, bool TAIL = false>
struct PlaneLayout {
  static constexpr int kTK = kPlaneTileKeys;
  static constexpr int kATile = kTK * D;                      // plane A codes, swizzled as the tensor map writes them
  static constexpr int kStage = kATile;                       // a ring stage (1 KB-aligned); the tiles' scales have a ring of their own
  static constexpr int kScales = kTK * 2;                     // one tile's scales
  static constexpr int kMeans = TAIL ? 1024 : 0;              // the mean ring: at most 1024 / (2 D) slots
  static constexpr int kMaxStages = TAIL ? 1024 / (2 * D) - 1 : 8;
  static constexpr int kBBuf = 16 * D;                        // plane B rows of one 16-key sub-slice, swizzled like a tile
  static constexpr int kVBuf = 16 * D * 2;                    // value rows of one sub-slice, [D/64][16][128 B] swizzled
  // gather buffers per warp: kBufs - 1 sub-slices' rows in flight while one is multiplied (measured: three at D = 128
  // cost a CTA per SM and lose; four at D = 64 fit and still lose -- there the instruction streams bind, not the rows in flight)
  static constexpr int kBufs = 2;
  static constexpr int kWarpBufs = kBufs * (kBBuf + kVBuf);
  __host__ __device__ static int off_scales(int stages) { return stages * kStage; }
  __host__ __device__ static int off_means(int stages) { return off_scales(stages) + 1024; }                  // scales: <= 8 x 128 B
  __host__ __device__ static int off_bufs(int stages) { return off_means(stages) + kMeans; }                 // 1 KB-aligned
  // the chunk-end reduction parks in the gather buffers (drained by then): 4 warps x R x D floats <= 4 x kWarpBufs
  __host__ __device__ static int off_redl(int stages) { return off_bufs(stages) + kConsumerWarps * kWarpBufs; }
  __host__ __device__ static int off_bar(int stages) { return off_redl(stages) + kConsumerWarps * kMaxRows * 4; }
  __host__ __device__ static int total(int stages) {
    return off_bar(stages) + 2 * stages * 8 + kConsumerWarps * kBufs * 8 + 1024;
  }
};

// Byte offset of 16-byte chunk `ch` of key row `key` in a tile of D-byte rows: the 128-byte swizzle for 128-byte
// rows, the 64-byte swizzle for 64-byte rows (what the tensor map writes; the gather buffers use the same).
template <int D>
__device__ __forceinline__ uint32_t plane_off(int key, int ch) {
  return D == 128 ? (uint32_t)(key * 128 + ((ch ^ (key & 7)) << 4)) : (uint32_t)(key * 64 + ((ch ^ ((key >> 1) & 3)) << 4));
}

__device__ __forceinline__ void mma_s8(int (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// c^xa, c^xb [16 keys, 8 rows] (per row tile) = plane X of 16 keys (rows key0.. of the tile at `tile`) times [Q^a; Q^b]^T.
// c[0], c[1]: key lane/4, rows (lane%4)*2 + {0,1};  c[2], c[3]: key lane/4 + 8.
// NT 8-row tiles of query rows (rows 8 q + ...): one ldmatrix of the key slice feeds every tile's products.
template <int D, int NT>
__device__ __forceinline__ void plane_products(uint32_t tile, int key0, int lane, const uint32_t (&qa)[NT][D / 32][2],
                                               const uint32_t (&qb)[NT][D / 32][2], int (&ca)[NT][4], int (&cb)[NT][4]) {
  // ldmatrix matrix i = lane/8: keys (i&1)*8 + lane%8, 16-byte chunk 2*kk + (i>>1)
  const int key = key0 + (((lane >> 3) & 1) << 3) + (lane & 7);
#pragma unroll
  for (int q = 0; q < NT; ++q) {
    ca[q][0] = ca[q][1] = ca[q][2] = ca[q][3] = 0;
    cb[q][0] = cb[q][1] = cb[q][2] = cb[q][3] = 0;
  }
#pragma unroll
  for (int kk = 0; kk < D / 32; ++kk) {
    uint32_t a[4];
    const int ch = 2 * kk + (lane >> 4);
    ldsm_x4(tile + plane_off<D>(key, ch), a[0], a[1], a[2], a[3]);
#pragma unroll
    for (int q = 0; q < NT; ++q) {
      mma_s8(ca[q], a, qa[q][kk][0], qa[q][kk][1]);
      mma_s8(cb[q], a, qb[q][kk][0], qb[q][kk][1]);
    }
  }
}

// Producer thread: plane A tiles by TMA, their scales by bulk copies, one stage per 128-key tile.
template <int D, bool TAIL>
__device__ __forceinline__ void produce_plane_tiles(const CUtensorMap *tmA, const PlaneScanParams &pp, const SeqWork &w,
                                                    int split, int kvh, int seq, uint32_t ring, uint32_t full0,
                                                    uint32_t empty0) {
  using LO = PlaneLayout<D, TAIL>;
  const ScanParams &p = pp.s;
  tma_prefetch_desc(tmA);
  const uint64_t pol = policy_evict_first();
  bool dead = false;
  int stage = 0, mslot = 0;
  uint32_t wrapped = 0, phase = 0;
  const int boxes_per_tile = LO::kTK / p.box_tok;
  const int page_mask = (1 << p.page_shift) - 1;
  for (TileCursor k = cursor_begin(w, split); cursor_valid(k, w); cursor_next(k, w, p.num_splits)) {
    if (wrapped && !mbar_wait(empty0 + 8u * stage, phase ^ 1u, dead)) break;
    const int tok0 = k.t * LO::kTK;
    const int nbox = min(boxes_per_tile, (w.n - tok0 + p.box_tok - 1) / p.box_tok);
    const uint32_t full = full0 + 8u * stage;
    int sc_tokens = 0;                                       // scale tokens copied: whole groups of 8 (16 bytes)
    for (int bx = 0; bx < nbox; ++bx) sc_tokens += min(p.box_tok, (w.n - (tok0 + bx * p.box_tok) + 7) & ~7);
    mbar_expect_tx(full, nbox * p.box_tok * D + sc_tokens * 2 + (TAIL ? D * 2 : 0));
    const uint32_t dst = ring + stage * LO::kStage;
    if (TAIL) {                                               // the tile is one 64-key block: its mean value row
      bulk_load(ring + LO::off_means(p.stages) + mslot * (D * 2),
                p.vmean + (long long)seq * p.vm_stride_seq + (long long)k.t * p.vm_stride_block + (long long)kvh * p.vm_stride_head,
                D * 2, full);
      if (++mslot == p.stages + 1) mslot = 0;
    }
    for (int bx = 0; bx < nbox; ++bx) {
      const int j0 = tok0 + bx * p.box_tok;
      int c_seq = seq, c_tok = j0;
      if (p.paged) {
        c_seq = min(max(p.page_table[(long long)seq * p.max_pages + (j0 >> p.page_shift)], 0), p.num_pages - 1);
        c_tok = j0 & page_mask;
      }
      const int c1 = p.pos_tok == 1 ? c_tok : (p.pos_head == 1 ? kvh : c_seq);
      const int c2 = p.pos_tok == 2 ? c_tok : (p.pos_head == 2 ? kvh : c_seq);
      const int c3 = p.pos_tok == 3 ? c_tok : (p.pos_head == 3 ? kvh : c_seq);
      tma_load_4d(dst + bx * p.box_tok * D, tmA, full, 0, c1, c2, c3, pol);
      const int cnt = min(p.box_tok, (w.n - j0 + 7) & ~7);
      bulk_load(ring + LO::off_scales(p.stages) + stage * LO::kScales + bx * p.box_tok * 2,
                pp.kv.scale + (long long)c_seq * pp.kv.sc_stride_seq + (long long)kvh * pp.kv.sc_stride_head + c_tok,
                cnt * 2, full);
    }
    if (++stage == p.stages) { stage = 0; wrapped = 1u; phase ^= 1u; }
  }
  if (dead) atomicOr(&p.hdr->wait_timeouts, 1u);
}

// One sub-slice (16 keys) between its coarse pass and its second pass.
template <int NT>
struct PlanePending {
  float x[NT][4];        // coarse score minus reference: key lane/4 (+8), rows 8 q + (lane%4)*2 + {0,1}; -inf if unused
  float e[2];            // the two keys' scales
  uint32_t live, refine; // verdict bits of the 16 keys, ORed over the rows
  uint32_t refv;         // E4M3 value planes: keys whose second value plane is read
  int buf;               // the gather buffer its rows land in
  int ms;                // block tail: the ring slot of its tile's mean value row
};

// DRAFTS: the rows carry draft masks (a separate instantiation: the plain one is at its register limit).
// TAIL: cut keys add weight x the mean value row of their 64-key block (Section 4, "Depth as a dial").
// VFP8: values come from two E4M3 planes (plane 1 for live keys, plane 2 for refine-V keys), widened to BF16 in place.
// NT = 2: 9 to 16 rows per (sequence, kv head) as two 8-row tiles (one ldmatrix feeds both tiles' products; the verdicts
// are ORed over all the rows, as Algorithm 1 takes them over the group); the accumulators double, two CTAs per SM.
template <int D, bool DRAFTS, bool TAIL, bool VFP8 = false, int NT = 1>
__global__ void __launch_bounds__(kDenseThreads, NT == 1 ? kPlaneCtasPerSm : 2)
fold_scan_planes_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmV,
                        const PlaneScanParams pp) {
  using LO = PlaneLayout<D, TAIL>;
  static_assert(!TAIL || LO::kTK == 64, "a tile is one block of the block model");
  constexpr int TK = LO::kTK, U = TK / (16 * kConsumerWarps);          // sub-slices per warp and tile
  constexpr int CV = D / 8, CB = D / 16;                               // 16-byte chunks per value row / plane row
  const ScanParams &p = pp.s;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t *gen = smem_raw + (base - raw);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // x = row group + row_groups * kv head: more than 16 stacked rows (a cascade's shared level) are cut into blocks of
  // 16 rows in row order, each block a CTA of its own that runs Algorithm 1 over its rows (its verdicts are ORed over
  // the block); the blocks of a kv head sit side by side and share its tiles in L2
  const int rg = blockIdx.x % p.row_groups, kvh = blockIdx.x / p.row_groups, split = blockIdx.y, seq = blockIdx.z;
  const SeqWork w = seq_work<TK>(p, seq);
  if (split >= w.n_chunks) return;
  const int rbase = rg * kMaxRows;                            // the block's first row among the (sequence, kv head)'s rows
  const int stages = p.stages, R = min(p.R - rbase, 8 * NT), n = w.n;
  const uint32_t full0 = base + LO::off_bar(stages), empty0 = full0 + 8u * stages;
  const uint32_t gbar0 = empty0 + 8u * stages;               // one barrier per (warp, gather buffer)

  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) {
      mbar_init(full0 + 8u * s, 1);
      mbar_init(empty0 + 8u * s, kConsumerWarps);
    }
    for (int i = 0; i < kConsumerWarps * LO::kBufs; ++i) mbar_init(gbar0 + 8u * i, 1);
    mbar_fence_init();
  }
  __syncthreads();
  pdl_launch_dependents();
  if (warp == kConsumerWarps) {                              // plane A and the scales depend on nothing the front kernel writes
    if (lane == 0) produce_plane_tiles<D, TAIL>(&tmA, pp, w, split, kvh, seq, base, full0, empty0);
    return;
  }
  pdl_wait();                                                // z and the split query rows come from the kernel before

  // query rows: B fragments of the INT8 products (row lane/4), scales and references of the score rows
  uint32_t qa[NT][D / 32][2], qb[NT][D / 32][2];
#pragma unroll
  for (int q = 0; q < NT; ++q) {
    const int r = 8 * q + (lane >> 2);
    const bool ok = r < R;
    const int req = seq * p.stack + (rbase + r) / p.G, head = kvh * p.G + (rbase + r) % p.G;
    const int8_t *qp = pp.qplanes + ((long long)req * p.Hq + head) * (2 * D) + (lane & 3) * 4;
#pragma unroll
    for (int kk = 0; kk < D / 32; ++kk) {
      qa[q][kk][0] = ok ? *reinterpret_cast<const uint32_t *>(qp + kk * 32) : 0u;
      qa[q][kk][1] = ok ? *reinterpret_cast<const uint32_t *>(qp + kk * 32 + 16) : 0u;
      qb[q][kk][0] = ok ? *reinterpret_cast<const uint32_t *>(qp + D + kk * 32) : 0u;
      qb[q][kk][1] = ok ? *reinterpret_cast<const uint32_t *>(qp + D + kk * 32 + 16) : 0u;
    }
  }
  float eta[NT][2], zr[NT][2];
  uint32_t dm[NT][2];                                        // the rows' requests' draft masks (all ones without drafts)
  bool rv[NT][2];
#pragma unroll
  for (int q = 0; q < NT; ++q)
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      const int r = 8 * q + (lane & 3) * 2 + e;
      rv[q][e] = r < R;
      const int req = seq * p.stack + (rbase + r) / p.G;
      const long long row = (long long)req * p.Hq + kvh * p.G + (rbase + r) % p.G;
      eta[q][e] = rv[q][e] ? pp.qeta[row] : 0.f;
      zr[q][e] = rv[q][e] ? p.z[row] : 0.f;
      dm[q][e] = (DRAFTS && rv[q][e]) ? p.draft_mask[req] : 0xffffffffu;
    }
  const int dstart = DRAFTS ? draft_start(p, n) : n;         // keys from here on are per-request drafts
  const float neg_T = p.neg_T;
  const float neg_tau = pp.auto_tau ? -fmaxf(log2f((float)max(n, 1)) - 2.f, 4.f) : pp.neg_tau;
  const float neg_tau_v = pp.auto_tau_v ? -fmaxf(log2f((float)max(n, 1)) + 1.f, 4.f) : pp.neg_tau_v;

  float o[NT][D / 16][4];
  float l_lo[NT], l_hi[NT];
#pragma unroll
  for (int q = 0; q < NT; ++q) {
#pragma unroll
    for (int i = 0; i < D / 16; ++i) o[q][i][0] = o[q][i][1] = o[q][i][2] = o[q][i][3] = 0.f;
    l_lo[q] = l_hi[q] = 0.f;
  }
  const uint32_t bufs = base + LO::off_bufs(stages) + warp * LO::kWarpBufs;
  float *red = reinterpret_cast<float *>(gen + LO::off_bufs(stages));
  float *redl = reinterpret_cast<float *>(gen + LO::off_redl(stages));
  const int klo = lane >> 2;
  const uint32_t gbar_w = gbar0 + 8u * (warp * LO::kBufs);
  bool dead = false;

  // The buffers must never hold bit patterns that read as non-finite BF16: zero them before the first rows land and
  // after the chunk-end reduction has parked FP32 partials in them.
  auto clear_bufs = [&]() {
    for (int i = lane; i < LO::kWarpBufs / 16; i += 32)
      *reinterpret_cast<uint4 *>(gen + LO::off_bufs(stages) + warp * LO::kWarpBufs + i * 16) = make_uint4(0, 0, 0, 0);
    __syncwarp();
  };
  clear_bufs();
  uint32_t gphase = 0;                                       // bit b: parity of buffer b's next completed phase
  // second pass of a sub-slice: plane B product, final weights, value product
  // Block tail: c0 / c1 = this thread's share of the mass rows (lane%4)*2 + {0,1} cut in the sub-slice; the eight lanes that
  // scored the rows' keys are summed, then every channel this thread accumulates takes cut mass x the block's mean value.
  const __nv_bfloat16 *means = reinterpret_cast<const __nv_bfloat16 *>(gen + LO::off_means(stages));
  auto add_tail = [&](float (&c0)[NT], float (&c1)[NT], int ms) {
#pragma unroll
    for (int q = 0; q < NT; ++q)
#pragma unroll
      for (int m = 4; m <= 16; m <<= 1) {
        c0[q] += __shfl_xor_sync(0xffffffffu, c0[q], m);
        c1[q] += __shfl_xor_sync(0xffffffffu, c1[q], m);
      }
    const __nv_bfloat16 *mrow = means + ms * D + klo;
#pragma unroll
    for (int mt = 0; mt < D / 16; ++mt) {
      const float m0 = __bfloat162float(mrow[mt * 16]), m1 = __bfloat162float(mrow[mt * 16 + 8]);
#pragma unroll
      for (int q = 0; q < NT; ++q) {
        o[q][mt][0] = fmaf(c0[q], m0, o[q][mt][0]); o[q][mt][1] = fmaf(c1[q], m0, o[q][mt][1]);
        o[q][mt][2] = fmaf(c0[q], m1, o[q][mt][2]); o[q][mt][3] = fmaf(c1[q], m1, o[q][mt][3]);
      }
    }
  };
  // E4M3 value planes: the mass this thread's two rows cut in the chunk (their share of the sequence's mean value row is
  // added once, at the chunk's end)
  float rcut0[NT], rcut1[NT];
#pragma unroll
  for (int q = 0; q < NT; ++q) rcut0[q] = rcut1[q] = 0.f;
  auto finish = [&](const PlanePending<NT> &pd) {
    const uint32_t bbuf = bufs + pd.buf * (LO::kBBuf + LO::kVBuf), vbuf = bbuf + LO::kBBuf;
    const bool landed = mbar_wait(gbar_w + 8u * pd.buf, (gphase >> pd.buf) & 1u, dead);
    gphase ^= 1u << pd.buf;
    if (!landed) return;
    int ca[NT][4], cb[NT][4];
#pragma unroll
    for (int q = 0; q < NT; ++q)
#pragma unroll
      for (int i = 0; i < 4; ++i) ca[q][i] = cb[q][i] = 0;
    if (pd.refine) plane_products<D, NT>(bbuf, 0, lane, qa, qb, ca, cb);
    uint32_t bh[NT][2], bl[NT][2];
    float cut0[NT], cut1[NT];
#pragma unroll
    for (int q = 0; q < NT; ++q) {
      cut0[q] = cut1[q] = 0.f;
#pragma unroll
      for (int kh = 0; kh < 2; ++kh) {
        const bool klive = (pd.live >> (klo + 8 * kh)) & 1u;
        const bool kref = (pd.refine >> (klo + 8 * kh)) & 1u;   // an unrefined key's buffer row is stale: no correction
        float pw[2], pm[2];
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const int i = 2 * kh + e;
          const float corr = kref ? ((float)ca[q][i] + (float)cb[q][i] * 0.00390625f) * 0.00390625f : 0.f;
          const float x = fmaf(corr, eta[q][e] * pd.e[kh], pd.x[q][i]);
          const bool live = klive && (x >= neg_T);
          pw[e] = ex2_approx(x);
          pm[e] = live ? pw[e] : 0.f;
        }
        const uint32_t hi2 = pack_bf16(pm[0], pm[1]);
        const float h0 = __uint_as_float(hi2 << 16), h1 = __uint_as_float(hi2 & 0xffff0000u);
        const uint32_t lo2 = pack_bf16(pm[0] - h0, pm[1] - h1);
        const float g0 = __uint_as_float(lo2 << 16), g1 = __uint_as_float(lo2 & 0xffff0000u);
        l_lo[q] += (h0 + g0) + (pw[0] - pm[0]);
        l_hi[q] += (h1 + g1) + (pw[1] - pm[1]);
        if (TAIL || VFP8) { cut0[q] += pw[0] - pm[0]; cut1[q] += pw[1] - pm[1]; }
        if (VFP8) {
          // E4M3 values enter the product without their power-of-two scale: it multiplies the weights' BF16 terms instead
          // (exactly: a power of two), while L keeps the weights themselves
          const float vs = pp.kv.v_scale;
          bh[q][kh] = movmatrix_trans(pack_bf16(h0 * vs, h1 * vs));
          bl[q][kh] = movmatrix_trans(pack_bf16(g0 * vs, g1 * vs));
        } else {
          bh[q][kh] = movmatrix_trans(hi2);
          bl[q][kh] = movmatrix_trans(lo2);
        }
      }
    }
    if (VFP8 && pd.live) {
      // widen the landed E4M3 rows to BF16 in place: all reads (two planes, D / 32 units of 16 codes per lane), then
      // all writes into the [D/64][16][128 B] swizzled layout the value product reads.  v1 and v2 widen exactly (to
      // FP16 here), their sum is exact in FP16 and is rounded to BF16 once; rows of keys that are not live become zeros.
      constexpr int UPL = CB / 2;                            // units per lane and plane
      // (the planes' power-of-two scale rides on the weights instead: see the weights above)
      uint4 w1[UPL], w2[UPL];
      uint8_t *vb = gen + (vbuf - base);
      const bool any2 = pd.refv != 0u;                       // warp-uniform: is any second plane there at all?
#pragma unroll
      for (int i = 0; i < UPL; ++i) {
        const int idx = lane + 32 * i, key = idx / CB, u = idx % CB;
        const bool lv = (pd.live >> key) & 1u, r2 = (pd.refv >> key) & 1u;
        w1[i] = lv ? *reinterpret_cast<const uint4 *>(vb + key * D + u * 16) : make_uint4(0, 0, 0, 0);
        w2[i] = r2 ? *reinterpret_cast<const uint4 *>(vb + 16 * D + key * D + u * 16) : make_uint4(0, 0, 0, 0);
      }
      __syncwarp();
#pragma unroll
      for (int i = 0; i < UPL; ++i) {
        const int idx = lane + 32 * i, key = idx / CB, u = idx % CB;
        const uint32_t a[4] = {w1[i].x, w1[i].y, w1[i].z, w1[i].w}, b[4] = {w2[i].x, w2[i].y, w2[i].z, w2[i].w};
        uint32_t outw[8];
#pragma unroll
        for (int j = 0; j < 4; ++j)
#pragma unroll
          for (int hl = 0; hl < 2; ++hl) {
            __half2 h = __half2(__nv_cvt_fp8x2_to_halfraw2((__nv_fp8x2_storage_t)(a[j] >> (16 * hl)), __NV_E4M3));
            if (any2) h = __hadd2(h, __half2(__nv_cvt_fp8x2_to_halfraw2((__nv_fp8x2_storage_t)(b[j] >> (16 * hl)), __NV_E4M3)));
            const float2 f = __half22float2(h);
            outw[2 * j + hl] = pack_bf16(f.x, f.y);
          }
#pragma unroll
        for (int c2 = 0; c2 < 2; ++c2) {
          const int oc = 2 * u + c2;                          // 16-byte chunk of the BF16 row: channels 8 oc .. 8 oc + 7
          *reinterpret_cast<uint4 *>(vb + (oc >> 3) * (16 * 128) + key * 128 + (((oc & 7) ^ (key & 7)) << 4)) =
              make_uint4(outw[4 * c2], outw[4 * c2 + 1], outw[4 * c2 + 2], outw[4 * c2 + 3]);
        }
      }
      __syncwarp();
    }
    if (pd.live) {
      if constexpr (NT == 1) value_product_n<D, true, 0, 16>(o[0], vbuf, 0, lane, bh[0], bl[0]);
      else value_product_nt<D, 16, NT>(o, vbuf, 0, lane, bh, bl, 0u);
    }
    if (VFP8) {
#pragma unroll
      for (int q = 0; q < NT; ++q) { rcut0[q] += cut0[q]; rcut1[q] += cut1[q]; }
    }
    if (TAIL) add_tail(cut0, cut1, pd.ms);                   // (sums the cut mass over the lanes in place)
  };

  int stage = 0, buf = 0, n_pend = 0, mslot = 0;
  uint32_t phase = 0;
  unsigned long long st_total = 0, st_live = 0, st_ref = 0, st_refv = 0;
  PlanePending<NT> pend[LO::kBufs - 1];
  const int page_mask = (1 << p.page_shift) - 1;
  const uint64_t vpol = policy_evict_first();

  for (int c = split; c < w.n_chunks; c += p.num_splits) {
    const int t_end = min((c + 1) * w.ctiles, w.n_tiles);
    for (int t = c * w.ctiles; t < t_end; ++t) {
      const int my_stage = stage, my_ms = mslot;
      const bool ready = mbar_wait(full0 + 8u * my_stage, phase, dead);
      if (++stage == stages) { stage = 0; phase ^= 1u; }
      if (TAIL && ++mslot == stages + 1) mslot = 0;
      if (!ready) continue;
      const uint32_t at = base + my_stage * LO::kStage;
      const __nv_bfloat16 *scales = reinterpret_cast<const __nv_bfloat16 *>(gen + LO::off_scales(stages) + my_stage * LO::kScales);
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int sub = warp * U + u;                         // 16-key sub-slice of the tile
        const int key0 = t * TK + sub * 16;
        if (key0 >= n) continue;                              // warp-uniform
        st_total += min(16, n - key0);
        // coarse pass: plane A against both query planes
        PlanePending<NT> cur;
        int ca[NT][4], cb[NT][4];
        plane_products<D, NT>(at, sub * 16, lane, qa, qb, ca, cb);
        uint32_t lm = 0, rm = 0, vm = 0;
#pragma unroll
        for (int kh = 0; kh < 2; ++kh) {
          const int key = key0 + klo + 8 * kh;
          cur.e[kh] = key < n ? __bfloat162float(scales[sub * 16 + klo + 8 * kh]) : 0.f;
#pragma unroll
          for (int q = 0; q < NT; ++q)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
              const int i = 2 * kh + e;
              const bool ok = key < n && rv[q][e] && (!DRAFTS || draft_ok(dm[q][e], key, dstart));   // an unused draft key: -inf
              const float f = (float)ca[q][i] + (float)cb[q][i] * 0.00390625f;
              const float x = ok ? fmaf(f, eta[q][e] * cur.e[kh], -zr[q][e]) : -INFINITY;
              cur.x[q][i] = x;
              if (ok && x >= neg_T) lm |= 1u << (klo + 8 * kh);
              if (ok && x >= neg_tau) rm |= 1u << (klo + 8 * kh);
              if (VFP8 && ok && x >= neg_tau_v) vm |= 1u << (klo + 8 * kh);
            }
        }
        cur.live = __reduce_or_sync(0xffffffffu, lm);
        cur.refine = __reduce_or_sync(0xffffffffu, rm) & cur.live;
        cur.refv = VFP8 ? __reduce_or_sync(0xffffffffu, vm) & cur.live : 0u;
        if (VFP8) st_refv += __popc(cur.refv);
        cur.buf = buf;
        cur.ms = my_ms;
        st_live += __popc(cur.live);
        st_ref += __popc(cur.refine);
        if (cur.live == 0u) {
          // every key of the sub-slice is cut for every row: no bytes are asked for, nothing is queued, and the weights
          // (the coarse scores are all this scan will ever have for these keys) only add to L
          float cut0[NT], cut1[NT];
#pragma unroll
          for (int q = 0; q < NT; ++q) {
            cut0[q] = cut1[q] = 0.f;
#pragma unroll
            for (int kh = 0; kh < 2; ++kh) {
              cut0[q] += ex2_approx(cur.x[q][2 * kh]);
              cut1[q] += ex2_approx(cur.x[q][2 * kh + 1]);
            }
            l_lo[q] += cut0[q];
            l_hi[q] += cut1[q];
            if (VFP8) { rcut0[q] += cut0[q]; rcut1[q] += cut1[q]; }
          }
          if (TAIL) {
            add_tail(cut0, cut1, my_ms);
            // a queued sub-slice must be finished while its tile's mean row is still in the ring (stages + 1 slots):
            // with the tail on, a dead sub-slice does not let it wait any longer than a live one would
#pragma unroll
            for (int i = 0; i < LO::kBufs - 1; ++i)
              if (i >= LO::kBufs - 1 - n_pend) finish(pend[i]);
            n_pend = 0;
          }
          continue;
        }
        // only now are bytes requested: plane B rows of refined keys, value rows of live keys.  A sub-slice with (nearly)
        // every key live takes its value rows as one tensor-map box; otherwise the live rows are copied one by one.
        // A row that is not fetched keeps what the buffer held -- zeros or an earlier value row, finite either way,
        // times a weight of exactly 0; an unrefined key's plane B row likewise, its correction masked in registers.
        __syncwarp();                                         // the buffer's last readers are done
        {
          const uint32_t bbuf = bufs + buf * (LO::kBBuf + LO::kVBuf), vbuf = bbuf + LO::kBBuf;
          const uint32_t gbar = gbar_w + 8u * buf;
          if (cur.live) {
            long long s_row = seq, t_row = key0;
            if (p.paged) {
              s_row = min(max(p.page_table[(long long)seq * p.max_pages + (key0 >> p.page_shift)], 0), p.num_pages - 1);
              t_row = key0 & page_mask;
            }
            const bool box = !VFP8 && __popc(cur.live) >= pp.box_min && key0 + 16 <= n;
            if (VFP8) {
              // E4M3 planes: plane-1 rows of live keys into the first half of the value buffer (16 rows of D bytes),
              // plane-2 rows of refine-V keys into the second half; the second pass widens them in place
              constexpr int BK = 32 / CB;
              const int ch = lane % CB, k0 = lane / CB;
              const long long off = s_row * pp.kv.stride_seq + (t_row + k0) * pp.kv.stride_tok + (long long)kvh * pp.kv.stride_head + ch * 16;
              const uint8_t *s1 = pp.kv.v1 + off, *s2 = pp.kv.v2 + off;
#pragma unroll
              for (int i = 0; i < 16 / BK; ++i) {
                const int key = k0 + i * BK;
                if ((cur.live >> key) & 1u) cp_async_16(vbuf + key * D + ch * 16, s1, 16u);
                if ((cur.refv >> key) & 1u) cp_async_16(vbuf + 16 * D + key * D + ch * 16, s2, 16u);
                s1 += BK * pp.kv.stride_tok;
                s2 += BK * pp.kv.stride_tok;
              }
            } else if (box) {
              fence_proxy_async_smem();                       // the buffer's earlier generic-proxy traffic, then TMA writes
              __syncwarp();
              if (lane == 0) {
                mbar_expect_tx_only(gbar, 16 * D * 2);
                const int c_seq = (int)s_row, c_tok = (int)t_row;
                const int c1 = pp.vpos_tok == 1 ? c_tok : (pp.vpos_head == 1 ? kvh : c_seq);
                const int c2 = pp.vpos_tok == 2 ? c_tok : (pp.vpos_head == 2 ? kvh : c_seq);
                const int c3 = pp.vpos_tok == 3 ? c_tok : (pp.vpos_head == 3 ? kvh : c_seq);
#pragma unroll
                for (int h = 0; h < D / 64; ++h) tma_load_4d(vbuf + h * (16 * 128), &tmV, gbar, h * 64, c1, c2, c3, vpol);
              }
            } else {
              // lane -> chunk lane % CV of keys lane / CV, + 32 / CV, ...: one pointer step per copy
              constexpr int VK = 32 / CV;
              const int ch = lane % CV, k0 = lane / CV;
              const __nv_bfloat16 *src = p.v + s_row * p.v_stride_seq + (t_row + k0) * p.v_stride_tok +
                                         (long long)kvh * p.v_stride_head + ch * 8;
              const uint32_t dst = vbuf + (ch >> 3) * (16 * 128) + k0 * 128;
#pragma unroll
              for (int i = 0; i < 16 / VK; ++i) {
                const int key = k0 + i * VK;
                if ((cur.live >> key) & 1u) cp_async_16(dst + i * VK * 128 + (((ch & 7) ^ (key & 7)) << 4), src, 16u);
                src += VK * p.v_stride_tok;
              }
            }
            if (cur.refine) {
              constexpr int BK = 32 / CB;
              const int ch = lane % CB, k0 = lane / CB;
              const int8_t *src = pp.kv.b + s_row * pp.kv.stride_seq + (t_row + k0) * pp.kv.stride_tok +
                                  (long long)kvh * pp.kv.stride_head + ch * 16;
#pragma unroll
              for (int i = 0; i < 16 / BK; ++i) {
                const int key = k0 + i * BK;
                if ((cur.refine >> key) & 1u) cp_async_16(bbuf + plane_off<D>(key, ch), src, 16u);
                src += BK * pp.kv.stride_tok;
              }
            }
            if (!box || cur.refine) cp_async_mbar_arrive(gbar);   // this lane's copies hold the phase open
            __syncwarp();
          }
          if (lane == 0) mbar_arrive(gbar);
        }
        // with every buffer now taken, the oldest sub-slice in flight is finished while the newest one's rows travel
        // (the queue is kept at the tail of pend[], so every index is a constant and the entries stay in registers)
        if (n_pend == LO::kBufs - 1) finish(pend[0]);
        else ++n_pend;
#pragma unroll
        for (int i = 0; i + 1 < LO::kBufs - 1; ++i) pend[i] = pend[i + 1];
        pend[LO::kBufs - 2] = cur;
        buf = buf + 1 == LO::kBufs ? 0 : buf + 1;
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(empty0 + 8u * my_stage);     // plane A and the scales are no longer needed
    }
#pragma unroll
    for (int i = 0; i < LO::kBufs - 1; ++i)
      if (i >= LO::kBufs - 1 - n_pend) finish(pend[i]);
    n_pend = 0;
    if (VFP8) {
      if (pp.vrun) {                                          // cut mass x the sequence's mean value row (the 8-bit cut model)
        const __nv_bfloat16 *mrow = pp.vrun + (long long)seq * pp.vrun_stride_seq + (long long)kvh * pp.vrun_stride_head + klo;
#pragma unroll
        for (int q = 0; q < NT; ++q) {
          float c0 = rcut0[q], c1 = rcut1[q];
#pragma unroll
          for (int m = 4; m <= 16; m <<= 1) {
            c0 += __shfl_xor_sync(0xffffffffu, c0, m);
            c1 += __shfl_xor_sync(0xffffffffu, c1, m);
          }
#pragma unroll
          for (int mt = 0; mt < D / 16; ++mt) {
            const float m0 = __bfloat162float(mrow[mt * 16]), m1 = __bfloat162float(mrow[mt * 16 + 8]);
            o[q][mt][0] = fmaf(c0, m0, o[q][mt][0]); o[q][mt][1] = fmaf(c1, m0, o[q][mt][1]);
            o[q][mt][2] = fmaf(c0, m1, o[q][mt][2]); o[q][mt][3] = fmaf(c1, m1, o[q][mt][3]);
          }
        }
      }
#pragma unroll
      for (int q = 0; q < NT; ++q) rcut0[q] = rcut1[q] = 0.f;
    }
    named_bar(1, kConsumerWarps * 32);                        // every warp's buffers are drained: park there
    float *slot = p.slots + (((long long)seq * p.Hkv + kvh) * p.max_slots + c) * p.slot_stride;
#pragma unroll
    for (int q = 0; q < NT; ++q) {                            // a tile's rows: 8 q .. 8 q + 7, as many as the block has
      const int Rq = min(8, R - 8 * q);
      reduce_store_L_n<kConsumerWarps>(l_lo[q], l_hi[q], redl, slot + p.R * D + rbase + 8 * q, Rq, warp, lane, threadIdx.x, 1);
      reduce_store_A_n<D, kConsumerWarps>(o[q], red, slot + (rbase + 8 * q) * D, Rq, warp, lane, threadIdx.x, 1);
    }
    if (c + p.num_splits < w.n_chunks) clear_bufs();
  }

  if (lane == 0) {
    if (dead) atomicOr(&p.hdr->wait_timeouts, 2u);
    atomicAdd(reinterpret_cast<unsigned long long *>(&p.hdr->v_rows_fetched), st_live);
    atomicAdd(reinterpret_cast<unsigned long long *>(&p.hdr->v_rows_total), st_total);
    atomicAdd(reinterpret_cast<unsigned long long *>(&p.hdr->k_rows_refined), st_ref);
    if (VFP8) atomicAdd(reinterpret_cast<unsigned long long *>(&p.hdr->v2_rows_refined), st_refv);
  }
}

}  // namespace fold
