// Reference kernels: the 192-key estimate of Z (Section 3, "Choosing the reference") and
// the exact-maximum test mode.
//
// Estimate, per (request, q head), over the request's logical key sequence (the
// concatenation of up to four cache levels): rows of at most 192 keys use their exact
// base-2 log-sum-exp; longer rows score key 0 (the sink) and the last 63 keys exactly and
// take the mass of the n-64 keys between them as (n-64) * mean of the 128 stratum-centre
// weights with the 8 largest dropped.
#pragma once

#include "fold_common.cuh"

namespace fold {

constexpr int kEstSamples = 192;
constexpr int kEstRecent = 63;
constexpr int kEstStrata = 128;
constexpr int kEstTrim = 8;
constexpr int kEstThreads = 256;

struct KvLevel {
  const __nv_bfloat16 *k;
  long long stride_seq, stride_tok, stride_head;
  const int *page_table;
  const int *seqlens;
  int paged, page_shift, max_pages, num_pages, stack, max_seqlen;
};

struct EstParams {
  const __nv_bfloat16 *q;
  long long q_stride_b, q_stride_h;
  float *z;
  KvLevel lv[kMaxLevels];
  int n_levels, Hq, Hkv, G;
  float scale_log2;
  const uint32_t *draft_mask;    // drafts: the last draft_len keys (of the concatenated levels) are used by request
  int draft_len;                 // req only where its mask has the bit
  fold_ws_header *hdr[kMaxLevels];   // not null: this launch also zeroes that level's workspace header (a memset less)
};

__device__ __forceinline__ int level_len(const KvLevel &L, int req) {
  int n = L.seqlens[req / L.stack];
  return n < 0 ? 0 : (n > L.max_seqlen ? L.max_seqlen : n);
}

// Address of key row `tok` of sequence `seq` (caller guarantees tok < that sequence's length).
__device__ __forceinline__ const __nv_bfloat16 *key_row(const KvLevel &L, int seq, int tok, int kvh) {
  long long s = seq, t = tok;
  if (L.paged) {
    int pg = L.page_table[(long long)seq * L.max_pages + (tok >> L.page_shift)];
    pg = min(max(pg, 0), L.num_pages - 1);
    s = pg;
    t = tok & ((1 << L.page_shift) - 1);
  }
  return L.k + s * L.stride_seq + t * L.stride_tok + (long long)kvh * L.stride_head;
}

// Which logical key the i-th sample of a row of n keys is.
__device__ __forceinline__ int est_sample_key(int i, int n) {
  if (n <= kEstSamples) return i;
  if (i == 0) return 0;
  if (i <= kEstRecent) return n - kEstRecent + (i - 1);
  const int k = i - 1 - kEstRecent;
  const long long n_mid = n - 1 - kEstRecent;
  const int e0 = 1 + (int)((k * n_mid) / kEstStrata);
  const int e1 = 1 + (int)(((k + 1) * n_mid) / kEstStrata);
  return (e0 + e1) >> 1;
}

// One warp finishes one row from its sampled scores row[0 .. n_samples): maximum, exact part, trimmed
// stratified part.  n = the row's key count.  Every lane returns the row's reference.
__device__ __forceinline__ float est_reduce_row(const float *row, int n, int n_samples, int lane) {
  float zval = 0.f;
  if (n_samples > 0) {
    float m = -INFINITY;
    for (int k = lane; k < n_samples; k += 32) m = fmaxf(m, row[k]);
#pragma unroll
    for (int k = 16; k > 0; k >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, k));
    float total = 0.f;                             // fixed summation order: lane-strided, then a shuffle tree
    if (n <= kEstSamples) {
      for (int k = lane; k < n_samples; k += 32) total += exp2f(row[k] - m);
    } else {
      for (int k = lane; k <= kEstRecent; k += 32) total += exp2f(row[k] - m);      // sink + 63 recent
      // the 128 centre scores, four per lane (centre lane + 32 i); drop the 8 largest, one per round:
      // the warp-wide maximum, owned by the lowest index among equals
      float c[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) c[i] = row[1 + kEstRecent + lane + 32 * i];
      // (floats compared as order-preserving unsigned keys, so that the warp-wide maximum is one redux instruction)
      auto key_of = [](float f) { const uint32_t b = __float_as_uint(f); return (b & 0x80000000u) ? ~b : (b | 0x80000000u); };
#pragma unroll 1
      for (int r = 0; r < kEstTrim; ++r) {
        const uint32_t k0 = key_of(c[0]), k1 = key_of(c[1]), k2 = key_of(c[2]), k3 = key_of(c[3]);
        const uint32_t mine = max(max(k0, k1), max(k2, k3));
        const uint32_t wm = __reduce_max_sync(0xffffffffu, mine);
        const unsigned owners = __ballot_sync(0xffffffffu, mine == wm);
        if (lane == __ffs(owners) - 1) {                     // the lowest lane among equals drops one of its own
          if (k0 == wm) c[0] = -INFINITY;
          else if (k1 == wm) c[1] = -INFINITY;
          else if (k2 == wm) c[2] = -INFINITY;
          else c[3] = -INFINITY;
        }
      }
      float kept = 0.f;
#pragma unroll
      for (int i = 0; i < 4; ++i) kept += exp2f(c[i] - m);                              // dropped ones add 2^-inf = 0
      total += kept * ((float)(n - 1 - kEstRecent) / (float)(kEstStrata - kEstTrim));
    }
#pragma unroll
    for (int k = 16; k > 0; k >>= 1) total += __shfl_xor_sync(0xffffffffu, total, k);
    zval = m + log2f(total);
  }
  return zval;
}

// The 192 x G scores of one (kv head, request) are one small matrix product, formed in blocks of 16 sampled keys: a
// warp takes block `blk` (samples 16 blk .. 16 blk + 15) on M and the group's query rows on N (mma.sync m16n8k16,
// BF16 in, FP32 accumulate) and writes the scaled scores to sc[row][sample].  Each lane loads its A fragments
// straight from the cache rows (all loads issued before the first MMA, so a block pays one memory latency).
// n = the request's key count over all levels, lens[] per level.  A score's bits do not depend on which warp of
// which kernel forms it.
constexpr int kEstWarps = kEstSamples / 16;              // 12
constexpr int kEstSampleThreads = kEstWarps * 32;        // 384

// NB blocks at once (blk0, blk0 + blk_step, ...): all their cache rows are requested before the first product, so
// the warp pays one memory latency for the lot.
template <int D, int NB>
__device__ __forceinline__ void est_score_blocks(const EstParams &p, int req, int kvh, int blk0, int blk_step, int lane,
                                                 int n, const int (&lens)[kMaxLevels], float (*sc)[kEstSamples]) {
  constexpr int KS = D / 16;
  const int G = p.G;
  const int n_samples = n < kEstSamples ? n : kEstSamples;
  const int qcol = (lane & 3) * 2;
  const int qcol4 = (lane & 3) * 8;                          // this lane's 8 consecutive channels of every 32
  // A dot product does not care in which order its terms meet: the k slots of each pair of MMAs are assigned so
  // that a lane's fragments of 32 channels are 8 CONSECUTIVE channels of its row (one 16-byte load) -- MMA 2j takes
  // channels 32j + 8t + {0,1 | 2,3} in its slots {2t,2t+1 | 2t+8,2t+9}, MMA 2j+1 takes 32j + 8t + {4,5 | 6,7} -- and
  // the query fragments below follow the same assignment.
  uint4 ka[NB][2][KS / 2];                                   // [block][row lane/4, row lane/4 + 8][32-channel group]
#pragma unroll
  for (int b = 0; b < NB; ++b) {
    const int blk = blk0 + b * blk_step;
#pragma unroll
    for (int hlf = 0; hlf < 2; ++hlf) {
      // the two sampled key rows this lane reads fragments of
      const int i = blk * 16 + (lane >> 2) + hlf * 8;
      const __nv_bfloat16 *rowp = nullptr;
      if (blk < kEstWarps && i < n_samples) {
        int j = est_sample_key(i, n), l = 0;
        while (l < p.n_levels - 1 && j >= lens[l]) { j -= lens[l]; ++l; }
        rowp = key_row(p.lv[l], req / p.lv[l].stack, j, kvh) + qcol4;
      }
#pragma unroll
      for (int j = 0; j < KS / 2; ++j)
        ka[b][hlf][j] = rowp ? *reinterpret_cast<const uint4 *>(rowp + j * 32) : make_uint4(0, 0, 0, 0);
    }
  }
  // query rows of the group as B fragments (n = lane / 4), eight rows per n-tile
#pragma unroll 1
  for (int nt = 0; nt * 8 < G; ++nt) {
    const int g = nt * 8 + (lane >> 2);
    const __nv_bfloat16 *qrow = p.q + (long long)req * p.q_stride_b + (long long)(kvh * G + g) * p.q_stride_h + qcol4;
    uint4 qb[KS / 2];
#pragma unroll
    for (int j = 0; j < KS / 2; ++j) qb[j] = g < G ? *reinterpret_cast<const uint4 *>(qrow + j * 32) : make_uint4(0, 0, 0, 0);
#pragma unroll
    for (int b = 0; b < NB; ++b) {
      const int blk = blk0 + b * blk_step;
      if (blk >= kEstWarps || blk * 16 >= n_samples) continue;
      float c[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int j = 0; j < KS / 2; ++j) {
        const uint4 r0 = ka[b][0][j], r1 = ka[b][1][j];
        const uint32_t a0[4] = {r0.x, r1.x, r0.y, r1.y}, a1[4] = {r0.z, r1.z, r0.w, r1.w};
        mma_bf16(c, a0, qb[j].x, qb[j].y);
        mma_bf16(c, a1, qb[j].z, qb[j].w);
      }
      // c0, c1: key lane/4, rows 2*(lane%4) + {0,1};  c2, c3: key lane/4 + 8
      const int i0 = blk * 16 + (lane >> 2), g0 = nt * 8 + qcol;
      if (p.draft_len) {                                     // a draft key the request does not use weighs nothing
        const uint32_t dm = p.draft_mask[req];
        const int dstart = n - p.draft_len;
#pragma unroll
        for (int hlf = 0; hlf < 2; ++hlf) {
          const int i = i0 + 8 * hlf;
          const int t = i < n_samples ? est_sample_key(i, n) - dstart : -1;
          if (t >= 0 && t < 32 && !((dm >> t) & 1u)) c[2 * hlf] = c[2 * hlf + 1] = -INFINITY;
        }
      }
      if (g0 < G) { sc[g0][i0] = c[0] * p.scale_log2; sc[g0][i0 + 8] = c[2] * p.scale_log2; }
      if (g0 + 1 < G) { sc[g0 + 1][i0] = c[1] * p.scale_log2; sc[g0 + 1][i0 + 8] = c[3] * p.scale_log2; }
    }
  }
}

// One CTA per (kv head, request), 12 warps, a block of 16 samples each; warp g then reduces row g.
template <int D>
__global__ void __launch_bounds__(kEstSampleThreads) fold_estimate_kernel(const EstParams p) {
  __shared__ float sc[kMaxRows][kEstSamples];
  const int kvh = blockIdx.x, req = blockIdx.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int G = p.G;
  pdl_launch_dependents();                           // the scan may set up while the estimate runs

  int lens[kMaxLevels];
  int n = 0;
#pragma unroll
  for (int l = 0; l < kMaxLevels; ++l) {
    lens[l] = l < p.n_levels ? level_len(p.lv[l], req) : 0;
    n += lens[l];
  }
  const int n_samples = n < kEstSamples ? n : kEstSamples;
  est_score_blocks<D, 1>(p, req, kvh, warp, 1, lane, n, lens, sc);
  __syncthreads();
  // Everything above reads only the caller's inputs.  What follows writes: z, which the partial add of a call before
  // this one may still be reading, and the workspace headers -- so it waits for the kernels before (a no-op unless this
  // kernel was launched early behind one that allows it).
  pdl_wait();
  if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x < 16)
    for (int l = 0; l < p.n_levels; ++l)                  // the scans touch their headers only after their dependency wait
      if (p.hdr[l]) reinterpret_cast<uint32_t *>(p.hdr[l])[threadIdx.x] = 0u;

  // warp g finishes row g
  for (int g = warp; g < G; g += kEstSampleThreads / 32) {
    const float zval = est_reduce_row(sc[g], n, n_samples, lane);
    if (lane == 0) p.z[(long long)req * p.Hq + kvh * G + g] = zval;
  }
}

// Test mode: z = max_j s_ij over every key of a single level.
template <int D>
__global__ void __launch_bounds__(kEstThreads) fold_exact_max_kernel(const EstParams p) {
  constexpr int EPL = D / 32;
  __shared__ float qs[kMaxRows][D];
  __shared__ float wm[kEstThreads / 32][kMaxRows];
  const int kvh = blockIdx.x, req = blockIdx.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int G = p.G;
  const int n = level_len(p.lv[0], req);
  for (int i = threadIdx.x; i < G * D; i += kEstThreads) {
    const int g = i / D, d = i % D;
    qs[g][d] = __bfloat162float(p.q[(long long)req * p.q_stride_b + (long long)(kvh * G + g) * p.q_stride_h + d]);
  }
  __syncthreads();
  float best[kMaxRows];
  for (int g = 0; g < kMaxRows; ++g) best[g] = -INFINITY;
  for (int j = warp; j < n; j += kEstThreads / 32) {
    const __nv_bfloat16 *row = key_row(p.lv[0], req / p.lv[0].stack, j, kvh) + lane * EPL;
    float kf[EPL];
#pragma unroll
    for (int e = 0; e < EPL; ++e) kf[e] = __bfloat162float(row[e]);
    for (int g = 0; g < G; ++g) {
      float acc = 0.f;
#pragma unroll
      for (int e = 0; e < EPL; ++e) acc = fmaf(kf[e], qs[g][lane * EPL + e], acc);
#pragma unroll
      for (int m = 16; m > 0; m >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, m);
      best[g] = fmaxf(best[g], acc * p.scale_log2);
    }
  }
  if (lane == 0)
    for (int g = 0; g < G; ++g) wm[warp][g] = best[g];
  __syncthreads();
  if (threadIdx.x < G) {
    float m = -INFINITY;
    for (int w = 0; w < kEstThreads / 32; ++w) m = fmaxf(m, wm[w][threadIdx.x]);
    p.z[(long long)req * p.Hq + kvh * G + threadIdx.x] = n > 0 ? m : 0.f;
  }
}

__global__ void fold_fill_kernel(float *z, int count, float value) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < count) z[i] = value;
}

// ------------------------------------------------------------------------------------------------
// Block means for the block tail (Section 4, "Depth as a dial"): one warp per (sequence, 64-key block, kv head),
// each lane D / 32 channels; the block's value rows are summed in float64 in key order, divided by the key count
// and rounded to FP32, then to BF16.
struct MeanParams {
  const __nv_bfloat16 *v;
  long long v_stride_seq, v_stride_tok, v_stride_head;
  __nv_bfloat16 *mean;
  long long m_stride_seq, m_stride_block, m_stride_head;
  const int *seqlens;
  const int *page_table;
  int max_seqlen, page_shift, max_pages, num_pages, Hkv;
};

template <int D>
__global__ void __launch_bounds__(128) fold_block_mean_kernel(const MeanParams p) {
  constexpr int EPT = D / 32;
  const int lane = threadIdx.x, blk = blockIdx.x * 4 + threadIdx.y, kvh = blockIdx.y, seq = blockIdx.z;
  int n = p.seqlens[seq];
  n = n < 0 ? 0 : (n > p.max_seqlen ? p.max_seqlen : n);
  const int j0 = blk * 64, j1 = min(j0 + 64, n);
  if (j0 >= n) return;
  double acc[EPT];
#pragma unroll
  for (int e = 0; e < EPT; ++e) acc[e] = 0.0;
  const int page_mask = (1 << p.page_shift) - 1;
  for (int j = j0; j < j1; ++j) {
    long long s_row = seq, t_row = j;
    if (p.page_table) {
      const int pg = p.page_table[(long long)seq * p.max_pages + (j >> p.page_shift)];
      s_row = min(max(pg, 0), p.num_pages - 1);
      t_row = j & page_mask;
    }
    const __nv_bfloat16 *row = p.v + s_row * p.v_stride_seq + t_row * p.v_stride_tok + (long long)kvh * p.v_stride_head + lane * EPT;
    if (EPT == 4) {
      const uint2 w = *reinterpret_cast<const uint2 *>(row);
      acc[0] += (double)__uint_as_float(w.x << 16); acc[1] += (double)__uint_as_float(w.x & 0xffff0000u);
      acc[EPT - 2] += (double)__uint_as_float(w.y << 16); acc[EPT - 1] += (double)__uint_as_float(w.y & 0xffff0000u);
    } else {
      const uint32_t w = *reinterpret_cast<const uint32_t *>(row);
      acc[0] += (double)__uint_as_float(w << 16); acc[1] += (double)__uint_as_float(w & 0xffff0000u);
    }
  }
  const double cnt = (double)(j1 - j0);
  __nv_bfloat16 *dst = p.mean + (long long)seq * p.m_stride_seq + (long long)blk * p.m_stride_block +
                       (long long)kvh * p.m_stride_head + lane * EPT;
#pragma unroll
  for (int e = 0; e < EPT; ++e) dst[e] = __float2bfloat16_rn(__double2float_rn(acc[e] / cnt));
}

// The cut model of the 8-bit value format (Section 4, "Depth as a dial": a mean kept per request): the mean of all
// the value rows of a (sequence, kv head), written as block 0 of the mean table.  One CTA of 32 warps per (kv head,
// sequence): warp w sums rows w, w + 32, ... in float64, the warps' sums are added in warp order, the quotient is rounded
// to FP32 and then to BF16 like the block means.
constexpr int kRunMeanWarps = 32;
template <int D>
__global__ void __launch_bounds__(32 * kRunMeanWarps) fold_running_mean_kernel(const MeanParams p) {
  constexpr int EPT = D / 32;
  __shared__ double part[kRunMeanWarps][D];
  const int lane = threadIdx.x, wy = threadIdx.y, kvh = blockIdx.x, seq = blockIdx.y;
  int n = p.seqlens[seq];
  n = n < 0 ? 0 : (n > p.max_seqlen ? p.max_seqlen : n);
  double acc[EPT];
#pragma unroll
  for (int e = 0; e < EPT; ++e) acc[e] = 0.0;
  const int page_mask = (1 << p.page_shift) - 1;
#pragma unroll 4
  for (int j = wy; j < n; j += kRunMeanWarps) {
    long long s_row = seq, t_row = j;
    if (p.page_table) {
      const int pg = p.page_table[(long long)seq * p.max_pages + (j >> p.page_shift)];
      s_row = min(max(pg, 0), p.num_pages - 1);
      t_row = j & page_mask;
    }
    const __nv_bfloat16 *row = p.v + s_row * p.v_stride_seq + t_row * p.v_stride_tok + (long long)kvh * p.v_stride_head + lane * EPT;
    if (EPT == 4) {
      const uint2 w = *reinterpret_cast<const uint2 *>(row);
      acc[0] += (double)__uint_as_float(w.x << 16); acc[1] += (double)__uint_as_float(w.x & 0xffff0000u);
      acc[EPT - 2] += (double)__uint_as_float(w.y << 16); acc[EPT - 1] += (double)__uint_as_float(w.y & 0xffff0000u);
    } else {
      const uint32_t w = *reinterpret_cast<const uint32_t *>(row);
      acc[0] += (double)__uint_as_float(w << 16); acc[1] += (double)__uint_as_float(w & 0xffff0000u);
    }
  }
#pragma unroll
  for (int e = 0; e < EPT; ++e) part[wy][lane * EPT + e] = acc[e];
  __syncthreads();
  if (wy != 0) return;
  __nv_bfloat16 *dst = p.mean + (long long)seq * p.m_stride_seq + (long long)kvh * p.m_stride_head + lane * EPT;
#pragma unroll
  for (int e = 0; e < EPT; ++e) {
    double t = 0.0;
#pragma unroll
    for (int w = 0; w < kRunMeanWarps; ++w) t += part[w][lane * EPT + e];
    dst[e] = n > 0 ? __float2bfloat16_rn(__double2float_rn(t / (double)n)) : __float2bfloat16_rn(0.f);
  }
}

}  // namespace fold
