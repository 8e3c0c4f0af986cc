// Order-free partial add (Prop. 1(i)), used for the split-KV merge and the shared-prefix
// cascade merge.  Partials are FP32; to make the result a function of the SET of partials
// (any slot order, any grouping, any level order gives the same bits) each element is
// summed on an integer grid declared before the reduction (Eq. 3 / Prop. 2): the largest
// magnitude among the C terms is found with an order-free integer maximum over their bit
// patterns, the grid is alpha = 2^(61 - ceil(log2 C) - e_max - 1) (e_max >= -126: subnormal maxima
// use their fixed scale), every term is rounded to nearest-even on it (exactly: a power-of-two
// product in double, then a round-to-nearest-even conversion) and added as a 64-bit integer.
#pragma once

#include "fold_common.cuh"

namespace fold {

constexpr int kMergeMaxWarps = 16;

struct MergeLevel {
  const float *slots;
  const int *seqlens;
  long long slot_stride;
  int stack, max_slots, rows, max_seqlen;
};

struct MergeParams {
  MergeLevel lv[kMaxLevels];
  const float *z;
  __nv_bfloat16 *out;
  float *lse;
  int *row_status;
  int n_levels, Hq, Hkv, G, D;
};

__device__ __forceinline__ int ceil_log2_u32(unsigned c) { return c <= 1 ? 0 : 32 - __clz(c - 1); }

// log2(alpha) for C terms whose largest magnitude has bit pattern maxbits (sign cleared); subnormal
// maxima use their fixed scale (e_max = -126).
__device__ __forceinline__ int grid_shift(unsigned maxbits, int clog2C) {
  const int ef = (int)(maxbits >> 23);
  const int e_max = ef == 0 ? -126 : ef - 127;
  return 61 - (clog2C + e_max + 1);
}
__device__ __forceinline__ double pow2_double(int e) {       // 2^e, e in the normal range
  return __longlong_as_double((long long)(e + 1023) << 52);
}
// RNE(alpha * g) as an integer: the product with a power of two is exact in double, the conversion rounds to
// nearest even; |result| < 2^61 / C.
__device__ __forceinline__ long long to_grid(float g, double alpha) { return __double2ll_rn((double)g * alpha); }

// One row (a row = one (request, q head)) summed by W in {1, 2, 4, 8, 16} warps that share its slots (warp `sub`
// takes slots sub, sub + W, ... of every level); wi = this warp's index among the warps that meet at `sync` (its row
// of the staging arrays), the row's first warp being wi - sub.  Lane x owns EPT = D / 32
// consecutive elements of A (one vector load per slot); lane 0 also carries L.  Two passes over the slots (the
// second hits L1): the order-free maximum, then the integer sum.  The W warps of a row combine through staged
// partials in shared memory: maxima by max, integer sums by integer addition, both exact, so neither the warp
// count nor the slot order can change a bit.  Every warp that shares the staging arrays calls this together (sync
// is their barrier; it is crossed twice when W > 1), active or not.
// RESIDENT (one level, at most kMergeResident slots per warp): the slots are loaded once and stay in registers for
// the second pass.
constexpr int kMergeResident = 8;
template <int EPT, bool RESIDENT, typename Sync>
__device__ __forceinline__ void merge_row(const MergeParams &p, const int W, const long long row, const bool active,
                                          const int sub, const int wi, const int x, unsigned (*s_max)[32 * EPT + 1],
                                          long long (*s_sum)[32 * EPT + 1], Sync sync) {
  constexpr int D = 32 * EPT;
  const int b = active ? (int)(row / p.Hq) : 0, h = active ? (int)(row % p.Hq) : 0;
  const int G = p.G, kvh = h / G, hg = h % G;
  const float zrow = active ? p.z[row] : 0.f;        // requested early: only needed at the very end

  auto load_vec = [](const float *a, float (&v)[EPT]) {
    if (EPT == 4) {
      const float4 t = *reinterpret_cast<const float4 *>(a);
      v[0] = t.x; v[1] = t.y; v[EPT - 2] = t.z; v[EPT - 1] = t.w;
    } else {
      const float2 t = *reinterpret_cast<const float2 *>(a);
      v[0] = t.x; v[1] = t.y;
    }
  };
  // level l as this warp sees it: slot count, this lane's first A vector, the row's first L element, the step
  auto level = [&](int l, int &cnt, const float *&a, const float *&q, long long &step) {
    const MergeLevel &L = p.lv[l];
    const int seq = b / L.stack;
    int n = L.seqlens[seq];
    n = n < 0 ? 0 : (n > L.max_seqlen ? L.max_seqlen : n);
    cnt = active ? num_chunks_of(n) : 0;
    const int r = (b % L.stack) * G + hg;
    const float *s0 = L.slots + (((long long)seq * p.Hkv + kvh) * L.max_slots + sub) * L.slot_stride;
    a = s0 + r * D + x * EPT;
    q = s0 + L.rows * D + r;
    step = L.slot_stride * W;
  };

  // pass 1: order-free maximum of |g| through the bit patterns; C = the number of terms
  unsigned mx[EPT], mxl = 0u, C = 0;
#pragma unroll
  for (int e = 0; e < EPT; ++e) mx[e] = 0u;
  float rv[RESIDENT ? kMergeResident : 1][EPT], rl[RESIDENT ? kMergeResident : 1];
  if (RESIDENT) {
    int cnt; const float *a, *q; long long step;
    level(0, cnt, a, q, step);
    C = cnt;
#pragma unroll
    for (int i = 0; i < kMergeResident; ++i) {
      const bool on = sub + i * W < cnt;
#pragma unroll
      for (int e = 0; e < EPT; ++e) rv[i][e] = 0.f;
      rl[i] = 0.f;
      if (on) {
        load_vec(a + i * step, rv[i]);
        if (x == 0) rl[i] = q[i * step];
      }
#pragma unroll
      for (int e = 0; e < EPT; ++e) mx[e] = max(mx[e], __float_as_uint(rv[i][e]) & 0x7fffffffu);
      mxl = max(mxl, __float_as_uint(rl[i]) & 0x7fffffffu);
    }
  }
#pragma unroll 1
  for (int l = 0; l < (RESIDENT ? 0 : p.n_levels); ++l) {
    int cnt; const float *a, *q; long long step;
    level(l, cnt, a, q, step);
    C += cnt;
#pragma unroll 4
    for (int k = sub; k < cnt; k += W, a += step, q += step) {
      float v[EPT];
      load_vec(a, v);
#pragma unroll
      for (int e = 0; e < EPT; ++e) mx[e] = max(mx[e], __float_as_uint(v[e]) & 0x7fffffffu);
      if (x == 0) mxl = max(mxl, __float_as_uint(*q) & 0x7fffffffu);
    }
  }
  if (W > 1) {
#pragma unroll
    for (int e = 0; e < EPT; ++e) s_max[wi][e * 32 + x] = mx[e];
    if (x == 0) s_max[wi][D] = mxl;
    sync();
    const int w0 = wi - sub;
    for (int o = 0; o < W; ++o) {
#pragma unroll
      for (int e = 0; e < EPT; ++e) mx[e] = max(mx[e], s_max[w0 + o][e * 32 + x]);
      mxl = max(mxl, s_max[w0 + o][D]);              // lanes other than 0 carry it along unused
    }
  }
  mxl = __shfl_sync(0xffffffffu, mxl, 0);
  const int clog2C = ceil_log2_u32(C);

  // pass 2: integer sums on the declared grid
  long long acc[EPT], accl = 0;
  double alpha[EPT];
  bool fin[EPT];
#pragma unroll
  for (int e = 0; e < EPT; ++e) {
    acc[e] = 0;
    alpha[e] = pow2_double(grid_shift(mx[e], clog2C));
    fin[e] = (mx[e] >> 23) != 255u;
  }
  const double alpha_l = pow2_double(grid_shift(mxl, clog2C));
  const bool fin_l = (mxl >> 23) != 255u;
  if (RESIDENT) {                                    // absent slots hold zeros, which add nothing
#pragma unroll
    for (int i = 0; i < kMergeResident; ++i) {
#pragma unroll
      for (int e = 0; e < EPT; ++e) if (fin[e]) acc[e] += to_grid(rv[i][e], alpha[e]);
      if (x == 0 && fin_l) accl += to_grid(rl[i], alpha_l);
    }
  }
#pragma unroll 1
  for (int l = 0; l < (RESIDENT ? 0 : p.n_levels); ++l) {
    int cnt; const float *a, *q; long long step;
    level(l, cnt, a, q, step);
#pragma unroll 4
    for (int k = sub; k < cnt; k += W, a += step, q += step) {
      float v[EPT];
      load_vec(a, v);
#pragma unroll
      for (int e = 0; e < EPT; ++e) if (fin[e]) acc[e] += to_grid(v[e], alpha[e]);
      if (x == 0 && fin_l) accl += to_grid(*q, alpha_l);
    }
  }
  if (W > 1) {
#pragma unroll
    for (int e = 0; e < EPT; ++e) s_sum[wi][e * 32 + x] = acc[e];
    if (x == 0) s_sum[wi][D] = accl;
    sync();
    if (sub != 0) return;
    for (int o = 1; o < W; ++o) {
#pragma unroll
      for (int e = 0; e < EPT; ++e) acc[e] += s_sum[wi + o][e * 32 + x];
      accl += s_sum[wi + o][D];
    }
  }
  if (!active) return;

  // the row's first warp finishes it
  float Lf = fin_l ? (float)((double)accl * pow2_double(-grid_shift(mxl, clog2C))) : __int_as_float(0x7fc00000);
  Lf = __shfl_sync(0xffffffffu, Lf, 0);
  bool bad = false;
  __nv_bfloat16 ob[EPT];
#pragma unroll
  for (int e = 0; e < EPT; ++e) {
    const float Af = fin[e] ? (float)((double)acc[e] * pow2_double(-grid_shift(mx[e], clog2C)))
                            : __int_as_float(0x7fc00000);
    const float ov = C == 0 ? 0.f : Af / Lf;
    bad |= !(fabsf(ov) <= 3.4e38f);
    ob[e] = __float2bfloat16_rn(ov);
  }
  if (EPT == 4) *reinterpret_cast<uint2 *>(p.out + row * D + x * EPT) = *reinterpret_cast<uint2 *>(ob);
  else *reinterpret_cast<uint32_t *>(p.out + row * D + x * EPT) = *reinterpret_cast<uint32_t *>(ob);
  const unsigned any_bad = __ballot_sync(0xffffffffu, bad);
  if (x == 0) {
    int flags = any_bad ? FOLD_ROW_NONFINITE : 0;
    float lse;
    if (C == 0) {
      flags = FOLD_ROW_EMPTY;
      lse = -INFINITY;
    } else {
      if (!(fabsf(Lf) <= 3.4e38f)) flags |= FOLD_ROW_NONFINITE;
      if (!(Lf >= 0.5f && Lf <= 1.2676506e30f)) flags |= FOLD_ROW_RANGE;      // [2^-1, 2^100]
      lse = zrow + log2f(Lf);
    }
    if (p.lse) p.lse[row] = lse;
    if (p.row_status) p.row_status[row] = flags;
  }
}

// One CTA of blockDim.x / 32 warps (at most kMergeMaxWarps) covers that many / W rows.
template <int EPT, bool RESIDENT>
__global__ void __launch_bounds__(32 * kMergeMaxWarps) fold_merge_kernel(const MergeParams p, const int W,
                                                                         const long long n_rows) {
  constexpr int D = 32 * EPT;
  __shared__ unsigned s_max[kMergeMaxWarps][D + 1];
  __shared__ long long s_sum[kMergeMaxWarps][D + 1];
  const int x = threadIdx.x & 31, wi = threadIdx.x >> 5;
  const long long row = (long long)blockIdx.x * ((blockDim.x >> 5) / W) + wi / W;
  pdl_launch_dependents();                           // the next call's reference kernel may set up and load meanwhile
  pdl_wait();                                        // slots and z come from the kernels before
  merge_row<EPT, RESIDENT>(p, W, row, row < n_rows, wi % W, wi, x, s_max, s_sum, [] { __syncthreads(); });
}

}  // namespace fold
