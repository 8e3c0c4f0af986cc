// Order-free partial add (Prop. 1(i)), used for the split-KV merge and the shared-prefix
// cascade merge.  Partials are FP32; to make the result a function of the SET of partials
// (any slot order, any grouping, any level order gives the same bits) each element is
// summed on an integer grid declared before the reduction (Eq. 3 / Prop. 2): the largest
// magnitude among the C terms is found with an order-free integer maximum over their bit
// patterns, the grid is alpha = 2^(61 - ceil(log2 C) - e_max - 1), every term is rounded to
// nearest-even on it (exactly, through a double) and added as a 64-bit integer.
#pragma once

#include "fold_common.cuh"

namespace fold {

constexpr int kMergeSlices = 4;
constexpr int kMergeCache = 8;

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

// log2(alpha) for C terms whose largest magnitude has bit pattern maxbits (sign cleared).
__device__ __forceinline__ int grid_shift(unsigned maxbits, unsigned C) {
  const int ef = (int)(maxbits >> 23);
  const int e_max = ef == 0 ? -126 : ef - 127;
  return 61 - (ceil_log2_u32(C) + e_max + 1);
}
__device__ __forceinline__ double pow2_double(int e) {       // 2^e, e in the normal range
  return __longlong_as_double((long long)(e + 1023) << 52);
}

// grid (Hq, batch); block (D, kMergeSlices).  Thread (x, y): element x of A (and, for
// x == 0, L as well) over the slots k = y, y + kMergeSlices, ... of the flattened slot list
// of all levels.  The first kMergeCache terms of a thread stay in registers between the two
// passes; longer lists are read again.
__global__ void __launch_bounds__(128 * kMergeSlices) fold_merge_kernel(const MergeParams p) {
  __shared__ unsigned s_max[129];
  __shared__ unsigned long long s_sum[129];
  __shared__ float s_l;
  __shared__ int s_flags;
  const int h = blockIdx.x, b = blockIdx.y;
  const int x = threadIdx.x, y = threadIdx.y;
  const int D = p.D, G = p.G, kvh = h / G;
  const int tid = y * D + x;

  for (int i = tid; i <= D; i += D * kMergeSlices) { s_max[i] = 0u; s_sum[i] = 0ull; }
  if (tid == 0) s_flags = 0;

  const float *lbase[kMaxLevels];
  const float *llbase[kMaxLevels];
  long long lstride[kMaxLevels];
  int cnt[kMaxLevels];
  unsigned C = 0;
#pragma unroll
  for (int l = 0; l < kMaxLevels; ++l) {
    cnt[l] = 0; lbase[l] = nullptr; llbase[l] = nullptr; lstride[l] = 0;
    if (l < p.n_levels) {
      const MergeLevel &L = p.lv[l];
      const int seq = b / L.stack;
      int n = L.seqlens[seq];
      n = n < 0 ? 0 : (n > L.max_seqlen ? L.max_seqlen : n);
      cnt[l] = num_chunks_of(n);
      C += cnt[l];
      const int r = (b % L.stack) * G + (h % G);
      const float *s0 = L.slots + ((long long)seq * p.Hkv + kvh) * L.max_slots * L.slot_stride;
      lbase[l] = s0 + (long long)r * D + x;
      llbase[l] = s0 + (long long)L.rows * D + r;
      lstride[l] = L.slot_stride;
    }
  }
  // term t of this thread is flattened slot y + t * kMergeSlices
  auto locate = [&](int k, const float *&pa, const float *&pl) {
    int l = 0;
#pragma unroll
    for (int i = 0; i < kMaxLevels - 1; ++i)
      if (l == i && k >= cnt[i]) { k -= cnt[i]; l = i + 1; }
    pa = lbase[l] + k * lstride[l];
    pl = llbase[l] + k * lstride[l];
  };
  const int my_terms = ((int)C > y) ? ((int)C - y + kMergeSlices - 1) / kMergeSlices : 0;

  // pass 1: order-free maximum of |g| through the bit patterns
  float ca[kMergeCache], cl[kMergeCache];
  unsigned mx = 0u, mxl = 0u;
#pragma unroll
  for (int t = 0; t < kMergeCache; ++t) {
    ca[t] = 0.f; cl[t] = 0.f;
    if (t < my_terms) {
      const float *pa, *pl;
      locate(y + t * kMergeSlices, pa, pl);
      ca[t] = *pa;
      if (x == 0) cl[t] = *pl;
    }
  }
#pragma unroll
  for (int t = 0; t < kMergeCache; ++t) {
    mx = max(mx, __float_as_uint(ca[t]) & 0x7fffffffu);
    mxl = max(mxl, __float_as_uint(cl[t]) & 0x7fffffffu);
  }
  for (int t = kMergeCache; t < my_terms; ++t) {
    const float *pa, *pl;
    locate(y + t * kMergeSlices, pa, pl);
    mx = max(mx, __float_as_uint(*pa) & 0x7fffffffu);
    if (x == 0) mxl = max(mxl, __float_as_uint(*pl) & 0x7fffffffu);
  }
  __syncthreads();                                   // s_max / s_sum are zeroed
  if (mx) atomicMax(&s_max[x], mx);
  if (x == 0 && mxl) atomicMax(&s_max[D], mxl);
  __syncthreads();

  // pass 2: integer sums on the declared grid
  {
    const unsigned ma = s_max[x], ml = s_max[D];
    const double mul_a = pow2_double(grid_shift(ma, C)), mul_l = pow2_double(grid_shift(ml, C));
    const bool fin_a = (ma >> 23) != 255u, fin_l = (ml >> 23) != 255u;
    long long acc = 0, accl = 0;
#pragma unroll
    for (int t = 0; t < kMergeCache; ++t) {
      if (fin_a) acc += __double2ll_rn((double)ca[t] * mul_a);
      if (x == 0 && fin_l) accl += __double2ll_rn((double)cl[t] * mul_l);
    }
    for (int t = kMergeCache; t < my_terms; ++t) {
      const float *pa, *pl;
      locate(y + t * kMergeSlices, pa, pl);
      if (fin_a) acc += __double2ll_rn((double)*pa * mul_a);
      if (x == 0 && fin_l) accl += __double2ll_rn((double)*pl * mul_l);
    }
    if (acc) atomicAdd(&s_sum[x], (unsigned long long)acc);
    if (x == 0 && accl) atomicAdd(&s_sum[D], (unsigned long long)accl);
  }
  __syncthreads();

  if (y != 0) return;
  const long long row = (long long)b * p.Hq + h;
  if (x == 0) {
    const unsigned ml = s_max[D];
    float Lf;
    if ((ml >> 23) == 255u) Lf = __int_as_float(0x7fc00000);
    else Lf = (float)((double)(long long)s_sum[D] * pow2_double(-grid_shift(ml, C)));
    s_l = Lf;
  }
  // only the y == 0 threads are left: a named barrier over those D threads
  asm volatile("bar.sync 2, %0;" ::"r"(D) : "memory");
  const float Lf = s_l;
  const unsigned ma = s_max[x];
  float Af;
  if ((ma >> 23) == 255u) Af = __int_as_float(0x7fc00000);
  else Af = (float)((double)(long long)s_sum[x] * pow2_double(-grid_shift(ma, C)));
  float ov = C == 0 ? 0.f : Af / Lf;
  p.out[row * D + x] = __float2bfloat16_rn(ov);
  if (!(fabsf(ov) <= 3.4e38f)) atomicOr(&s_flags, FOLD_ROW_NONFINITE);
  asm volatile("bar.sync 2, %0;" ::"r"(D) : "memory");
  if (x == 0) {
    int flags = s_flags;
    float lse;
    if (C == 0) {
      flags = FOLD_ROW_EMPTY;
      lse = -INFINITY;
    } else {
      if (!(fabsf(Lf) <= 3.4e38f)) flags |= FOLD_ROW_NONFINITE;
      if (!(Lf >= 0.5f && Lf <= 1.2676506e30f)) flags |= FOLD_ROW_RANGE;      // [2^-1, 2^100]
      lse = p.z[row] + log2f(Lf);
    }
    if (p.lse) p.lse[row] = lse;
    if (p.row_status) p.row_status[row] = flags;
  }
}

}  // namespace fold
