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

constexpr int kMergeSlices = 8;

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
// x == 0, L as well) over the slots k = y, y + kMergeSlices, ...
__global__ void __launch_bounds__(1024) fold_merge_kernel(const MergeParams p) {
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
  int cnt[kMaxLevels];
  unsigned C = 0;
  for (int l = 0; l < p.n_levels; ++l) {
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
  }
  __syncthreads();

  // pass 1: order-free maximum of |g| through the bit patterns
  unsigned mx = 0u, mxl = 0u;
  for (int l = 0; l < p.n_levels; ++l) {
    const long long st = p.lv[l].slot_stride;
    for (int k = y; k < cnt[l]; k += kMergeSlices) {
      mx = max(mx, __float_as_uint(lbase[l][k * st]) & 0x7fffffffu);
      if (x == 0) mxl = max(mxl, __float_as_uint(llbase[l][k * st]) & 0x7fffffffu);
    }
  }
  atomicMax(&s_max[x], mx);
  if (x == 0) atomicMax(&s_max[D], mxl);
  __syncthreads();

  // pass 2: integer sums on the declared grid
  {
    const unsigned ma = s_max[x], ml = s_max[D];
    const int sh_a = grid_shift(ma, C), sh_l = grid_shift(ml, C);
    const double mul_a = pow2_double(sh_a), mul_l = pow2_double(sh_l);
    const bool fin_a = (ma >> 23) != 255u, fin_l = (ml >> 23) != 255u;
    long long acc = 0, accl = 0;
    for (int l = 0; l < p.n_levels; ++l) {
      const long long st = p.lv[l].slot_stride;
      for (int k = y; k < cnt[l]; k += kMergeSlices) {
        if (fin_a) acc += __double2ll_rn((double)lbase[l][k * st] * mul_a);
        if (x == 0 && fin_l) accl += __double2ll_rn((double)llbase[l][k * st] * mul_l);
      }
    }
    atomicAdd(&s_sum[x], (unsigned long long)acc);
    if (x == 0) atomicAdd(&s_sum[D], (unsigned long long)accl);
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
  // every y == 0 thread passes the same barrier count: use a named barrier over D threads
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
