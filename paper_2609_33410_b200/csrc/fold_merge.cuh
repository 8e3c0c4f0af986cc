// Order-free partial add (Prop. 1(i)), used for the split-KV merge and the shared-prefix
// cascade merge.  Partials are FP32; to make the result a function of the SET of partials
// (any slot order, any grouping, any level order gives the same bits) each element is
// summed on an integer grid declared before the reduction (Eq. 3 / Prop. 2): the largest
// magnitude among the C terms is found with an order-free integer maximum over their bit
// patterns, the grid is alpha = 2^(61 - ceil(log2 C) - e_max - 1) (e_max >= -126: subnormal maxima
// use their fixed scale), every term is rounded to nearest-even on it with integer shifts of its
// mantissa and added as a 64-bit integer.
#pragma once

#include "fold_common.cuh"

namespace fold {

constexpr int kMergeMaxSlices = 8;

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

// Biased exponent of a bit pattern with subnormals counted as exponent 1 (their scale).
__device__ __forceinline__ int norm_exp(unsigned bits) {
  const int e = (int)((bits >> 23) & 0xffu);
  return e == 0 ? 1 : e;
}
// RNE(alpha * g) as an exact integer, alpha = 2^(61 - clog2C - (eb_max - 127) - 1): with g = m * 2^(e - 150),
// alpha * g = m * 2^(e - eb_max + 37 - clog2C).  Integer shifts only; |result| < 2^61 / C.
__device__ __forceinline__ long long to_grid(float g, int eb_max, int clog2C) {
  const unsigned u = __float_as_uint(g);
  const int e = (int)((u >> 23) & 0xffu);
  unsigned m = u & 0x7fffffu;
  if (e != 0) m |= 0x800000u;
  const int s = (e == 0 ? 1 : e) - eb_max + 37 - clog2C;
  long long v;
  if (s >= 0) {
    v = (long long)m << s;
  } else if (s < -25) {
    v = 0;
  } else {
    const int r = -s;
    unsigned q = m >> r;
    const unsigned rem = m & ((1u << r) - 1u), half = 1u << (r - 1);
    if (rem > half || (rem == half && (q & 1u))) ++q;
    v = q;
  }
  return (u >> 31) ? -v : v;
}
__device__ __forceinline__ float from_grid(long long sum, int eb_max, int clog2C) {
  // alpha^-1 = 2^-(187 - clog2C - eb_max); exponent stays inside the double range
  const int sh = 187 - clog2C - eb_max;
  return (float)((double)sum * __longlong_as_double((long long)(1023 - sh) << 52));
}

// grid (Hq, batch); block (D, S), S = blockDim.y <= kMergeMaxSlices chosen from the slot count.
// Thread (x, y): element x of A over the slots y, y + S, ... of every level; the x == 0 threads
// also carry L.  Two passes over the (cache-resident) slots: the maximum, then the integer sum.
__global__ void __launch_bounds__(128 * kMergeMaxSlices) fold_merge_kernel(const MergeParams p) {
  __shared__ unsigned s_max[129];
  __shared__ unsigned long long s_sum[129];
  __shared__ float s_l;
  __shared__ int s_flags;
  const int h = blockIdx.x, b = blockIdx.y;
  const int x = threadIdx.x, y = threadIdx.y, S = blockDim.y;
  const int D = p.D, G = p.G, kvh = h / G;
  const int tid = y * D + x;
  const long long row = (long long)b * p.Hq + h;
  pdl_wait();                                        // slots and z come from the kernels before
  const float zrow = p.z[row];                       // requested early: only needed at the very end

  for (int i = tid; i <= D; i += D * S) { s_max[i] = 0u; s_sum[i] = 0ull; }
  if (tid == 0) s_flags = 0;

  // per level: this thread's first A element, the row's L element, the slot stride and count
  const float *pa[kMaxLevels], *pl[kMaxLevels];
  long long step[kMaxLevels];
  int cnt[kMaxLevels];
  unsigned C = 0;
#pragma unroll
  for (int l = 0; l < kMaxLevels; ++l) {
    cnt[l] = 0; pa[l] = nullptr; pl[l] = nullptr; step[l] = 0;
    if (l < p.n_levels) {
      const MergeLevel &L = p.lv[l];
      const int seq = b / L.stack;
      int n = L.seqlens[seq];
      n = n < 0 ? 0 : (n > L.max_seqlen ? L.max_seqlen : n);
      cnt[l] = num_chunks_of(n);
      C += cnt[l];
      const int r = (b % L.stack) * G + (h % G);
      const float *s0 = L.slots + (((long long)seq * p.Hkv + kvh) * L.max_slots + y) * L.slot_stride;
      pa[l] = s0 + r * D + x;
      pl[l] = s0 + L.rows * D + r;
      step[l] = L.slot_stride * S;
    }
  }
  const int clog2C = ceil_log2_u32(C);

  // pass 1: order-free maximum of |g| through the bit patterns
  unsigned mx = 0u, mxl = 0u;
#pragma unroll
  for (int l = 0; l < kMaxLevels; ++l) {
    const float *a = pa[l];
#pragma unroll 4
    for (int k = y; k < cnt[l]; k += S, a += step[l]) mx = max(mx, __float_as_uint(*a) & 0x7fffffffu);
    if (x == 0) {
      const float *q = pl[l];
      for (int k = y; k < cnt[l]; k += S, q += step[l]) mxl = max(mxl, __float_as_uint(*q) & 0x7fffffffu);
    }
  }
  __syncthreads();                                   // s_max / s_sum are zeroed
  if (mx) atomicMax(&s_max[x], mx);
  if (x == 0 && mxl) atomicMax(&s_max[D], mxl);
  __syncthreads();

  // pass 2: integer sums on the declared grid
  {
    const unsigned ma = s_max[x], ml = s_max[D];
    const int eb_a = norm_exp(ma), eb_l = norm_exp(ml);
    const bool fin_a = (ma >> 23) != 255u, fin_l = (ml >> 23) != 255u;
    long long acc = 0, accl = 0;
#pragma unroll
    for (int l = 0; l < kMaxLevels; ++l) {
      const float *a = pa[l];
      if (fin_a) {
#pragma unroll 4
        for (int k = y; k < cnt[l]; k += S, a += step[l]) acc += to_grid(*a, eb_a, clog2C);
      }
      if (x == 0 && fin_l) {
        const float *q = pl[l];
        for (int k = y; k < cnt[l]; k += S, q += step[l]) accl += to_grid(*q, eb_l, clog2C);
      }
    }
    if (acc) atomicAdd(&s_sum[x], (unsigned long long)acc);
    if (x == 0 && accl) atomicAdd(&s_sum[D], (unsigned long long)accl);
  }
  __syncthreads();

  if (y != 0) return;
  if (x == 0) {
    const unsigned ml = s_max[D];
    s_l = (ml >> 23) == 255u ? __int_as_float(0x7fc00000) : from_grid((long long)s_sum[D], norm_exp(ml), clog2C);
  }
  // only the y == 0 threads are left: a named barrier over those D threads
  asm volatile("bar.sync 2, %0;" ::"r"(D) : "memory");
  const float Lf = s_l;
  const unsigned ma = s_max[x];
  const float Af = (ma >> 23) == 255u ? __int_as_float(0x7fc00000) : from_grid((long long)s_sum[x], norm_exp(ma), clog2C);
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
      lse = zrow + log2f(Lf);
    }
    if (p.lse) p.lse[row] = lse;
    if (p.row_status) p.row_status[row] = flags;
  }
}

}  // namespace fold
