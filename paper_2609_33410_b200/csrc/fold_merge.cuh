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

constexpr int kMergeMaxWarps = 8;

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

// grid (Hq, batch); block (32, W), W = blockDim.y <= kMergeMaxWarps chosen from the slot count.  One CTA
// per (request, q head).  Lane x of every warp owns EPT = D / 32 consecutive elements of A (one vector load
// per slot); warp y takes the slots y, y + W, ... of every level; lane 0 also carries L.  Two passes over
// the (cache-resident) slots: the order-free maximum, then the integer sum; warps combine through
// shared-memory integer atomics, which are order-free by construction.
template <int EPT>
__global__ void __launch_bounds__(32 * kMergeMaxWarps) fold_merge_kernel(const MergeParams p) {
  __shared__ unsigned s_max[129];
  __shared__ unsigned long long s_sum[129];
  __shared__ int s_flags;
  constexpr int D = 32 * EPT;
  const int h = blockIdx.x, b = blockIdx.y;
  const int x = threadIdx.x, y = threadIdx.y, W = blockDim.y;
  const int G = p.G, kvh = h / G;
  const int tid = y * 32 + x;
  const long long row = (long long)b * p.Hq + h;
  pdl_wait();                                        // slots and z come from the kernels before
  const float zrow = p.z[row];                       // requested early: only needed at the very end

  for (int i = tid; i <= D; i += 32 * W) { s_max[i] = 0u; s_sum[i] = 0ull; }
  if (tid == 0) s_flags = 0;

  // per level: this lane's first A vector, the row's L element, the slot stride and count
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
      pa[l] = s0 + r * D + x * EPT;
      pl[l] = s0 + L.rows * D + r;
      step[l] = L.slot_stride * W;
    }
  }
  const int clog2C = ceil_log2_u32(C);

  auto load_vec = [](const float *a, float (&v)[EPT]) {
    if (EPT == 4) {
      const float4 t = *reinterpret_cast<const float4 *>(a);
      v[0] = t.x; v[1] = t.y; v[EPT - 2] = t.z; v[EPT - 1] = t.w;
    } else {
      const float2 t = *reinterpret_cast<const float2 *>(a);
      v[0] = t.x; v[1] = t.y;
    }
  };

  // pass 1: order-free maximum of |g| through the bit patterns
  unsigned mx[EPT], mxl = 0u;
#pragma unroll
  for (int e = 0; e < EPT; ++e) mx[e] = 0u;
#pragma unroll
  for (int l = 0; l < kMaxLevels; ++l) {
    const float *a = pa[l], *q = pl[l];
#pragma unroll 4
    for (int k = y; k < cnt[l]; k += W, a += step[l], q += step[l]) {
      float v[EPT];
      load_vec(a, v);
#pragma unroll
      for (int e = 0; e < EPT; ++e) mx[e] = max(mx[e], __float_as_uint(v[e]) & 0x7fffffffu);
      if (x == 0) mxl = max(mxl, __float_as_uint(*q) & 0x7fffffffu);
    }
  }
  __syncthreads();                                   // s_max / s_sum are zeroed
  if (W > 1) {
#pragma unroll
    for (int e = 0; e < EPT; ++e) if (mx[e]) atomicMax(&s_max[x * EPT + e], mx[e]);
    if (x == 0 && mxl) atomicMax(&s_max[D], mxl);
    __syncthreads();
#pragma unroll
    for (int e = 0; e < EPT; ++e) mx[e] = s_max[x * EPT + e];
    mxl = s_max[D];
  }
  mxl = __shfl_sync(0xffffffffu, mxl, 0);

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
#pragma unroll
  for (int l = 0; l < kMaxLevels; ++l) {
    const float *a = pa[l], *q = pl[l];
#pragma unroll 4
    for (int k = y; k < cnt[l]; k += W, a += step[l], q += step[l]) {
      float v[EPT];
      load_vec(a, v);
#pragma unroll
      for (int e = 0; e < EPT; ++e) if (fin[e]) acc[e] += to_grid(v[e], alpha[e]);
      if (x == 0 && fin_l) accl += to_grid(*q, alpha_l);
    }
  }
  if (W > 1) {
#pragma unroll
    for (int e = 0; e < EPT; ++e) if (acc[e]) atomicAdd(&s_sum[x * EPT + e], (unsigned long long)acc[e]);
    if (x == 0 && accl) atomicAdd(&s_sum[D], (unsigned long long)accl);
    __syncthreads();
    if (y != 0) return;
#pragma unroll
    for (int e = 0; e < EPT; ++e) acc[e] = (long long)s_sum[x * EPT + e];
    accl = (long long)s_sum[D];
  }

  // warp 0 finishes the row
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

}  // namespace fold
